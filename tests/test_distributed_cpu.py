"""The distributed deployment's host logic on CPU: which process holds which workers, and
that the message exchange delivers every row (gloo, world sizes 2 and 3).  The tensors stand
for the library's message buffers (n x words sign words, n x q scales)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2111_00705_b200 import distributed as dd

N, WORDS, Q = 4, 5, 3


def test_partition_deals_equal_contiguous_blocks():
    assert [dd.partition(8, 4, r) for r in range(4)] == [(0, 2), (2, 2), (4, 2), (6, 2)]
    assert dd.partition(8, 1, 0) == (0, 8)
    # a separate server holds no worker; the others are numbered around it
    assert [dd.partition(8, 3, r, server_rank=1) for r in range(3)] == [(0, 4), (0, 0), (4, 4)]
    assert [dd.partition(6, 4, r, server_rank=0) for r in range(4)] == [(0, 0), (0, 2), (2, 2), (4, 2)]
    covered = sorted(j for r in range(5) for j in range(*(lambda f, p: (f, f + p))(*dd.partition(8, 5, r, server_rank=4))))
    assert covered == list(range(8))
    with pytest.raises(ValueError):
        dd.partition(7, 2, 0)
    with pytest.raises(ValueError):
        dd.partition(8, 1, 0, server_rank=0)
    with pytest.raises(ValueError):
        dd.partition(8, 2, 2)


def _row_bits(i):
    return (torch.arange(WORDS, dtype=torch.int64) * 7919 + i * 104729 - 2 ** 31).to(torch.int32)


def _row_scales(i):
    return torch.arange(Q, dtype=torch.float32) * 0.25 + i


def _rank_main(rank, world, port, server_rank, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    first, per = dd.partition(N, world, rank, server_rank)
    bits = torch.full((N, WORDS), -1, dtype=torch.int32)
    scales = torch.full((N, Q), -1.0)
    for i in range(first, first + per):
        bits[i], scales[i] = _row_bits(i), _row_scales(i)
    dd.exchange_worker_messages(bits, scales, N, None, server_rank)
    sbits = torch.zeros(WORDS, dtype=torch.int32)
    sscales = torch.zeros(Q)
    if server_rank is not None:
        if rank == server_rank:
            sbits, sscales = _row_bits(99), _row_scales(99)
        dd.broadcast_server_message(sbits, sscales, None, server_rank)
    torch.save({"bits": bits, "scales": scales, "sbits": sbits, "sscales": sscales, "own": (first, per)},
               os.path.join(out_dir, "r%d.pt" % rank))
    dist.barrier()
    dist.destroy_process_group()


def _run(world, server_rank, tmp_path):
    port = 23000 + (os.getpid() * 7 + world * 13 + (server_rank or 0)) % 4000
    mp.spawn(_rank_main, args=(world, port, server_rank, str(tmp_path)), nprocs=world, join=True)
    return [torch.load(os.path.join(str(tmp_path), "r%d.pt" % r)) for r in range(world)]


def test_two_ranks_all_gather_every_worker_message(tmp_path):
    full_bits = torch.stack([_row_bits(i) for i in range(N)])
    full_scales = torch.stack([_row_scales(i) for i in range(N)])
    for got in _run(2, None, tmp_path):
        assert torch.equal(got["bits"], full_bits) and torch.equal(got["scales"], full_scales)


def test_three_ranks_with_a_server_gather_then_broadcast(tmp_path):
    full_bits = torch.stack([_row_bits(i) for i in range(N)])
    full_scales = torch.stack([_row_scales(i) for i in range(N)])
    res = _run(3, 1, tmp_path)
    assert torch.equal(res[1]["bits"], full_bits) and torch.equal(res[1]["scales"], full_scales)
    for r in (0, 2):                       # a worker process keeps its own rows and receives no others
        first, per = res[r]["own"]
        assert torch.equal(res[r]["bits"][first:first + per], full_bits[first:first + per])
        others = [i for i in range(N) if not first <= i < first + per]
        assert (res[r]["bits"][others] == -1).all()
    for got in res:                        # the server message reaches everyone
        assert torch.equal(got["sbits"], _row_bits(99)) and torch.equal(got["sscales"], _row_scales(99))
