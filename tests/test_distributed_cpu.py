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


# ---- coordinate-sharded deployment: the ranges and the exchange of the l1 parts ---------------

def test_range_partition_covers_the_coordinates_with_aligned_cuts():
    for d, world, align in ((112000, 3, 4096), (110_000_000, 8, 16384), (65536, 4, 16384), (1_500_000_000, 8, 16384),
                            (100, 2, 64)):
        cuts = [dd.range_partition(d, world, r, align) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == d
        for (a, b), (c, e) in zip(cuts, cuts[1:]):
            assert b == c and b % align == 0 and a < b
        sizes = [b - a for a, b in cuts[:-1]]
        assert max(sizes) - min(sizes) <= align
    with pytest.raises(ValueError):
        dd.range_partition(100, 4, 0, 64)               # fewer aligned units than ranges
    with pytest.raises(ValueError):
        dd.range_partition(1000, 2, 2, 64)


def _sums_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n, q = 3, 4
    # the exchange buffer as the library lays it out: [ranks, n, q, 2] doubles, own slot filled
    sums = torch.full((world, n, q, 2), float("nan"), dtype=torch.float64)
    sums[rank] = _own_sums(rank, n, q)
    dd.gather_range_sums(sums)
    # what every process then does with them (in the library's kernel): add range by range
    total = torch.zeros(n, q, dtype=torch.float64)
    for r in range(world):
        total = total + sums[r, :, :, 0]
    torch.save({"sums": sums, "total": total}, os.path.join(out_dir, "s%d.pt" % rank))
    dist.barrier()
    dist.destroy_process_group()


def _own_sums(rank, n, q):
    # values whose sum depends on the order of the additions in binary64
    base = torch.tensor([1e16, 1.0, -1e16, 3.0], dtype=torch.float64)[rank % 4]
    t = torch.zeros(n, q, 2, dtype=torch.float64)
    t[:, :, 0] = base + torch.arange(n * q, dtype=torch.float64).view(n, q)
    t[:, :, 1] = 2.0 ** -60 * (rank + 1)
    return t


@pytest.mark.parametrize("world", [2, 3])
def test_l1_parts_are_gathered_slot_by_slot_and_added_in_rank_order(world, tmp_path):
    port = 27000 + (os.getpid() * 11 + world * 17) % 3000
    mp.spawn(_sums_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(os.path.join(str(tmp_path), "s%d.pt" % r)) for r in range(world)]
    want = torch.stack([_own_sums(r, 3, 4) for r in range(world)])
    for got in res:
        assert torch.equal(got["sums"], want)           # slot r holds rank r's parts, bit for bit
        assert torch.equal(got["total"], res[0]["total"])   # the same additions everywhere


def _hist_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # the top-k exchange buffer: [ranks, rows * 2048] words, own slot filled (histogram counts)
    buf = torch.full((world, 2 * 2048), -1, dtype=torch.int32)
    buf[rank] = torch.arange(2 * 2048, dtype=torch.int32) * (rank + 1)
    dd.gather_range_sums(buf)
    torch.save(buf, os.path.join(out_dir, "h%d.pt" % rank))
    dist.barrier()
    dist.destroy_process_group()


def test_topk_histogram_slots_are_gathered_in_place(tmp_path):
    world = 3
    port = 25000 + (os.getpid() * 5) % 1500
    mp.spawn(_hist_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    want = torch.stack([torch.arange(2 * 2048, dtype=torch.int32) * (r + 1) for r in range(world)])
    for r in range(world):
        assert torch.equal(torch.load(os.path.join(str(tmp_path), "h%d.pt" % r)), want)
    # summed over the ranges (what the next stage does) every process gets the same histogram
    assert torch.equal(want.sum(0), torch.arange(2 * 2048, dtype=torch.int32) * 6)
