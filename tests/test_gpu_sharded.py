"""Distributed deployment on one GPU: the processes of a deployment are emulated by separate
contexts whose kernels run one after the other on one stream; device copies of the message
rows stand in for the collectives (nothing waits on anything else).  The result must be that
of one context holding all n workers and of the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2111_00705_b200 import binding as cd
from paper_2111_00705_b200 import distributed as dd
from paper_2111_00705_b200 import synth

pytestmark = pytest.mark.gpu


def u32(t):
    return t.cpu().numpy().view(np.uint32)


def make_shards(w, world, server_rank, x0, mode=cd.MARKOV):
    out = []
    for r in range(world):
        first, per = dd.partition(w.n, world, r, server_rank)
        out.append(cd.CDAdamShard(w.d, w.n, first, per, beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps,
                                  offsets=w.offsets, x0=x0.cuda(), mode=mode, compressor=w.compressor, k=w.k))
    return out


def emulated_step(shards, grads, server_rank):
    """One iteration over all emulated processes; returns nothing, state lives in the contexts."""
    for s in shards:
        lo, hi = s.first_worker, s.first_worker + s.n_local
        s.step_workers(grads[lo:hi].contiguous().reshape(-1) if s.n_local else None)
    bufs = [s.exchange_buffers() for s in shards]
    receivers = range(len(shards)) if server_rank is None else [server_rank]
    for r in receivers:                                 # the gather of the worker messages
        for s, b in zip(shards, bufs):
            lo, hi = s.first_worker, s.first_worker + s.n_local
            if s is not shards[r] and s.n_local:
                bufs[r]["worker_bits"][lo:hi].copy_(b["worker_bits"][lo:hi])
                bufs[r]["worker_scales"][lo:hi].copy_(b["worker_scales"][lo:hi])
    for r in receivers:
        shards[r].step_server()
    if server_rank is not None:                         # the server's broadcast
        for r, b in enumerate(bufs):
            if r != server_rank:
                b["server_bits"].copy_(bufs[server_rank]["server_bits"])
                b["server_scales"].copy_(bufs[server_rank]["server_scales"])
    for s in shards:
        s.step_update()


def run_case(w, world, server_rank, steps, mode=cd.MARKOV):
    x0 = w.x0("cpu")
    shards = make_shards(w, world, server_rank, x0, mode)
    args = dict(beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps)
    full = cd.CDAdam(w.d, w.n, w.compressor, k=w.k, offsets=w.offsets, x0=x0.cuda(), mode=mode, **args)
    o = orc.Oracle(w.d, w.n, w.compressor, k=w.k, offsets=w.offsets, x0=x0.numpy(), mode=mode, **args)
    for t in range(1, steps + 1):
        grads = w.grads(t, "cpu")
        gd = grads.cuda().reshape(w.n, w.d)
        emulated_step(shards, gd, server_rank)
        full.step(gd.reshape(-1))
        o.step(grads.numpy())
        torch.cuda.synchronize()
        holder = shards[server_rank if server_rank is not None else 0]
        for who in list(range(w.n)) + [cd.SERVER]:
            oa, ob = o.payload(who)
            a, b = holder.last_payload(who)
            assert np.array_equal(u32(a), oa) and np.array_equal(u32(b), ob.view(np.uint32)), (t, who)
        for s in shards:
            assert s.step_count() == t
            for name in ("gtil", "m", "v", "vhat", "x"):
                got = s.get_state(name).cpu().numpy()
                assert np.array_equal(got, o.state(name).ravel()), (t, name, s.first_worker)
                assert np.array_equal(got, full.get_state(name).cpu().numpy()), (t, name)
            if s.n_local and (t % 2 == 0 or t == steps):     # alternate: deferred and materialised worker state
                lo, hi = s.first_worker, s.first_worker + s.n_local
                assert np.array_equal(s.get_state("ghat_w").cpu().numpy(), o.state("ghat_w")[lo:hi]), (t, lo)
        if mode == cd.MARKOV:
            assert np.array_equal(holder.get_state("ghat_s").cpu().numpy(), o.state("ghat_s").ravel())
    for s in shards:
        s.device_status()
        s.close()
    full.close(); o.close()


@pytest.mark.parametrize("world,server_rank", [(2, None), (4, None), (3, 1), (5, 0)])
def test_sharded_iteration_equals_the_single_context_and_the_oracle(world, server_rank):
    w = synth.workload("C2", scale=0.01, steps=4)       # d = 112,000, n = 8, 62 unaligned segments
    run_case(w, world, server_rank, 4)


def test_sharded_flat_ragged_dimension_and_one_wave_grids():
    w = synth.workload("C1", scale=0.5, steps=4)        # launch-bound size: scales finished inside the passes
    w.d -= 13                                           # d % 32 != 0, rows not 16-byte aligned
    run_case(w, 2, None, 4)
    run_case(w, 3, 2, 3)


def test_sharded_large_tiles_use_the_prefetch_ring():
    w = synth.workload("C4", scale=0.01, steps=3)       # d = 1.1 M
    x0 = w.x0("cpu")
    shards = make_shards(w, 2, None, x0)
    for s in shards:
        s.set_tile(16384)                               # the tile of the full-size workload
    o = orc.Oracle(w.d, w.n, orc.SIGN, offsets=w.offsets, x0=x0.numpy(), beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps)
    for t in range(1, 4):
        grads = w.grads(t, "cpu")
        emulated_step(shards, grads.cuda().reshape(w.n, w.d), None)
        o.step(grads.numpy())
    for s in shards:
        assert np.array_equal(s.get_state("x").cpu().numpy(), o.state("x").ravel())
        lo, hi = s.first_worker, s.first_worker + s.n_local
        assert np.array_equal(s.get_state("ghat_w").cpu().numpy(), o.state("ghat_w")[lo:hi])
        s.close()
    o.close()


def test_sharded_error_feedback_mode():
    w = synth.workload("C2", scale=0.005, steps=3)
    run_case(w, 2, None, 3, mode=cd.EF)


@pytest.mark.parametrize("world,server_rank", [(2, None), (4, None), (3, 0), (5, 2)])
def test_sharded_top_k_equals_the_single_context_and_the_oracle(world, server_rank):
    w = synth.workload("C3", scale=0.004, steps=4)      # d = 102,400, n = 16, k = 1,024
    run_case(w, world, server_rank, 4)


def test_sharded_top_k_ties_and_ragged_dimension():
    w = synth.workload("C3", scale=0.001, steps=3)
    w.d -= 7
    w.n, w.k = 4, 300
    w.grads = lambda t, device="cpu", d=w.d, n=w.n: torch.randint(-3, 4, (n, d), generator=torch.Generator().manual_seed(t)).float().to(device)
    run_case(w, 2, None, 3)
    run_case(w, 3, 1, 3)


def test_staged_top_k_on_a_context_with_all_workers():
    w = synth.workload("C3", scale=0.002, steps=3)
    x0 = w.x0("cpu")
    s = cd.CDAdamShard(w.d, w.n, 0, w.n, x0=x0.cuda(), compressor=cd.TOPK, k=w.k)
    o = orc.Oracle(w.d, w.n, orc.TOPK, k=w.k, x0=x0.numpy())
    for t in range(1, 4):
        grads = w.grads(t, "cpu")
        s.step_workers(grads.cuda().reshape(-1)); s.step_server(); s.step_update()
        o.step(grads.numpy())
        for name in ("x", "gtil", "ghat_s", "ghat_w"):
            assert np.array_equal(s.get_state(name).cpu().numpy().ravel(), o.state(name).ravel()), (t, name)
    s.close(); o.close()


def test_staged_calls_on_a_context_with_all_workers_and_call_order():
    w = synth.workload("C1", scale=0.25, steps=3)
    x0 = w.x0("cpu")
    s = cd.CDAdamShard(w.d, w.n, 0, w.n, x0=x0.cuda())
    o = orc.Oracle(w.d, w.n, orc.SIGN, x0=x0.numpy())
    with pytest.raises(cd.CdadamError):
        s.step_server()                                  # no worker stage yet
    with pytest.raises(cd.CdadamError):
        s.step_update()
    for t in range(1, 4):
        grads = w.grads(t, "cpu")
        g = grads.cuda().reshape(-1)
        if t == 2:
            s.step(g)                                    # the one-call step and the stages mix freely between iterations
        else:
            s.step_workers(g)
            with pytest.raises(cd.CdadamError):
                s.step_workers(g)                        # the iteration is not complete
            with pytest.raises(cd.CdadamError):
                s.step(g)
            s.step_server()
            with pytest.raises(cd.CdadamError):
                s.step_server()
            s.step_update()
        o.step(grads.numpy())
        assert np.array_equal(s.get_state("x").cpu().numpy(), o.state("x").ravel())
    s.close(); o.close()
    part = cd.CDAdamShard(w.d, w.n, 1, 2, x0=x0.cuda())
    with pytest.raises(cd.CdadamError):
        part.step(w.grads(1, "cuda").reshape(-1))        # a part of the workers: staged calls only
    part.close()
    lib = cd.lib()
    assert not lib.cdadam_create_shard(100, 4, 3, 2, cd.SIGN, 0, 0.9, 0.999, 1e-3, 1e-8)     # workers 3, 4 of 4
    assert not lib.cdadam_create_shard(100, 4, -1, 2, cd.SIGN, 0, 0.9, 0.999, 1e-3, 1e-8)
    assert not lib.cdadam_create_shard(100, 4, 0, 2, cd.IDENTITY, 0, 0.9, 0.999, 1e-3, 1e-8)
    assert not lib.cdadam_create_shard(100, 4, 0, 2, cd.TOPK, 0, 0.9, 0.999, 1e-3, 1e-8)     # k out of range


def test_distributed_class_over_a_one_rank_nccl_group(tmp_path):
    """The deployment class end to end (stages, in-place all-gather on the library's buffers)
    with NCCL on a group of one process; more ranks need more GPUs."""
    import torch.distributed as dist
    w = synth.workload("C2", scale=0.01, steps=3)
    x0 = w.x0("cpu")
    try:
        dist.init_process_group("nccl", init_method="file://" + str(tmp_path / "rendezvous"), rank=0, world_size=1,
                                device_id=torch.device("cuda", torch.cuda.current_device()))
    except Exception as exc:                       # no usable NCCL on this machine: nothing of ours to test
        pytest.skip("NCCL process group could not be created: %s" % exc)
    try:
        opt = dd.DistributedCDAdam(w.d, w.n, offsets=w.offsets, x0=x0.cuda())
        o = orc.Oracle(w.d, w.n, orc.SIGN, offsets=w.offsets, x0=x0.numpy())
        for t in range(1, 4):
            grads = w.grads(t, "cpu")
            opt.step(grads.cuda().reshape(-1))
            o.step(grads.numpy())
            torch.cuda.synchronize()
            assert np.array_equal(opt.params().cpu().numpy(), o.state("x").ravel()), t
        assert np.array_equal(opt.shard.get_state("ghat_w").cpu().numpy(), o.state("ghat_w"))
        opt.close(); o.close()
    finally:
        dist.destroy_process_group()
