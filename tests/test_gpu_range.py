"""Coordinate-sharded iteration on one GPU: the processes of such a deployment are emulated by
separate contexts, one per coordinate range, whose kernels run one after the other on one
stream; device copies of the l1 parts stand in for the two all-gathers (nothing waits on
anything else).  The result must be that of one context holding the whole problem and of the
CPU oracle, bit for bit: the scales on every range, the sign bits and every state vector on
the ranges put side by side."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2111_00705_b200 import binding as cd
from paper_2111_00705_b200 import distributed as dd
from paper_2111_00705_b200 import synth

pytestmark = pytest.mark.gpu


def unpack(words, count):
    w = words.cpu().numpy().view(np.uint32)
    j = np.arange(count)
    return ((w[j // 32] >> (j % 32)) & 1).astype(bool)


def make_ranges(w, cuts, x0, mode=cd.MARKOV, tile=0):
    out = []
    for r in range(len(cuts) - 1):
        lo, hi = cuts[r], cuts[r + 1]
        c = cd.CDAdamRange(w.d, w.n, lo, hi, r, len(cuts) - 1, beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps,
                           offsets=w.offsets, x0=x0[lo:hi].contiguous().cuda(), mode=mode)
        if tile:
            c.set_tile(tile)
        out.append(c)
    return out


def emulated_step(ranges, grads):
    """One iteration over all emulated processes.  grads: n x d on the device."""
    for c in ranges:
        c.range_workers(grads[:, c.lo:c.hi].contiguous().reshape(-1))
    for key, stage in (("worker_sums", "range_server"), ("server_sums", "range_update")):
        bufs = [c.range_buffers()[key] for c in ranges]
        for r, b in enumerate(bufs):                    # the all-gather: slot r comes from range r
            for other in bufs:
                if other is not b:
                    other[r].copy_(b[r])
        for c in ranges:
            getattr(c, stage)()


def run_case(w, cuts, steps, mode=cd.MARKOV, tile=0):
    x0 = w.x0("cpu")
    ranges = make_ranges(w, cuts, x0, mode, tile)
    args = dict(beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps)
    full = cd.CDAdam(w.d, w.n, cd.SIGN, offsets=w.offsets, x0=x0.cuda(), mode=mode, **args)
    o = orc.Oracle(w.d, w.n, orc.SIGN, offsets=w.offsets, x0=x0.numpy(), mode=mode, **args)
    off = np.array([0, w.d]) if w.offsets is None else np.asarray(w.offsets)
    for t in range(1, steps + 1):
        grads = w.grads(t, "cpu")
        gd = grads.cuda().reshape(w.n, w.d)
        emulated_step(ranges, gd)
        full.step(gd.reshape(-1))
        o.step(grads.numpy())
        torch.cuda.synchronize()
        for c in ranges:
            assert c.step_count() == t
            seg = c.range_buffers()["segment_of_local"].cpu().numpy()
            # the segments that meet [lo, hi), in order
            want = [r for r in range(off.size - 1) if off[r] < c.hi and off[r + 1] > c.lo]
            assert seg.tolist() == want and c.q == len(want)
            for who in list(range(w.n)) + [cd.SERVER]:
                obits, oscales = o.payload(who)
                bits, scales = c.last_payload(who)
                j = np.arange(c.lo, c.hi)
                assert np.array_equal(unpack(bits, c.d), ((obits[j // 32] >> (j % 32)) & 1).astype(bool)), (t, who, c.lo)
                assert np.array_equal(scales.cpu().numpy().view(np.uint32), oscales[seg].view(np.uint32)), (t, who, c.lo)
                fbits, fscales = full.last_payload(who)
                assert np.array_equal(scales.cpu().numpy().view(np.uint32), fscales.cpu().numpy()[seg].view(np.uint32))
            names = ("ghat_s", "gtil", "m", "v", "vhat", "x") if mode == cd.MARKOV else ("gtil", "m", "v", "vhat", "x")
            for name in names:
                got = c.get_state(name).cpu().numpy()
                assert np.array_equal(got, o.state(name)[c.lo:c.hi]), (t, name, c.lo)
            if t % 2 == 0 or t == steps:                # alternate: deferred and materialised worker state
                assert np.array_equal(c.get_state("ghat_w").cpu().numpy(), o.state("ghat_w")[:, c.lo:c.hi]), (t, c.lo)
        for name in ("x", "gtil"):
            side_by_side = torch.cat([c.get_state(name) for c in ranges])
            assert torch.equal(side_by_side, full.get_state(name)), (t, name)
    for c in ranges:
        c.device_status()
        c.close()
    full.close(); o.close()


@pytest.mark.parametrize("cuts", [(0, 57344, 112000), (0, 16384, 65536, 112000),
                                  (0, 20000, 40001, 60003, 99999, 112000)])
def test_coordinate_ranges_equal_the_single_context_and_the_oracle(cuts):
    """2, 3 and 5 ranges; tile-aligned cuts and cuts at odd coordinates (inside segments, not
    multiples of 4 or 32); 62 unaligned segments, so most cuts fall inside a segment and some
    ranges hold several whole segments."""
    w = synth.workload("C2", scale=0.01, steps=4)       # d = 112,000, n = 8
    assert w.d == 112000
    run_case(w, cuts, 4)


def test_coordinate_ranges_flat_ragged_dimension():
    """One segment shared by all ranges (every scale needs every range's part), d % 32 != 0."""
    w = synth.workload("C1", scale=0.5, steps=4)
    w.d -= 13
    run_case(w, (0, 8192, w.d), 4)
    run_case(w, (0, 1, 2, 30000, w.d), 3)               # ranges of a single coordinate


def test_coordinate_ranges_large_tiles_and_error_feedback():
    w = synth.workload("C4", scale=0.01, steps=3)       # d = 1.1 M, 15 segments
    lo, mid = dd.range_partition(w.d, 2, 0)
    run_case(w, (0, mid, w.d), 3, tile=16384)           # the prefetch-ring worker kernel on both ranges
    w = synth.workload("C2", scale=0.005, steps=3)
    run_case(w, (0, 30000, w.d), 3, mode=cd.EF)


def test_range_context_refuses_what_it_cannot_do():
    c = cd.CDAdamRange(1000, 2, 100, 600, 0, 2)
    g = torch.zeros(2 * 500, device="cuda")
    with pytest.raises(cd.CdadamError) as e:
        c.step(g)
    assert e.value.code == cd.ERR_STATE
    with pytest.raises(cd.CdadamError):
        c.range_server()                                # before the worker stage
    c.range_workers(g)
    with pytest.raises(cd.CdadamError):
        c.range_update()                                # before the server stage
    with pytest.raises(cd.CdadamError):
        c.get_state("ghat_w")                           # this iteration's scales are not known yet
    c.range_server(); c.range_update()
    assert c.step_count() == 1
    c.close()
    lib = cd.lib()
    for lo, hi, r, R in ((5, 5, 0, 1), (-1, 5, 0, 1), (0, 1001, 0, 1), (0, 10, 2, 2), (0, 10, 0, 0)):
        assert not lib.cdadam_create_range(1000, 2, lo, hi, r, R, cd.SIGN, 0, 0.9, 0.999, 1e-3, 1e-8)
    assert not lib.cdadam_create_range(1000, 2, 0, 10, 0, 1, cd.IDENTITY, 0, 0.9, 0.999, 1e-3, 1e-8)


def test_range_sharded_optimizer_over_a_one_rank_group():
    """RangeShardedCDAdam end to end (its own all-gathers) over an NCCL group of one process."""
    import os
    import torch.distributed as dist
    if dist.is_initialized():
        pytest.skip("a process group is already initialised in this process")
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", str(29650 + os.getpid() % 300))
    try:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    except Exception as exc:                            # no NCCL group can be created here
        pytest.skip("NCCL group unavailable: %s" % str(exc)[:80])
    try:
        w = synth.workload("C2", scale=0.005, steps=3)
        x0 = w.x0("cpu")
        opt = dd.RangeShardedCDAdam(w.d, w.n, offsets=w.offsets, x0=x0.cuda(), beta1=w.beta1, beta2=w.beta2,
                                    lr=w.lr, eps=w.eps)
        o = orc.Oracle(w.d, w.n, orc.SIGN, offsets=w.offsets, x0=x0.numpy(), beta1=w.beta1, beta2=w.beta2,
                       lr=w.lr, eps=w.eps)
        for t in range(1, 4):
            grads = w.grads(t, "cpu")
            opt.step(grads.cuda().reshape(-1))
            o.step(grads.numpy())
        torch.cuda.synchronize()
        assert np.array_equal(opt.params().cpu().numpy(), o.state("x"))
        opt.close(); o.close()
    finally:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------- top-k

def make_topk_ranges(w, cuts, x0):
    return [cd.CDAdamRange(w.d, w.n, cuts[r], cuts[r + 1], r, len(cuts) - 1, beta1=w.beta1, beta2=w.beta2, lr=w.lr,
                           eps=w.eps, x0=x0[cuts[r]:cuts[r + 1]].contiguous().cuda(), compressor=cd.TOPK, k=w.k)
            for r in range(len(cuts) - 1)]


def emulated_topk_step(ranges, grads):
    local = [grads[:, c.lo:c.hi].contiguous().reshape(-1) for c in ranges]
    for stage in range(cd.CDAdamRange.TOPK_STAGES):
        for c, g in zip(ranges, local):
            c.range_topk(stage, g if stage <= 4 else None)
        bufs = [c.range_topk_buffer(stage) for c in ranges]
        if bufs[0] is None:
            assert stage in (4, 9)
            continue
        for r, b in enumerate(bufs):                    # the all-gather: slot r comes from range r
            for other in bufs:
                if other is not b:
                    other[r].copy_(b[r])


def gathered_payload(ranges, who):
    """The message of `who` put together from the ranges: coordinates of the whole vector."""
    idx, val = [], []
    for c in ranges:
        i, v = c.last_payload(who)
        i = i.cpu().numpy().view(np.uint32); v = v.cpu().numpy()
        keep = i != 0xffffffff
        assert not keep[np.argmin(keep):].any() or keep.all()      # the marked entries come last
        assert np.all(np.diff(i[keep].astype(np.int64)) > 0) and (i[keep] < c.d).all()
        idx.append(i[keep].astype(np.int64) + c.lo); val.append(v[keep])
    return np.concatenate(idx), np.concatenate(val)


def run_topk_case(w, cuts, grads_of, steps):
    x0 = w.x0("cpu")
    ranges = make_topk_ranges(w, cuts, x0)
    o = orc.Oracle(w.d, w.n, orc.TOPK, k=w.k, x0=x0.numpy(), beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps)
    for t in range(1, steps + 1):
        grads = grads_of(t)
        emulated_topk_step(ranges, torch.from_numpy(grads).cuda().reshape(w.n, w.d))
        o.step(grads)
        torch.cuda.synchronize()
        for who in list(range(w.n)) + [cd.SERVER]:
            oi, ov = o.payload(who)
            gi, gv = gathered_payload(ranges, who)
            assert np.array_equal(gi, oi.astype(np.int64)), (t, who)
            assert np.array_equal(gv.view(np.uint32), ov.view(np.uint32)), (t, who)
        for c in ranges:
            assert c.step_count() == t
            for name in orc.STATE_NAMES:
                got = c.get_state(name).cpu().numpy()
                want = o.state(name)[..., c.lo:c.hi]
                assert np.array_equal(got, want), (t, name, c.lo)
    for c in ranges:
        c.device_status()
        c.close()
    o.close()


@pytest.mark.parametrize("cuts", [(0, 131072, 256000), (0, 4096, 100001, 256000), (0, 50000, 50001, 120000, 200003, 256000)])
def test_topk_coordinate_ranges_equal_the_oracle(cuts):
    """Top-k of the whole vector selected by 2, 3 and 5 ranges between them (the C3 recipe at
    d = 256,000, n = 16, k = 2,560): aligned and odd cuts, a range of one coordinate."""
    w = synth.workload("C3", scale=0.01, steps=3)
    assert w.d == 256000
    run_topk_case(w, cuts, lambda t: w.grads(t, "cpu").numpy(), 3)


def test_topk_coordinate_ranges_share_the_ties_in_coordinate_order():
    """Tie-dominated rows: few distinct magnitudes, so the k-th largest is shared by many
    coordinates in every range and the lower coordinates must win across the cuts; also all
    values equal, k = 1 and k = d."""
    rng = np.random.default_rng(17)
    d, n = 30000, 3
    cuts = (0, 7000, 7001, 20480, 30000)

    def tied(t):
        return (rng.integers(-3, 4, size=(n, d)) * 0.5).astype(np.float32)

    for k in (1, 2500, 29999, d):
        w = synth.Workload("TIES", d, n, synth.TOPK, 3, k=k)
        run_topk_case(w, cuts, tied, 3)
    w = synth.Workload("FLAT", d, n, synth.TOPK, 2, k=777)
    run_topk_case(w, cuts, lambda t: np.full((n, d), 1.5 * t, np.float32), 2)


def test_topk_range_context_refuses_wrong_stages():
    c = cd.CDAdamRange(10000, 2, 1000, 6000, 0, 2, compressor=cd.TOPK, k=50)
    g = torch.zeros(2 * 5000, device="cuda")
    with pytest.raises(cd.CdadamError) as e:
        c.range_topk(1, g)
    assert e.value.code == cd.ERR_STATE
    with pytest.raises(cd.CdadamError):
        c.range_workers(g)                              # the scaled-sign stages
    with pytest.raises(cd.CdadamError):
        c.step(g)
    c.range_topk(0, g)
    assert c.range_topk_buffer(0).shape == (2, 2 * 2048) and c.range_topk_buffer(5).shape == (2, 2048)
    assert c.range_topk_buffer(4) is None
    c.close()
    assert not cd.lib().cdadam_create_range(1000, 2, 0, 10, 0, 1, cd.TOPK, 1001, 0.9, 0.999, 1e-3, 1e-8)
