"""GPU parity: the CUDA library (through its C interface) against the CPU oracle, element
by element, on the same seeded inputs.

Bar: sign words, scales, top-k index sets and values bit-exact after a single step from the
same state; every float state vector within max relative error 1e-5 after every step of a
free run and 1e-4 after the last one, relative error = max_j |a_j - b_j| / max(|b_j|, tau)
with tau = 1e-6 * max_j |b_j| so that exact zeros do not dominate.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2111_00705_b200 import binding as cd
from paper_2111_00705_b200 import synth

pytestmark = pytest.mark.gpu

STEP_TOL, FINAL_TOL = 1e-5, 1e-4


def rel_err(a, b):
    a = a.astype(np.float64).ravel(); b = b.astype(np.float64).ravel()
    if a.size == 0:
        return 0.0
    tau = 1e-6 * max(np.abs(b).max(), 1e-300)
    return float(np.max(np.abs(a - b) / np.maximum(np.abs(b), tau)))


def u32(t):
    return t.cpu().numpy().view(np.uint32)


def make_pair(w, x0=None, **kw):
    dev = torch.device("cuda")
    x0 = w.x0("cpu") if x0 is None else x0
    args = dict(beta1=w.beta1, beta2=w.beta2, lr=w.lr, eps=w.eps)
    args.update(kw)
    g = cd.CDAdam(w.d, w.n, w.compressor, k=w.k, offsets=w.offsets, x0=x0.to(dev), **args)
    o = orc.Oracle(w.d, w.n, w.compressor, k=w.k, offsets=w.offsets, x0=x0.numpy(), **args)
    return g, o


def check_payloads(g, o, w):
    if w.compressor == synth.IDENTITY:
        return
    for who in list(range(w.n)) + [cd.SERVER]:
        a, b = g.last_payload(who)
        oa, ob = o.payload(who)
        assert np.array_equal(u32(a), oa), "payload words/indices of %s differ" % who
        assert np.array_equal(b.cpu().numpy().view(np.uint32), ob.view(np.uint32)), \
            "scales/values of %s differ" % who


def check_state(g, o, tol, exact=False):
    worst = 0.0
    for name in orc.STATE_NAMES:
        if name == "ghat_s" and g.mode != cd.MARKOV:
            continue                                  # scratch outside Algorithm 1
        a = g.get_state(name).cpu().numpy()
        b = o.state(name)
        if exact:
            assert np.array_equal(a.ravel(), b.ravel()), name
        e = rel_err(a, b)
        assert e <= tol, "%s: rel err %g" % (name, e)
        worst = max(worst, e)
    return worst


def run_free(w, steps, exact=True, tile=0, launches=None, **kw):
    """Free run: both sides step independently from the same inputs."""
    g, o = make_pair(w, **kw)
    if tile:
        g.set_tile(tile)
    if launches is not None:
        assert g.launches_per_step() == launches
    for t in range(1, steps + 1):
        grads = w.grads(t, "cpu")
        g.step(grads.cuda())
        o.step(grads.numpy())
        torch.cuda.synchronize()
        check_payloads(g, o, w)
        # reading ghat_w applies the deferred payload: do it on alternate steps only so that
        # both the deferred and the materialised path are exercised
        if t % 2 == 0 or t == steps:
            check_state(g, o, FINAL_TOL if t == steps else STEP_TOL, exact=exact)
        else:
            for name in ("x", "m", "v", "vhat", "gtil") + (() if g.mode != cd.MARKOV else ("ghat_s",)):
                assert rel_err(g.get_state(name).cpu().numpy(), o.state(name)) <= STEP_TOL
    g.device_status()                     # no kernel gave up a bounded wait
    g.close(); o.close()


def run_teacher_forced(w, steps):
    """Single-step parity: load the oracle's state into the GPU before every step."""
    g, o = make_pair(w)
    for t in range(1, steps + 1):
        for name in orc.STATE_NAMES:
            g.set_state(name, torch.from_numpy(o.state(name).copy()).cuda().reshape(-1))
        grads = w.grads(t, "cpu")
        g.step(grads.cuda())
        o.step(grads.numpy())
        check_payloads(g, o, w)
        check_state(g, o, STEP_TOL, exact=True)
    g.close(); o.close()


# ---------------------------------------------------------------------------- configurations

def test_c1_full_free_run():
    run_free(synth.workload("C1"), 10)


@pytest.mark.parametrize("name,scale", [("C2", 0.01), ("C3", 0.004), ("C4", 0.002), ("C5", 0.0001)])
def test_configurations_run_their_own_number_of_steps(name, scale):
    """Free runs of the configurations' own lengths (C2 100, C3 50, C4 50, C5 20 steps) at a
    scaled-down d: payloads bit for bit after every step, every state vector within 1e-5
    after every step and within 1e-4 (and bit for bit) after the last one."""
    w = synth.workload(name, scale=scale)
    assert w.steps == {"C2": 100, "C3": 50, "C4": 50, "C5": 20}[name]
    run_free(w, w.steps)


def test_c1_teacher_forced():
    run_teacher_forced(synth.workload("C1"), 4)


def test_c2_scaled_segments():
    w = synth.workload("C2", scale=0.02)          # d = 224,000, 62 ragged segments, n = 8
    assert w.q == 62
    run_free(w, 6)


def test_c3_scaled_topk():
    w = synth.workload("C3", scale=0.01)          # d = 256,000, k = 2,560, n = 16
    run_free(w, 5)


def test_c3_teacher_forced():
    run_teacher_forced(synth.workload("C3", scale=0.004), 3)


def test_c4_scaled_heavy_tails():
    w = synth.workload("C4", scale=0.004)         # d = 440,000, 15 segments, Student-t
    assert w.q == 15
    run_free(w, 5)


def test_c5_scaled_flat():
    w = synth.workload("C5", scale=0.0004)        # d = 600,000 flat, n = 4
    run_free(w, 4)


@pytest.mark.parametrize("tile", [8192, 16384, 32768])
def test_large_tiles_and_prefetch_ring_give_the_same_bits(tile):
    """Tiles of 16384+ coordinates run the worker kernel with the asynchronous-copy ring;
    segments cut some tiles (scalar path) and d leaves a ragged last tile."""
    d = 5 * 32768 + 4321 * 4
    off = np.array([0, 1000, 40000, 40001, 3 * 32768, d])
    run_free(synth.Workload("RING", d, 3, synth.SIGN, 4, offsets=off, seed=tile), 4, tile=tile)
    run_free(synth.Workload("RINGF", 4 * 65536, 2, synth.SIGN, 3, seed=tile + 1), 3, tile=tile)


@pytest.mark.parametrize("n", [1, 5, 8, 9, 17, 32, 33, 40])
def test_sign_worker_counts_cover_table_and_sequential_server_sums(n):
    """n <= 8: the server sum comes from the pattern table alone; 9..32: table plus workers
    added one by one; above 32: the staged kernel; odd n: true division by n."""
    off = np.array([0, 5000, 3 * 4096 + 100, 5 * 4096])
    run_free(synth.Workload("N", 5 * 4096, n, synth.SIGN, 3, offsets=off, seed=n), 3)


def test_segment_of_more_than_4096_tiles_is_summed_by_several_blocks():
    """Flat buffer of 8195 tiles of 4096 coordinates: three blocks of the scale kernel share
    the segment and the last one to finish adds their sums; a second, short segment beside it
    is summed by one block (the others find nothing to add)."""
    d = 8195 * 4096 + 3
    off = np.array([0, d - 5000, d])
    run_free(synth.Workload("LS", d, 1, synth.SIGN, 2, offsets=off, seed=31), 2, tile=4096)


@pytest.mark.parametrize("n,launches", [(4, 3), (5, 5)])
@pytest.mark.parametrize("mode", [cd.MARKOV, cd.EF])
def test_scales_finished_in_the_passes_or_by_their_own_kernel(n, launches, mode):
    """148 tiles per worker: with 4 workers the worker pass is one wave of blocks and finishes
    its scales itself (tickets, last block adds); with 5 the separate kernel does.  Segments
    that cut tiles put several tickets on one block."""
    d = 148 * 4096
    off = np.array([0, 5, 4096, 9000, 300001, 300002, d - 4097, d])
    run_free(synth.Workload("F1", d, n, synth.SIGN, 4, offsets=off, seed=11), 4, mode=mode, launches=launches)
    run_free(synth.Workload("F2", d - 3, n, synth.SIGN, 3, seed=12), 3, mode=mode, launches=launches)


@pytest.mark.parametrize("case", ["sign_flat", "sign_segments", "sign_ring", "topk", "identity"])
def test_error_feedback_mode_matches_oracle(case):
    """Classical error feedback (the paper's comparison scheme, Section 4) through the same
    kernels: payloads bit-exact, worker and server error vectors and optimizer state exact."""
    if case == "sign_flat":
        run_free(synth.Workload("EF1", 3 * 4096 + 77, 4, synth.SIGN, 5, seed=1), 5, mode=cd.EF)
    elif case == "sign_segments":
        w = synth.workload("C2", scale=0.01)
        run_free(w, 5, mode=cd.EF)
    elif case == "sign_ring":
        off = np.array([0, 1000, 40000, 3 * 32768, 5 * 32768 + 444])
        run_free(synth.Workload("EF3", 5 * 32768 + 444, 3, synth.SIGN, 4, offsets=off, seed=3), 4,
                 tile=16384, mode=cd.EF)
    elif case == "topk":
        run_free(synth.workload("C3", scale=0.004), 5, mode=cd.EF)
    else:
        run_free(synth.Workload("EF5", 5000, 3, synth.IDENTITY, 4), 4, mode=cd.EF)


@pytest.mark.parametrize("case", ["sign_flat", "sign_segments", "sign_ring_tiles", "sign_bf16", "topk", "topk_small",
                                  "identity"])
def test_naive_compression_mode_matches_oracle(case):
    """AMSGrad with naive compression (Section 4; compared in Section 6): c^(i) = C(g^(i)),
    c = C(mean), no compression state.  Payloads bit-exact, moments and x exact, and the
    state vectors of Algorithm 1 stay zero."""
    if case == "sign_flat":
        run_free(synth.Workload("N1", 3 * 4096 + 77, 4, synth.SIGN, 5, seed=1), 5, mode=cd.NAIVE)
    elif case == "sign_segments":
        run_free(synth.workload("C2", scale=0.01), 5, mode=cd.NAIVE)
    elif case == "sign_ring_tiles":
        off = np.array([0, 1000, 40000, 3 * 32768, 5 * 32768 + 444])
        run_free(synth.Workload("N3", 5 * 32768 + 444, 3, synth.SIGN, 4, offsets=off, seed=3), 4,
                 tile=16384, mode=cd.NAIVE)
    elif case == "sign_bf16":
        w = synth.Workload("N4", 2 * 4096 + 40, 3, synth.SIGN, 3, seed=4)
        g, o = make_pair(w, mode=cd.NAIVE)
        for t in range(1, 4):
            gb = w.grads(t, "cuda").to(torch.bfloat16)
            g.step_bf16(gb.reshape(-1))
            o.step(gb.float().cpu().numpy())
            check_payloads(g, o, w)
        check_state(g, o, STEP_TOL, exact=True)
        g.close(); o.close()
    elif case == "topk":
        run_free(synth.workload("C3", scale=0.004), 5, mode=cd.NAIVE)
    elif case == "topk_small":
        run_free(synth.Workload("N6", 777, 5, synth.TOPK, 4, k=31, seed=6), 4, mode=cd.NAIVE)
    else:
        run_free(synth.Workload("N7", 5000, 3, synth.IDENTITY, 4), 4, mode=cd.NAIVE)


@pytest.mark.parametrize("comp", [cd.SIGN, cd.TOPK, cd.IDENTITY])
@pytest.mark.parametrize("mode", [cd.MARKOV, cd.EF, cd.NAIVE])
def test_weight_decay_and_lr_milestones_match_oracle(comp, mode):
    """Decoupled weight decay and step-size milestones (Section 6) in every update kernel."""
    w = synth.Workload("WD", 3 * 4096 + 5, 3, comp, 7, k=100 if comp == cd.TOPK else 0, seed=8, lr=1e-2)
    g, o = make_pair(w, mode=mode)
    for side in (g, o):
        side.set_weight_decay(0.05)
        side.set_lr_milestones(1e-2, [2, 5], 0.1)
    for t in range(1, 8):
        if t == 7:                                    # an explicit step size ends the schedule
            g.set_lr(3e-3); o.set_lr(3e-3)
        grads = w.grads(t, "cpu")
        g.step(grads.cuda())
        o.step(grads.numpy())
        check_payloads(g, o, w)
        for name in ("x", "m", "v", "vhat"):
            assert np.array_equal(g.get_state(name).cpu().numpy().ravel(), o.state(name).ravel()), (t, name)
    assert cd.lib().cdadam_set_weight_decay(g._h, -1.0) == cd.ERR_ARG
    bad = (ctypes.c_int64 * 2)(5, 2)
    assert cd.lib().cdadam_set_lr_milestones(g._h, 1e-2, 2, bad, 0.1) == cd.ERR_ARG
    assert cd.lib().cdadam_set_lr_milestones(g._h, 1e-2, 1, bad, 1.5) == cd.ERR_ARG
    g.close(); o.close()


@pytest.mark.parametrize("mode", [cd.MARKOV, cd.EF, cd.NAIVE])
@pytest.mark.parametrize("d,n,k", [(50000, 4, 500), (4097, 3, 4097), (70001, 2, 1)])
def test_randk_matches_oracle(mode, d, n, k):
    """Rand-k (Appendix A) with the random coordinate sets supplied to both sides."""
    w = synth.Workload("RK", d, n, synth.RANDK, 4, k=k, seed=d)
    g, o = make_pair(w, mode=mode)
    for t in range(1, 5):
        W = synth.random_sets(d, k, n, w.seed, t)
        S = synth.random_sets(d, k, 1, w.seed + 1, t)[0]
        g.set_random_sets(torch.from_numpy(W.view(np.int32)).cuda(),
                          torch.from_numpy(S.view(np.int32)).cuda())
        o.set_random_sets(W, S)
        grads = w.grads(t, "cpu")
        g.step(grads.cuda()); o.step(grads.numpy())
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)
    g.device_status()


def test_randk_malformed_sets_are_reported_not_dereferenced():
    d, n, k = 1000, 2, 5
    g = cd.CDAdam(d, n, cd.RANDK, k=k)
    with pytest.raises(cd.CdadamError):
        g.step(torch.zeros(n * d, device="cuda"))            # no sets yet
    bad = torch.tensor([[1, 2, 3, 4, 5], [9, 8, 7, 6, 2_000_000_000]], dtype=torch.int32, device="cuda")
    g.set_random_sets(bad, torch.arange(k, dtype=torch.int32, device="cuda"))
    g.step(torch.ones(n * d, device="cuda"))
    with pytest.raises(cd.CdadamError) as e:
        g.device_status()
    assert e.value.code == cd.ERR_ARG
    torch.cuda.synchronize()                                 # the device is still usable
    assert torch.ones(4, device="cuda").sum().item() == 4


@pytest.mark.parametrize("case", ["sign_ragged", "sign_segments", "sign_ring", "sign_ef", "topk", "identity"])
def test_bf16_gradients_equal_the_widened_fp32_run(case):
    """Gradients given in bfloat16: widening is exact, so payloads and state must equal the
    oracle's on the widened values, whichever kernel reads the 16-bit data."""
    tile, mode = 0, cd.MARKOV
    if case == "sign_ragged":
        w = synth.Workload("B1", 3 * 4096 + 77, 3, synth.SIGN, 4, seed=1)        # d % 8 != 0: scalar reads
    elif case == "sign_segments":
        w = synth.workload("C2", scale=0.01)
    elif case == "sign_ring":
        off = np.array([0, 1000, 40000, 3 * 32768, 5 * 32768 + 448])
        w = synth.Workload("B3", 5 * 32768 + 448, 3, synth.SIGN, 4, offsets=off, seed=3)
        tile = 16384
    elif case == "sign_ef":
        w = synth.Workload("B4", 8 * 4096, 4, synth.SIGN, 4, seed=4)
        mode = cd.EF
    elif case == "topk":
        w = synth.workload("C3", scale=0.004)
    else:
        w = synth.Workload("B6", 5000, 3, synth.IDENTITY, 4)
    g, o = make_pair(w, mode=mode)
    if tile:
        g.set_tile(tile)
    for t in range(1, 5):
        gb = w.grads(t, "cpu").to(torch.bfloat16)
        g.step_bf16(gb.cuda().reshape(-1))
        o.step(gb.to(torch.float32).numpy())
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)
    g.device_status()


def test_identity_matches_oracle():
    w = synth.Workload("ID", 5000, 3, synth.IDENTITY, 4)
    run_free(w, 4)


# ---------------------------------------------------------------------------- shapes and edges

@pytest.mark.parametrize("d", list(range(1, 70)) + [127, 128, 129, 1023, 1024, 1025, 4095, 4096,
                                                     4097, 8191, 8193, 12288, 12290])
def test_sign_every_small_and_ragged_size(d):
    w = synth.Workload("R", d, 2, synth.SIGN, 3, seed=d)
    run_free(w, 3)


@pytest.mark.parametrize("lo", [70, 400, 730])
def test_sign_and_topk_every_size_up_to_1025(lo):
    """Every d from 70 to 1025 (the smaller ones are above), two iterations each, scaled sign
    with a segment boundary at a position that moves with d, and top-k with k moving with d:
    messages bit-exact, x exact."""
    for d in range(lo, min(lo + 330, 1026)):
        grads = [torch.randn(2, d, generator=torch.Generator().manual_seed(1000 * t + d)) for t in (1, 2)]
        off = np.array([0, 1 + (d * 7) % (d - 1), d])
        for comp, kw in ((cd.SIGN, dict(offsets=off)), (cd.TOPK, dict(k=1 + (d * 13) % d))):
            g = cd.CDAdam(d, 2, comp, **kw)
            o = orc.Oracle(d, 2, comp, **kw)
            for gr in grads:
                g.step(gr.cuda().reshape(-1)); o.step(gr.numpy())
            for who in (0, 1, cd.SERVER):
                a, b = g.last_payload(who)
                oa, ob = o.payload(who)
                assert np.array_equal(u32(a), oa) and np.array_equal(u32(b), ob.view(np.uint32)), (d, comp, who)
            assert np.array_equal(g.params().cpu().numpy(), o.state("x")), (d, comp)
            g.close(); o.close()


@pytest.mark.parametrize("shift", range(0, 32, 3))
def test_sign_segment_boundaries_at_every_residue(shift):
    d = 3 * 4096 + 77
    off = np.array([0, 5 + shift, 4096 + shift, 4096 + shift + 1, 2 * 4096 - shift, d])
    w = synth.Workload("S", d, 3, synth.SIGN, 3, offsets=off, seed=shift)
    run_free(w, 3)


def test_many_tiny_segments_in_one_tile():
    d = 9000
    off = np.concatenate([np.arange(0, 640, 5), [700, 4096, 4100, 8192, d]])
    w = synth.Workload("T", d, 2, synth.SIGN, 3, offsets=off)
    run_free(w, 3)


def test_unaligned_gradient_pointer_gives_same_bits():
    w = synth.workload("C1", scale=0.25)
    g, o = make_pair(w)
    buf = torch.empty(w.n * w.d + 1, device="cuda")
    for t in range(1, 4):
        grads = w.grads(t, "cpu")
        view = buf[1:]                              # 4-byte aligned only
        view.copy_(grads.reshape(-1))
        assert view.data_ptr() % 16 != 0
        g.step(view)
        o.step(grads.numpy())
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)


@pytest.mark.parametrize("d,k", [(1, 1), (7, 7), (33, 1), (1000, 1000), (5000, 17), (40000, 400),
                                 (32768 + 5, 300)])
def test_topk_shapes(d, k):
    w = synth.Workload("K", d, 3, synth.TOPK, 3, k=k, seed=d + k)
    run_free(w, 3)


def test_topk_threshold_guess_hits_and_misses():
    """The selection reuses the previous threshold bucket as a guess.  Gradients whose scale
    stays, grows (guess holds) and collapses by 20x (guess fails, classic two passes) must
    all give the oracle's payloads."""
    rng = np.random.default_rng(3)
    d, n, k = 150000, 3, 1500
    w = synth.Workload("GUESS", d, n, synth.TOPK, 8, k=k)
    g, o = make_pair(w, x0=torch.zeros(d))
    for scale in (1.0, 1.0, 0.9, 0.05, 0.05, 3.0, 3.0, 1e-30, 1e-30, 0.0, 1.0):
        grads = (rng.standard_normal((n, d)) * scale).astype(np.float32)
        g.step(torch.from_numpy(grads).cuda()); o.step(grads)
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)


@pytest.mark.parametrize("mode", [cd.MARKOV, cd.EF])
def test_topk_selection_concentrated_in_a_few_tiles(mode):
    """One tensor with gradients 100x larger than the rest takes the whole selection: its
    4096-coordinate tiles have far more candidates than a tile's list holds (512), so the list
    passes read those tiles from the data again; the other tiles keep their (short) lists.
    Steady state (the guess holds) over several steps, ragged d."""
    rng = np.random.default_rng(5)
    d, n, k = 40 * 4096 + 123, 3, 6000
    big = slice(7 * 4096 + 100, 10 * 4096 + 50)             # 12238 coordinates, k of them kept
    w = synth.Workload("CONC", d, n, synth.TOPK, 6, k=k)
    g, o = make_pair(w, x0=torch.zeros(d), mode=mode)
    for t in range(6):
        grads = rng.standard_normal((n, d)).astype(np.float32)
        grads[:, big] *= 100.0
        if t == 4:
            grads[:, 20 * 4096:20 * 4096 + 700] = 1e4       # a second dense tile appears
        g.step(torch.from_numpy(grads).cuda()); o.step(grads)
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)
    g.close(); o.close()


@pytest.mark.parametrize("mode", [cd.MARKOV, cd.EF, cd.NAIVE])
def test_topk_dense_pass_with_the_prefetch_ring_at_small_sizes(mode):
    """Large problems make their dense pass with the prefetch-ring kernel; set_tile(16384)
    selects it at sizes the oracle finishes quickly.  Whole tiles go through the ring, the
    ragged last tile through the plain kernel; both with and without the state operand."""
    w = synth.workload("C3", scale=0.01)                    # d = 256,000 = 62.5 tiles, n = 16
    run_free(w, 5, tile=16384, mode=mode)
    w = synth.Workload("RING1", 9 * 4096, 2, synth.TOPK, 4, k=999, seed=5)       # whole tiles only, odd count
    run_free(w, 4, tile=16384, mode=mode)


def test_topk_prefetch_ring_with_failed_guesses_and_dense_tiles():
    rng = np.random.default_rng(11)
    d, n, k = 40 * 4096 + 2048, 3, 6000                     # rows stay 16-byte aligned, last tile ragged
    big = slice(7 * 4096 + 100, 10 * 4096 + 50)
    w = synth.Workload("RINGCONC", d, n, synth.TOPK, 8, k=k)
    g, o = make_pair(w, x0=torch.zeros(d))
    g.set_tile(16384)
    for t, scale in enumerate((1.0, 1.0, 0.05, 0.05, 3.0, 3.0, 1.0, 1.0)):
        grads = (rng.standard_normal((n, d)) * scale).astype(np.float32)
        if t >= 4:
            grads[:, big] *= 100.0                          # one tensor takes the whole selection: tiles without lists
        if t == 6:
            grads[:, 20 * 4096:20 * 4096 + 700] = 1e4
        g.step(torch.from_numpy(grads).cuda()); o.step(grads)
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)
    g.device_status()
    g.close(); o.close()


@pytest.mark.parametrize("n", [4, 5, 9, 16])
def test_topk_prefetch_ring_rows_that_hit_beside_rows_that_miss(n):
    """Scale jumps make the guesses of all rows fail; a jump in some workers only leaves rows
    selected from the dense pass's lists and rows on the classic chain side by side in the
    same launches (the two chains run as two branches of the step)."""
    rng = np.random.default_rng(100 + n)
    d, k = 12 * 4096 + 1000, 1500
    w = synth.Workload("GROUPS", d, n, synth.TOPK, 9, k=k)
    g, o = make_pair(w, x0=torch.zeros(d))
    g.set_tile(16384)
    some = np.arange(n) % 3 == 1
    for t, scale in enumerate((1.0, 1.0, 0.02, 0.02, 1.0, 1.0, 1.0, 50.0, 50.0)):
        grads = (rng.standard_normal((n, d)) * scale).astype(np.float32)
        if t in (5, 6):
            grads[some] *= 0.01                             # only these rows miss (and miss again coming back)
        g.step(torch.from_numpy(grads).cuda()); o.step(grads)
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)
    g.device_status()
    g.close(); o.close()


@pytest.mark.parametrize("n", [17, 24, 32, 33, 64, 65])
def test_topk_aggregation_of_many_workers(n):
    """The server's dense pass adds the workers' messages in batches of sixteen workers (up to
    64; beyond that worker by worker): sums in worker order whatever the batch a worker is in.
    A quarter of the coordinates is sent by every worker, so most sums have many terms."""
    rng = np.random.default_rng(n)
    d, k = 6 * 4096 + 123, 900
    w = synth.Workload("MANYW", d, n, synth.TOPK, 5, k=k)
    g, o = make_pair(w, x0=torch.zeros(d))
    common = rng.choice(d, 300, replace=False)
    for t in range(5):
        grads = rng.standard_normal((n, d)).astype(np.float32)
        grads[:, common] *= 50.0
        g.step(torch.from_numpy(grads).cuda()); o.step(grads)
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)
    g.close(); o.close()


@pytest.mark.parametrize("case", ["ragged", "aligned_large", "one_segment"])
def test_topk_per_segment_matches_oracle(case):
    """Top-k applied to every segment on its own (per tensor): concatenated payloads bit-exact,
    all state exact, over several steps (so the per-segment threshold guesses are used)."""
    if case == "ragged":
        d, n = 30011, 3
        off = [0, 5, 6, 4101, 4102, 20000, d]
        ks = [2, 1, 300, 1, 77, 1000]
    elif case == "aligned_large":
        d, n = 3 * 40960, 4
        off = [0, 40960, 2 * 40960, d]
        ks = [400, 41, 4000]
    else:
        d, n = 50000, 2
        off, ks = [0, d], [500]
    w = synth.Workload("SEGK", d, n, synth.TOPK, 5, k=1, seed=41)
    g, o = make_pair(w)
    g.set_topk_segments(off, ks)
    o.set_topk_segments(off, ks)
    if case == "aligned_large":
        g.set_tile(16384)                                       # dense passes through the prefetch ring, rows strided by d
    w.k = sum(ks)
    rng = np.random.default_rng(7)
    scale = np.repeat(10.0 ** rng.uniform(-2, 1, len(ks)), np.diff(off)).astype(np.float32)
    for t_ in range(1, 6):
        grads = w.grads(t_, "cpu") * torch.from_numpy(scale)        # tensors of different scales
        g.step(grads.cuda()); o.step(grads.numpy())
        check_payloads(g, o, w)
        check_state(g, o, STEP_TOL, exact=True)
    if case == "one_segment":                                   # = the whole-vector compressor
        h = cd.CDAdam(d, n, cd.TOPK, k=500, x0=w.x0("cpu").cuda())
        for t_ in range(1, 6):
            h.step((w.grads(t_, "cpu") * torch.from_numpy(scale)).cuda())
        assert torch.equal(h.params(), g.params())
        h.close()
    assert cd.lib().cdadam_set_topk_segments(g._h, 1, (ctypes.c_int64 * 2)(0, d), (ctypes.c_int64 * 1)(1)) == cd.ERR_STATE
    g.close(); o.close()
    f = cd.CDAdam(100, 2, cd.TOPK, k=3)
    with pytest.raises(cd.CdadamError):
        f.set_topk_segments([0, 10, 100], [11, 1])                  # k_r above the segment length
    with pytest.raises(cd.CdadamError):
        cd.CDAdam(100, 2, cd.SIGN).set_topk_segments([0, 100], [1])


def test_topk_ties_lower_index_wins():
    """Few distinct magnitudes: most of the selection is decided by the tie rule."""
    rng = np.random.default_rng(0)
    d, n, k = 70000, 2, 900
    g, o = None, None
    w = synth.Workload("TIE", d, n, synth.TOPK, 3, k=k)
    g, o = make_pair(w, x0=torch.zeros(d))
    for t in range(3):
        grads = (rng.integers(-2, 3, (n, d)) * 0.5).astype(np.float32)
        g.step(torch.from_numpy(grads).cuda()); o.step(grads)
        check_payloads(g, o, w)
    check_state(g, o, FINAL_TOL, exact=True)
    # all coordinates equal: the first k indices are kept
    idx, val = cd.compress_topk(torch.full((5000,), -1.5, device="cuda"), 123)
    assert idx.cpu().tolist() == list(range(123)) and torch.all(val == -1.5)
    idx, val = cd.compress_topk(torch.zeros(4097, device="cuda"), 4097)
    assert idx.cpu().tolist() == list(range(4097))


def test_standalone_compressors_match_oracle():
    rng = np.random.default_rng(1)
    for d in (1, 31, 32, 33, 4096, 4097, 100003):
        x = (rng.standard_normal(d) * np.exp2(rng.uniform(-20, 20, d))).astype(np.float32)
        bits, scales = cd.compress_sign(torch.from_numpy(x).cuda())
        ob, os_, _ = orc.compress_sign(x)
        assert np.array_equal(u32(bits), ob) and np.array_equal(scales.cpu().numpy(), os_)
        k = max(1, d // 50)
        idx, val = cd.compress_topk(torch.from_numpy(x).cuda(), k)
        oi, ov, _ = orc.compress_topk(x, k)
        assert np.array_equal(u32(idx), oi) and np.array_equal(val.cpu().numpy(), ov)
    off = np.array([0, 3, 4099, 50000, 100003])
    bits, scales = cd.compress_sign(torch.from_numpy(x).cuda(), off)
    ob, os_, _ = orc.compress_sign(x, off)
    assert np.array_equal(u32(bits), ob) and np.array_equal(scales.cpu().numpy(), os_)


def test_scale_is_correctly_rounded_on_hard_sums():
    """Magnitudes spread over 80 binades defeat plain double accumulation; the scale must
    still be the correctly rounded exact sum divided by d."""
    rng = np.random.default_rng(2)
    d = 1 << 20
    x = (rng.standard_normal(d) * np.exp2(rng.uniform(-40, 40, d))).astype(np.float32)
    _, scales = cd.compress_sign(torch.from_numpy(x).cuda())
    want = np.float32(orc.l1_exact(x) / d)
    assert scales.cpu().numpy()[0] == want


def test_set_lr_and_step_host_and_params_view():
    w = synth.workload("C1", scale=0.5)
    g, o = make_pair(w)
    grads = w.grads(1, "cpu")
    xh = torch.empty(w.d).pin_memory()
    g.step_host(grads.pin_memory(), xh)
    o.step(grads.numpy())
    assert np.array_equal(xh.numpy(), o.state("x"))
    g.set_lr(5e-4); o.set_lr(5e-4)
    grads = w.grads(2, "cpu")
    g.step(grads.cuda()); o.step(grads.numpy())
    torch.cuda.synchronize()
    assert np.array_equal(g.params().cpu().numpy(), o.state("x"))
    assert g.step_count() == 2 and g.launches_per_step() >= 3


@pytest.mark.parametrize("comp", [cd.SIGN, cd.TOPK, cd.IDENTITY])
def test_non_finite_gradients_neither_hang_nor_fault(comp):
    """The contract asks for finite gradients; NaN and infinities give an unspecified result
    but must leave the device usable (no out-of-range access, no endless wait)."""
    d, n = 3 * 4096 + 5, 3
    g = cd.CDAdam(d, n, comp, k=100 if comp == cd.TOPK else 0)
    grads = torch.randn(n, d, device="cuda")
    grads[0, 5] = float("nan"); grads[1, 4097] = float("inf"); grads[2, d - 1] = -float("inf")
    for _ in range(3):
        g.step(grads.reshape(-1))
    g.device_status()
    torch.cuda.synchronize()
    g.close()
    ok = cd.CDAdam(64, 1, cd.SIGN)
    ok.step(torch.ones(64, device="cuda"))
    assert torch.isfinite(ok.params()).all()


@pytest.mark.parametrize("comp,mode", [(cd.SIGN, cd.MARKOV), (cd.SIGN, cd.EF), (cd.TOPK, cd.MARKOV)])
def test_replayed_steps_match_oracle(comp, mode):
    """Launch-bound scaled-sign problems and every top-k step of Algorithm 1 replay their
    launches from a recorded graph once a gradient buffer has been seen twice.  Two buffers
    in turn, a side stream, a read of the worker states (which applies the deferred payload
    and changes the next step's arguments) and a change of step size (a launch argument) in
    between: every payload and state vector against the oracle."""
    d = 5 * 4096 + 13
    if comp == cd.SIGN:
        w = synth.Workload("G1", d, 4, synth.SIGN, 14, offsets=np.array([0, 4000, 9000, d]), seed=21)
    else:
        w = synth.Workload("G2", d, 4, synth.TOPK, 14, k=300, seed=22)
    g, o = make_pair(w, mode=mode)
    bufs = [torch.empty(w.n * w.d, device="cuda") for _ in range(2)]
    side = torch.cuda.Stream()
    for t in range(1, 15):
        grads = w.grads(t, "cpu")
        buf = bufs[0] if t < 6 else bufs[t % 2]
        buf.copy_(grads.reshape(-1))
        if t == 9:
            g.set_lr(5e-4); o.set_lr(5e-4)
        if t in (7, 8, 12):
            torch.cuda.synchronize()
            with torch.cuda.stream(side):
                g.step(buf, stream=side)
            side.synchronize()
        else:
            g.step(buf)
        o.step(grads.numpy())
        torch.cuda.synchronize()
        check_payloads(g, o, w)
        if t in (4, 10, 14):
            check_state(g, o, STEP_TOL, exact=True)
        else:
            for name in ("x", "m", "v", "vhat", "gtil"):
                assert np.array_equal(g.get_state(name).cpu().numpy().ravel(), o.state(name).ravel()), (t, name)
    g.device_status()
    g.close(); o.close()


@pytest.mark.parametrize("comp", [cd.SIGN, cd.TOPK])
def test_replay_with_a_step_size_per_step_and_many_buffers(comp):
    """A step size that changes every step makes recorded graphs stale every step (they are set
    aside, and recording stops after a few rounds); six gradient buffers in rotation exceed
    the four graphs a context keeps.  Results stay those of the oracle."""
    d = 2 * 4096 + 5
    w = synth.Workload("G3", d, 3, comp, 40, k=64 if comp == cd.TOPK else 0, seed=23)
    g, o = make_pair(w)
    bufs = [torch.empty(w.n * d, device="cuda") for _ in range(6)]
    for t in range(1, 41):
        grads = w.grads(t, "cpu")
        buf = bufs[t % 6] if t > 12 else bufs[t % 2]
        buf.copy_(grads.reshape(-1))
        if t <= 24:
            lr = 1e-3 / t
            g.set_lr(lr); o.set_lr(lr)
        g.step(buf)
        o.step(grads.numpy())
        if t % 8 == 0:
            check_payloads(g, o, w)
            for name in ("x", "m", "vhat", "gtil"):
                assert np.array_equal(g.get_state(name).cpu().numpy().ravel(), o.state(name).ravel()), (t, name)
    check_state(g, o, FINAL_TOL, exact=True)
    g.close(); o.close()


def test_step_on_a_capturing_stream_is_refused():
    g = cd.CDAdam(4096, 2, cd.SIGN)
    grads = torch.randn(2 * 4096, device="cuda")
    g.step(grads)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    other = torch.zeros(8, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        graph.capture_begin()
        other.add_(1.0)                                   # the caller's own work is recorded
        rc = cd.lib().cdadam_step(g._h, ctypes.c_void_p(grads.data_ptr()), ctypes.c_void_p(side.cuda_stream))
        graph.capture_end()
    assert rc == cd.ERR_STATE and "captur" in cd.last_error()
    g.step(grads)                                         # the context is unharmed
    assert g.step_count() == 2
    g.close()


def test_stage_timing_and_late_configuration_calls():
    # a grid of one wave finishes its scales inside the passes (3 launches); larger ones
    # use the separate scale kernel (5 launches)
    for d, names in ((3 * 4096, {"k_worker_sign", "k_server_sign", "k_update_sign"}),
                     (400 * 4096, {"k_worker_sign", "k_finalize_scales(workers)", "k_server_sign",
                                   "k_finalize_scales(server)", "k_update_sign"})):
        g = cd.CDAdam(d, 2, cd.SIGN)
        grads = torch.randn(2 * d, device="cuda")
        g.profile_enable(True)
        for _ in range(4):
            g.step(grads)
        ms, steps = g.profile_read()
        assert steps == 4 and set(ms) == names
        assert all(v > 0 for v in ms.values())
        assert g.profile_read()[1] == 0                   # reading forgets the events
        g.profile_enable(False)
        assert g.launches_per_step() == len(names)
    with pytest.raises(cd.CdadamError):
        g.set_tile(8192)                                  # after the first step
    assert cd.lib().cdadam_set_mode(g._h, cd.EF) == cd.ERR_STATE
    h = cd.CDAdam(100, 2, cd.IDENTITY)
    with pytest.raises(cd.CdadamError):
        h.set_tile(4096)                                  # the identity compressor has no tiles
    cd.CDAdam(100, 2, cd.TOPK, k=3).set_tile(4096)        # top-k: picks the kernel of the dense pass
    f = cd.CDAdam(100, 2, cd.SIGN)
    with pytest.raises(cd.CdadamError):
        f.set_tile(1000)                                  # not a multiple of 4096
    assert cd.lib().cdadam_set_mode(f._h, 7) == cd.ERR_ARG
    with pytest.raises(ValueError):
        f.step_bf16(torch.zeros(200, device="cuda"))      # wrong dtype is caught by the binding


def test_argument_errors_are_reported_not_fatal():
    with pytest.raises(cd.CdadamError):
        cd.CDAdam(0, 4)
    with pytest.raises(cd.CdadamError):
        cd.CDAdam(100, 0)
    with pytest.raises(cd.CdadamError):
        cd.CDAdam(100, 2, cd.TOPK, k=0)
    with pytest.raises(cd.CdadamError):
        cd.CDAdam(100, 2, cd.TOPK, k=101)
    with pytest.raises(cd.CdadamError):
        cd.CDAdam(100, 2, 7)
    g = cd.CDAdam(100, 2)
    with pytest.raises(cd.CdadamError):
        g.set_segments([0, 50, 50, 100])
    with pytest.raises(cd.CdadamError):
        g.set_segments([0, 60, 40, 100])
    with pytest.raises(cd.CdadamError):
        g.set_segments([1, 100])
    with pytest.raises(cd.CdadamError):
        g.last_payload(0)                            # no step yet
    g.step(torch.zeros(200, device="cuda"))
    with pytest.raises(cd.CdadamError):
        g.set_segments([0, 50, 100])                 # after the first step
    with pytest.raises(cd.CdadamError):
        g.last_payload(5)
    torch.cuda.synchronize()


@pytest.mark.parametrize("name,scale,mode", [("C2", 0.01, cd.MARKOV), ("C2", 0.005, cd.EF), ("C3", 0.004, cd.MARKOV),
                                             ("C1", 0.25, cd.NAIVE)])
def test_checkpoint_and_resume_continue_the_run_bit_for_bit(name, scale, mode):
    """Save after 3 iterations (state vectors + counter), load into a fresh context, run 3 more
    on both: same messages and state as the uninterrupted run and as the oracle.  The step-size
    milestones make the counter matter."""
    w = synth.workload(name, scale=scale)
    x0 = w.x0("cpu")

    def fresh():
        g = cd.CDAdam(w.d, w.n, w.compressor, k=w.k, offsets=w.offsets, x0=x0.cuda(), mode=mode)
        g.set_lr_milestones(1e-3, [2, 4], 0.5)
        g.set_weight_decay(1e-2)
        return g

    a = fresh()
    o = orc.Oracle(w.d, w.n, w.compressor, k=w.k, offsets=w.offsets, x0=x0.numpy(), mode=mode)
    o.set_lr_milestones(1e-3, [2, 4], 0.5)
    o.set_weight_decay(1e-2)
    for t in range(1, 4):
        grads = w.grads(t, "cpu")
        a.step(grads.cuda()); o.step(grads.numpy())
    saved = a.state_dict()
    assert saved["step_count"] == 3
    b = fresh()
    b.load_state_dict(saved)
    assert b.step_count() == 3
    for t in range(4, 7):
        grads = w.grads(t, "cpu")
        a.step(grads.cuda()); b.step(grads.cuda()); o.step(grads.numpy())
        check_payloads(b, o, w)
        for who in list(range(w.n)) + [cd.SERVER]:
            pa, pb = a.last_payload(who), b.last_payload(who)
            assert torch.equal(pa[0], pb[0]) and torch.equal(pa[1].view(torch.int32), pb[1].view(torch.int32))
    check_state(b, o, FINAL_TOL, exact=True)
    for nm in orc.STATE_NAMES:
        assert torch.equal(a.get_state(nm), b.get_state(nm)), nm
    with pytest.raises(cd.CdadamError):
        b.set_step_count(-1)
    a.close(); b.close(); o.close()
