"""CPU pins of the oracle: what the paper and the mathematics fix, independent of the oracle.

Each test compares the C oracle with something that is not the oracle: hand-worked values
(tests/golden), Python's exact summation, exact rationals, a brute-force sort, the closed
forms of Appendix A, or an independently written vanilla AMSGrad.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [float(v) for v in vals]
    return out


# ------------------------------------------------------------------ exact l1 sum

def test_l1_exact_matches_fsum_wide_range():
    rng = np.random.default_rng(1)
    for trial in range(40):
        nel = int(rng.integers(1, 5000))
        # magnitudes spread over ~200 binades, both signs, some exact zeros and subnormals
        x = (rng.standard_normal(nel) * np.exp2(rng.uniform(-140, 60, nel))).astype(np.float32)
        x[rng.random(nel) < 0.05] = 0.0
        x[rng.random(nel) < 0.02] = np.float32(1e-42)
        want = math.fsum(abs(float(v)) for v in x)
        assert orc.l1_exact(x) == want


def test_l1_exact_matches_rationals_and_rounds_ties_to_even():
    # 2^60 + 2^7 is a tie between two doubles (spacing 2^8): ties-to-even keeps 2^60
    x = np.array([2.0 ** 60, 2.0 ** 7], dtype=np.float32)
    assert orc.l1_exact(x) == float(Fraction(2) ** 60)
    # 2^60 + 2^8 + 2^7: tie again, the even neighbour is now the upper one
    x = np.array([2.0 ** 60, 2.0 ** 8, 2.0 ** 7], dtype=np.float32)
    assert orc.l1_exact(x) == 2.0 ** 60 + 2.0 ** 9
    # sticky bit breaks the tie upward
    x = np.array([2.0 ** 60, 2.0 ** 7, 2.0 ** -100], dtype=np.float32)
    assert orc.l1_exact(x) == 2.0 ** 60 + 2.0 ** 8
    rng = np.random.default_rng(2)
    for _ in range(20):
        x = (rng.standard_normal(37) * np.exp2(rng.integers(-60, 60, 37))).astype(np.float32)
        exact = sum(Fraction(abs(float(v))) for v in x)
        got = Fraction(orc.l1_exact(x))
        # correctly rounded: no double is strictly closer to the exact sum
        f = orc.l1_exact(x)
        for nb in (np.nextafter(f, np.inf), np.nextafter(f, -np.inf)):
            assert abs(got - exact) <= abs(Fraction(float(nb)) - exact)


def test_l1_exact_order_independent_and_large():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(300_000) * np.exp2(rng.uniform(-30, 30, 300_000))).astype(np.float32)
    a = orc.l1_exact(x)
    assert a == orc.l1_exact(x[::-1].copy()) == orc.l1_exact(np.sort(x))
    assert a == math.fsum(np.abs(x.astype(np.float64)).tolist())


# ------------------------------------------------------------------ scaled sign

def test_sign_closed_form_appendix_a():
    """||C(x) - x||^2 = ||x||^2 - ||x||_1^2 / d  (Appendix A, scaled sign, an equality)."""
    rng = np.random.default_rng(4)
    for d in (1, 2, 31, 32, 33, 1000, 4097):
        x = rng.standard_normal(d).astype(np.float32)
        bits, scales, c = orc.compress_sign(x)
        x64, c64 = x.astype(np.float64), c.astype(np.float64)
        lhs = np.sum((c64 - x64) ** 2)
        rhs = np.sum(x64 ** 2) - np.sum(np.abs(x64)) ** 2 / d
        assert lhs == pytest.approx(rhs, rel=1e-6, abs=1e-9)
        # payload: exactly d sign bits and one 32-bit scale
        assert bits.size == (d + 31) // 32 and scales.size == 1
        unpacked = (bits[np.arange(d) // 32] >> (np.arange(d) % 32)) & 1
        assert np.array_equal(unpacked.astype(bool), x >= 0)
        if d % 32:
            assert bits[-1] >> (d % 32) == 0
        assert np.array_equal(c, np.where(x >= 0, scales[0], -scales[0]).astype(np.float32))
        assert scales[0] == np.float32(math.fsum(abs(float(v)) for v in x) / d)


def test_sign_gaussian_limits():
    """Half-normal mean: scale -> sigma sqrt(2/pi); error ratio -> 1 - 2/pi."""
    rng = np.random.default_rng(5)
    sigma = 0.37
    x = (rng.standard_normal(2_000_000) * sigma).astype(np.float32)
    _, scales, c = orc.compress_sign(x)
    assert scales[0] == pytest.approx(sigma * math.sqrt(2 / math.pi), rel=3e-3)
    ratio = np.sum((c.astype(np.float64) - x) ** 2) / np.sum(x.astype(np.float64) ** 2)
    assert ratio == pytest.approx(1 - 2 / math.pi, rel=5e-3)


def test_sign_zero_maps_to_plus_and_zero_vector():
    bits, scales, c = orc.compress_sign(np.array([0.0, -0.0, -1.0, 2.0], dtype=np.float32))
    assert bits[0] == 0b1011 and scales[0] == np.float32(0.75)
    bits, scales, c = orc.compress_sign(np.zeros(40, dtype=np.float32))
    assert scales[0] == 0 and np.all(c == 0) and bits[0] == 0xFFFFFFFF and bits[1] == 0xFF


def test_sign_segments_equal_flat_on_slices():
    rng = np.random.default_rng(6)
    d = 1000
    off = np.array([0, 1, 34, 64, 65, 500, 997, 1000])
    x = (rng.standard_normal(d) * np.repeat(rng.uniform(1e-3, 10, 7), np.diff(off))).astype(np.float32)
    bits, scales, c = orc.compress_sign(x, off)
    fb, _, _ = orc.compress_sign(x)
    assert np.array_equal(bits, fb)                      # bits do not depend on segments
    for r in range(7):
        _, s, cs = orc.compress_sign(x[off[r]:off[r + 1]])
        assert scales[r] == s[0]
        assert np.array_equal(c[off[r]:off[r + 1]], cs)


# ------------------------------------------------------------------ top-k

def brute_topk(x, k):
    order = sorted(range(len(x)), key=lambda j: (-abs(float(x[j])), j))
    return sorted(order[:k])


def test_topk_brute_force_small_all_k_with_ties():
    rng = np.random.default_rng(7)
    for d in list(range(1, 20)) + [33, 64]:
        for trial in range(3):
            # few distinct magnitudes -> many ties
            x = (rng.integers(-3, 4, d) * 0.5).astype(np.float32)
            for k in range(1, d + 1):
                idx, val, c = orc.compress_topk(x, k)
                want = brute_topk(x, k)
                assert idx.tolist() == want
                assert np.array_equal(val, x[want])
                dense = np.zeros(d, np.float32)
                dense[want] = x[want]
                assert np.array_equal(c, dense)


def test_topk_inequality_appendix_a():
    """||C(x) - x||^2 <= (1 - k/d) ||x||^2 (Appendix A, top-k, squared on both sides)."""
    rng = np.random.default_rng(8)
    for d, k in ((100, 1), (100, 50), (1000, 10), (1000, 999), (257, 257)):
        x = rng.standard_normal(d).astype(np.float32)
        idx, val, c = orc.compress_topk(x, k)
        assert idx.size == k and np.all(np.diff(idx.astype(np.int64)) > 0) and idx[-1] < d
        err = np.sum((c.astype(np.float64) - x) ** 2)
        assert err <= (1 - k / d) * np.sum(x.astype(np.float64) ** 2) + 1e-12
        # every kept magnitude dominates every dropped one
        dropped = np.setdiff1d(np.arange(d), idx)
        if dropped.size:
            assert np.abs(x[idx]).min() >= np.abs(x[dropped]).max()


def test_topk_worked_example_ties():
    gold = read_golden("worked_example_topk.txt")
    d, k = int(gold["d"][0]), int(gold["k"][0])
    g = np.array(gold["g"], dtype=np.float32)
    o = orc.Oracle(d, 1, orc.TOPK, k=k)
    for t in (1, 2):
        o.step(g[None, :])
        idx, val = o.payload(0)
        assert idx.tolist() == gold["t%d.idx" % t]
        assert val.tolist() == gold["t%d.val" % t]
        assert o.state("ghat_w")[0].tolist() == gold["t%d.ghat" % t]


# ------------------------------------------------------------------ whole step

def test_sign_worked_example_two_iterations():
    gold = read_golden("worked_example_sign.txt")
    n, d = int(gold["n"][0]), int(gold["d"][0])
    o = orc.Oracle(d, n, orc.SIGN, beta1=gold["beta1"][0], beta2=gold["beta2"][0],
                   lr=gold["alpha"][0], eps=gold["nu"][0], x0=gold["x1"])
    for t in (1, 2):
        p = "t%d." % t
        o.step(np.array([gold[p + "g0"], gold[p + "g1"]], dtype=np.float32))
        for i in range(n):
            bits, scales = o.payload(i)
            assert scales[0] == gold[p + "w%d.scale" % i][0]
            assert bits[0] == gold[p + "w%d.word" % i][0]
            assert o.state("ghat_w")[i].tolist() == gold[p + "w%d.ghat" % i]
        bits, scales = o.payload(-1)
        assert scales[0] == gold[p + "s.scale"][0] and bits[0] == gold[p + "s.word"][0]
        assert o.state("ghat_s").tolist() == gold[p + "s.ghat"]
        assert o.state("gtil").tolist() == gold[p + "gtil"]
        assert o.state("m").tolist() == gold[p + "m"]
        assert o.state("v").tolist() == gold[p + "v"]
        assert o.state("vhat").tolist() == gold[p + "vhat"]
        if t == 1:
            assert o.state("x").tolist() == gold[p + "x"]
        else:
            np.testing.assert_allclose(o.state("x"), gold[p + "x"], rtol=0, atol=1.5e-7)   # fixture has 7 digits
            # and to full binary32 accuracy from the exact expression
            want = [0.75 - 0.5 * 1.0 / math.sqrt(223 / 128), 1.25 + 0.5 * 0.125 / 0.75,
                    0.75 - 0.5 * 1.0 / math.sqrt(223 / 128), 1.25 + 0.5 * 1.0 / math.sqrt(223 / 128)]
            np.testing.assert_allclose(o.state("x"), want, rtol=2e-7)


def vanilla_amsgrad(x0, grads_mean, b1, b2, lr, nu):
    """Distributed AMSGrad of the paper's Section 3, written independently in numpy fp32."""
    f = np.float32
    x = x0.astype(f).copy()
    m = np.zeros_like(x); v = np.zeros_like(x); vh = np.zeros_like(x)
    b1, b2, lr, nu = f(b1), f(b2), f(lr), f(nu)
    for g in grads_mean:
        g = g.astype(f)
        m = b1 * m + (f(1) - b1) * g
        v = b2 * v + (f(1) - b2) * (g * g)
        vh = np.maximum(vh, v)
        x = x - (lr * m) / np.sqrt(vh + nu)
    return x, m, v, vh


@pytest.mark.parametrize("mode", [orc.MARKOV, orc.EF])
def test_identity_compressor_is_vanilla_amsgrad(mode):
    rng = np.random.default_rng(9)
    d, n, T = 513, 4, 6
    x0 = (rng.standard_normal(d) * 0.02).astype(np.float32)
    G = rng.standard_normal((T, n, d)).astype(np.float32)
    o = orc.Oracle(d, n, orc.IDENTITY, beta1=0.9, beta2=0.99, lr=1e-2, eps=1e-8, x0=x0, mode=mode)
    means = []
    for t in range(T):
        o.step(G[t])
        acc = np.zeros(d, np.float32)
        for i in range(n):
            acc = acc + G[t, i]
        means.append(acc / np.float32(n))
        if t == 0:
            x, m, v, vh = vanilla_amsgrad(x0, means, 0.9, 0.99, 1e-2, 1e-8)
            assert np.array_equal(o.state("x"), x) and np.array_equal(o.state("m"), m)
            assert np.array_equal(o.state("v"), v) and np.array_equal(o.state("vhat"), vh)
    x, m, v, vh = vanilla_amsgrad(x0, means, 0.9, 0.99, 1e-2, 1e-8)
    if mode == orc.EF:          # error terms stay exactly zero: bitwise reduction
        assert np.array_equal(o.state("x"), x) and np.array_equal(o.state("vhat"), vh)
        assert not o.state("ghat_w").any() and not o.state("gtil").any()
    else:                       # ghat + fl(g - ghat) is g only to an ulp after step 1
        np.testing.assert_allclose(o.state("m"), m, rtol=1e-5, atol=1e-7)
        np.testing.assert_allclose(o.state("vhat"), vh, rtol=1e-5, atol=1e-9)
        np.testing.assert_allclose(o.state("x"), x, rtol=0, atol=1e-6)


def decode_sign(bits, scales, off, d):
    j = np.arange(d)
    b = ((bits[j // 32] >> (j % 32)) & 1).astype(bool)
    s = np.repeat(scales, np.diff(off)).astype(np.float32)
    return np.where(b, s, -s).astype(np.float32)


@pytest.mark.parametrize("comp", [orc.SIGN, orc.TOPK])
def test_markov_identity_contraction_and_invariants(comp):
    """ghat_t - ghat_{t-1} = c_t bit-exactly (decoded from the payload), the contraction of
    the Markov sequence (equality for scaled sign with pi from Appendix A), vhat monotone,
    |x_{t+1} - x_t| <= alpha |m| / sqrt(nu), and the n = 1 server equals the worker."""
    rng = np.random.default_rng(10)
    d, n, k, T = 777, 3, 20, 8
    off = np.array([0, 100, 131, 777])
    kw = dict(offsets=off) if comp == orc.SIGN else dict(k=k)
    x0 = (rng.standard_normal(d) * 0.02).astype(np.float32)
    o = orc.Oracle(d, n, comp, lr=1e-3, eps=1e-8, x0=x0, **kw)
    base = rng.standard_normal((n, d)).astype(np.float32)
    prev = {name: o.state(name).copy() for name in orc.STATE_NAMES}
    for t in range(T):
        g = base + 0.3 * rng.standard_normal((n, d)).astype(np.float32)
        o.step(g)
        acc = np.zeros(d, np.float32)
        for i in range(n):
            u = g[i] - prev["ghat_w"][i]
            if comp == orc.SIGN:
                bits, scales = o.payload(i)
                c = decode_sign(bits, scales, off, d)
                for r in range(3):      # contraction, equality form, per segment
                    sl = slice(off[r], off[r + 1])
                    u64 = u[sl].astype(np.float64)
                    pi_r = 1 - np.sum(np.abs(u64)) ** 2 / (u64.size * np.sum(u64 ** 2))
                    err = np.sum((o.state("ghat_w")[i][sl].astype(np.float64) - g[i][sl]) ** 2)
                    assert err == pytest.approx(pi_r * np.sum(u64 ** 2), rel=1e-4)
            else:
                idx, val = o.payload(i)
                assert np.array_equal(val, u[idx])
                c = np.zeros(d, np.float32); c[idx] = val
                err = np.sum((o.state("ghat_w")[i].astype(np.float64) - g[i]) ** 2)
                assert err <= (1 - k / d) * np.sum(u.astype(np.float64) ** 2) * (1 + 1e-6)
            assert np.array_equal(o.state("ghat_w")[i], prev["ghat_w"][i] + c)
            acc = acc + c
        assert np.array_equal(o.state("ghat_s"), prev["ghat_s"] + acc / np.float32(n))
        if comp == orc.SIGN:
            c = decode_sign(*o.payload(-1), off, d)
        else:
            idx, val = o.payload(-1)
            assert np.array_equal(val, (o.state("ghat_s") - prev["gtil"])[idx])
            c = np.zeros(d, np.float32); c[idx] = val
        assert np.array_equal(o.state("gtil"), prev["gtil"] + c)
        assert np.all(o.state("vhat") >= prev["vhat"]) and np.all(o.state("vhat") >= o.state("v"))
        dx = np.abs(o.state("x").astype(np.float64) - prev["x"])
        assert np.all(dx <= 1e-3 * np.abs(o.state("m")) / math.sqrt(1e-8) * (1 + 1e-5) + 1e-9)
        prev = {name: o.state(name).copy() for name in orc.STATE_NAMES}


def test_first_step_closed_form_and_single_worker():
    """Zero initial state: ghat_1^(i) = C(g_1^(i)); with n = 1 the server aggregate equals
    the worker state bit for bit."""
    rng = np.random.default_rng(11)
    d = 300
    g = rng.standard_normal((1, d)).astype(np.float32)
    o = orc.Oracle(d, 1, orc.SIGN)
    o.step(g)
    _, _, c = orc.compress_sign(g[0])
    assert np.array_equal(o.state("ghat_w")[0], c)
    assert np.array_equal(o.state("ghat_s"), o.state("ghat_w")[0])
    for _ in range(4):
        o.step(rng.standard_normal((1, d)).astype(np.float32))
    # n = 1: ghat_s accumulates the same c as ghat_w, in the same order
    assert np.array_equal(o.state("ghat_s"), o.state("ghat_w")[0])
    # identical gradients on every worker: average of equal payloads is the payload (n = 4)
    o4 = orc.Oracle(d, 4, orc.SIGN)
    o1 = orc.Oracle(d, 1, orc.SIGN)
    for _ in range(3):
        g = rng.standard_normal((1, d)).astype(np.float32)
        o4.step(np.repeat(g, 4, axis=0)); o1.step(g)
        assert np.array_equal(o4.state("x"), o1.state("x"))


def test_topk_constant_gradient_converges_exactly():
    """With a fixed gradient and top-k, every coordinate is transmitted once: after
    ceil(d/k) steps ghat = g exactly and all later payload values are zero."""
    rng = np.random.default_rng(12)
    d, k = 103, 10
    g = rng.standard_normal((1, d)).astype(np.float32)
    o = orc.Oracle(d, 1, orc.TOPK, k=k)
    for _ in range(-(-d // k)):
        o.step(g)
    assert np.array_equal(o.state("ghat_w")[0], g[0])
    o.step(g)
    assert not o.payload(0)[1].any()


def test_error_feedback_reconstruction():
    """Classical error feedback: delta_new + C(g + delta) gives back g + delta, exactly
    for top-k and identity, to rounding for scaled sign."""
    rng = np.random.default_rng(13)
    d, n = 200, 2
    for comp, kw in ((orc.TOPK, dict(k=7)), (orc.SIGN, {}), (orc.IDENTITY, {})):
        o = orc.Oracle(d, n, comp, mode=orc.EF, **kw)
        for _ in range(4):
            delta = o.state("ghat_w").copy()
            g = rng.standard_normal((n, d)).astype(np.float32)
            o.step(g)
            for i in range(n):
                p = g[i] + delta[i]
                if comp == orc.TOPK:
                    idx, val = o.payload(i)
                    c = np.zeros(d, np.float32); c[idx] = val
                    assert np.array_equal(o.state("ghat_w")[i] + c, p)
                elif comp == orc.SIGN:
                    c = decode_sign(*o.payload(i), np.array([0, d]), d)
                    np.testing.assert_allclose(o.state("ghat_w")[i] + c, p, rtol=0, atol=1e-6)
                else:
                    assert not o.state("ghat_w")[i].any()


def test_planted_mistakes_are_caught():
    """The pins above must be able to fail: perturb inputs the way a plausible slip would
    (wrong sign convention, transposed workers) and check the worked example notices."""
    gold = read_golden("worked_example_sign.txt")
    o = orc.Oracle(4, 2, orc.SIGN, beta1=0.5, beta2=0.5, lr=0.5, eps=0.28125, x0=gold["x1"])
    o.step(np.array([gold["t1.g1"], gold["t1.g0"]], dtype=np.float32))   # workers swapped
    assert o.payload(0)[0][0] != gold["t1.w0.word"][0]
    # server result is symmetric in the workers at step 1, so x agrees: the asymmetry shows
    # only from step 2 on, which is why the example has two iterations
    assert o.state("x").tolist() == gold["t1.x"]
    o.step(np.array([gold["t2.g0"], gold["t2.g1"]], dtype=np.float32))
    assert o.state("ghat_s").tolist() != gold["t2.s.ghat"]


# ------------------------------------------------------------------ rand-k

def test_randk_expected_error_appendix_a():
    """E ||C(x) - x||^2 = (1 - k/d) ||x||^2 over the random set (Appendix A, rand-k)."""
    from paper_2111_00705_b200 import synth
    rng = np.random.default_rng(20)
    d, k, draws = 400, 60, 4000
    x = rng.standard_normal(d).astype(np.float32)
    sets = synth.random_sets(d, k, draws, 5, 1)
    err = 0.0
    hits = np.zeros(d)
    for S in sets:
        idx, val, c = orc.compress_randk(x, S)
        assert idx.tolist() == S.tolist() and np.array_equal(val, x[S])
        dense = np.zeros(d, np.float32); dense[S] = x[S]
        assert np.array_equal(c, dense)
        err += np.sum((c.astype(np.float64) - x) ** 2)
        hits[S] += 1
    want = (1 - k / d) * np.sum(x.astype(np.float64) ** 2)
    assert err / draws == pytest.approx(want, rel=0.02)
    # every coordinate is drawn with probability k/d
    assert np.all(np.abs(hits / draws - k / d) < 5 * math.sqrt(k / d * (1 - k / d) / draws))


def test_randk_reduces_to_topk_and_identity_on_their_sets():
    """With S = the top-k set the iteration equals the top-k one; with S = everything it
    equals the identity compressor's (both already pinned), bit for bit."""
    rng = np.random.default_rng(21)
    d, n, k = 300, 3, 25
    a = orc.Oracle(d, n, orc.TOPK, k=k)
    b = orc.Oracle(d, n, orc.RANDK, k=k)
    for t in range(4):
        g = rng.standard_normal((n, d)).astype(np.float32)
        # the sets top-k will choose, computed from the states before the step
        W = np.stack([orc.compress_topk(g[i] - a.state("ghat_w")[i], k)[0] for i in range(n)])
        a.step(g)
        b.set_random_sets(W, a.payload(-1)[0])
        b.step(g)
        for name in orc.STATE_NAMES:
            assert np.array_equal(a.state(name), b.state(name)), name
        assert np.array_equal(a.payload(1)[1], b.payload(1)[1])
    full = np.arange(d, dtype=np.uint32)
    c = orc.Oracle(d, n, orc.IDENTITY)
    e = orc.Oracle(d, n, orc.RANDK, k=d)
    for t in range(3):
        g = rng.standard_normal((n, d)).astype(np.float32)
        e.set_random_sets(np.tile(full, (n, 1)), full)
        c.step(g); e.step(g)
        for name in orc.STATE_NAMES:
            assert np.array_equal(c.state(name), e.state(name)), name


# ------------------------------------------------------------------ naive compression mode

def test_naive_mode_worked_example():
    """AMSGrad with naive compression, both directions, hand-worked (golden file)."""
    gold = read_golden("worked_example_naive.txt")
    n, d = int(gold["n"][0]), int(gold["d"][0])
    o = orc.Oracle(d, n, orc.SIGN, beta1=gold["beta1"][0], beta2=gold["beta2"][0],
                   lr=gold["alpha"][0], eps=gold["nu"][0], x0=gold["x1"], mode=orc.NAIVE)
    for t in (1, 2):
        p = "t%d." % t
        o.step(np.array([gold[p + "g0"], gold[p + "g1"]], dtype=np.float32))
        for i in range(n):
            bits, scales = o.payload(i)
            assert scales[0] == gold[p + "w%d.scale" % i][0] and bits[0] == gold[p + "w%d.word" % i][0]
        bits, scales = o.payload(-1)
        assert scales[0] == gold[p + "s.scale"][0] and bits[0] == gold[p + "s.word"][0]
        for name in ("m", "v", "vhat"):
            assert o.state(name).tolist() == gold[p + name]
        if t == 1:
            assert o.state("x").tolist() == gold[p + "x"]
        else:
            np.testing.assert_allclose(o.state("x"), gold[p + "x"], rtol=0, atol=1.5e-7)
            r = 0.5 * 0.8125 / math.sqrt(77 / 64)
            np.testing.assert_allclose(o.state("x"), [0.75 - r, 1.25 + r, 0.75 - r, 1.25 + r], rtol=2e-7)
        for name in ("ghat_w", "ghat_s", "gtil"):
            assert not o.state(name).any()             # the scheme keeps no compression state


@pytest.mark.parametrize("comp", [orc.SIGN, orc.TOPK, orc.IDENTITY])
def test_naive_mode_is_stateless_and_first_step_equals_algorithm_1(comp):
    rng = np.random.default_rng(31)
    d, n, k = 300, 3, 17
    G = rng.standard_normal((4, n, d)).astype(np.float32)
    x0 = rng.standard_normal(d).astype(np.float32)
    a = orc.Oracle(d, n, comp, k=k, x0=x0, mode=orc.NAIVE)
    b = orc.Oracle(d, n, comp, k=k, x0=x0, mode=orc.MARKOV)
    a.step(G[0]); b.step(G[0])
    for name in ("m", "v", "vhat", "x"):               # from zero state Algorithm 1 sends C(g) too
        assert np.array_equal(a.state(name), b.state(name)), name
    # payloads of a later step depend on that step's gradients only: a fresh context that is
    # given the moments and x reproduces step 3 without having seen steps 1 and 2
    a.step(G[1])
    snap = {name: a.state(name).copy() for name in ("m", "v", "vhat", "x")}
    a.step(G[2])
    c = orc.Oracle(d, n, comp, k=k, mode=orc.NAIVE)
    for name, val in snap.items():
        c.state(name)[:] = val
    c.step(G[2])
    for name in ("m", "v", "vhat", "x"):
        assert np.array_equal(a.state(name), c.state(name)), name
    if comp != orc.IDENTITY:
        for who in list(range(n)) + [-1]:
            pa, pc = a.payload(who), c.payload(who)
            assert np.array_equal(pa[0], pc[0]) and np.array_equal(pa[1], pc[1])
        # worker payload = the compressor applied to the gradient itself
        if comp == orc.SIGN:
            bits, scales, _ = orc.compress_sign(G[2, 1])
            assert np.array_equal(a.payload(1)[0], bits) and np.array_equal(a.payload(1)[1], scales)
        else:
            order = sorted(range(d), key=lambda j: (-abs(float(G[2, 1, j])), j))[:k]
            assert sorted(order) == a.payload(1)[0].tolist()
    else:                                              # identity: vanilla AMSGrad, bit for bit
        means = []
        for t in range(3):
            acc = np.zeros(d, np.float32)
            for i in range(n):
                acc = acc + G[t, i]
            means.append(acc / np.float32(n))
        x, m, v, vh = vanilla_amsgrad(x0, means, 0.9, 0.999, 1e-3, 1e-8)
        assert np.array_equal(a.state("x"), x) and np.array_equal(a.state("vhat"), vh)


# ------------------------------------------------------------------ weight decay, milestones

def test_weight_decay_closed_form_at_zero_gradient():
    """With g = 0 the moments stay 0 and x_{t+1} = x_t - (alpha lambda) x_t: for
    alpha = lambda = 1/2 every x_t = (3/4)^(t-1) x_1 is exact in binary32 for small t."""
    d, n = 5, 2
    x1 = np.array([1.0, -2.0, 0.5, 3.0, 0.0], np.float32)
    o = orc.Oracle(d, n, orc.IDENTITY, lr=0.5, eps=1.0, x0=x1)
    o.set_weight_decay(0.5)
    for t in range(1, 11):
        o.step(np.zeros((n, d), np.float32))
        want = [float(Fraction(3, 4) ** t * Fraction(float(x))) for x in x1]
        assert o.state("x").tolist() == want
        assert not o.state("m").any() and not o.state("vhat").any()


def decayed_amsgrad(x0, grads, lrs, b1, b2, nu, wd):
    """AMSGrad with decoupled weight decay and a per-step step size, written independently."""
    f = np.float32
    x = x0.astype(f).copy()
    m = np.zeros_like(x); v = np.zeros_like(x); vh = np.zeros_like(x)
    b1, b2, nu, wd = f(b1), f(b2), f(nu), f(wd)
    for g, lr in zip(grads, lrs):
        lr = f(lr)
        m = b1 * m + (f(1) - b1) * g
        v = b2 * v + (f(1) - b2) * (g * g)
        vh = np.maximum(vh, v)
        step = (lr * m) / np.sqrt(vh + nu)
        x = (x - step) - (lr * wd) * x if wd != 0 else x - step
    return x, m, v, vh


@pytest.mark.parametrize("wd", [0.0, 5e-4, 0.1])
def test_weight_decay_and_lr_milestones_against_independent_recursion(wd):
    rng = np.random.default_rng(44)
    d, T = 257, 7
    x0 = rng.standard_normal(d).astype(np.float32)
    G = rng.standard_normal((T, 1, d)).astype(np.float32)
    f = np.float32
    base, gamma = f(1e-2), f(0.1)
    # milestones after 2 and after 5 completed steps: steps 1-2 base, 3-5 base*gamma, 6-7 base*gamma^2
    lrs = [base] * 2 + [base * gamma] * 3 + [(base * gamma) * gamma] * 2
    o = orc.Oracle(d, 1, orc.IDENTITY, beta2=0.99, lr=123.0, x0=x0, mode=orc.EF)   # EF + identity: exact
    o.set_weight_decay(wd)
    o.set_lr_milestones(base, [2, 5], gamma)
    p = orc.Oracle(d, 1, orc.IDENTITY, beta2=0.99, lr=float(base), x0=x0, mode=orc.EF)
    p.set_weight_decay(wd)
    for t in range(T):
        o.step(G[t])
        p.set_lr(float(lrs[t]))                        # the same schedule by explicit calls
        p.step(G[t])
    x, m, v, vh = decayed_amsgrad(x0, G[:, 0], lrs, 0.9, 0.99, 1e-8, wd)
    for side in (o, p):
        assert np.array_equal(side.state("x"), x) and np.array_equal(side.state("m"), m)
        assert np.array_equal(side.state("vhat"), vh)
    if wd:                                             # the decay really acts
        q = decayed_amsgrad(x0, G[:, 0], lrs, 0.9, 0.99, 1e-8, 0.0)[0]
        assert not np.array_equal(q, x)
    with pytest.raises(ValueError):
        o.set_lr_milestones(base, [5, 2], gamma)       # not increasing
    with pytest.raises(ValueError):
        o.set_lr_milestones(base, [2], 1.5)            # alpha_t must not increase
    with pytest.raises(ValueError):
        o.set_weight_decay(-1.0)


# ------------------------------------------------------------------ top-k per segment

def test_topk_per_segment_brute_force_and_reduction_to_whole_vector():
    """Top-k on every segment on its own: against a Python sort of every segment (ties to the
    lower index), against the whole-vector compressor on the slices, and with one segment
    against the whole-vector step."""
    rng = np.random.default_rng(77)
    d, n = 97, 3
    off = np.array([0, 5, 6, 40, 41, 97])
    ks = np.array([2, 1, 7, 1, 20])
    G = np.round(rng.standard_normal((3, n, d)) * 3).astype(np.float32) / 2        # many ties
    o = orc.Oracle(d, n, orc.TOPK, k=1)
    o.set_topk_segments(off, ks)
    prev = np.zeros((n, d), np.float32)
    for t in range(3):
        o.step(G[t])
        for i in range(n):
            u = G[t, i] - prev[i]
            idx, val = o.payload(i)
            assert idx.size == ks.sum() and np.all(np.diff(idx.astype(np.int64)) > 0)
            want = []
            for r in range(len(ks)):
                lo, hi = off[r], off[r + 1]
                order = sorted(range(lo, hi), key=lambda j: (-abs(float(u[j])), j))[:ks[r]]
                want += sorted(order)
                # the whole-vector compressor on the slice gives the same entries
                si, sv, _ = orc.compress_topk(u[lo:hi], int(ks[r]))
                assert (si + lo).tolist() == sorted(order)
            assert idx.tolist() == want
            assert np.array_equal(val, u[idx])
            dec = np.zeros(d, np.float32); dec[idx] = val
            assert np.array_equal(o.state("ghat_w")[i], prev[i] + dec)          # Markov identity
        prev = o.state("ghat_w").copy()
    # one segment holding everything = the compressor of Appendix A on the whole vector
    a = orc.Oracle(d, n, orc.TOPK, k=9); a.set_topk_segments([0, d], [9])
    b = orc.Oracle(d, n, orc.TOPK, k=9)
    for t in range(3):
        a.step(G[t]); b.step(G[t])
    for name in orc.STATE_NAMES:
        assert np.array_equal(a.state(name), b.state(name)), name
    with pytest.raises(ValueError):
        orc.Oracle(d, n, orc.TOPK, k=1).set_topk_segments([0, 5, d], [6, 1])     # k_r > |S_r|
    with pytest.raises(ValueError):
        orc.Oracle(d, n, orc.SIGN).set_topk_segments([0, d], [1])


# ------------------------------------------------------------------ error feedback, server half

def run_ef_example(o, gold, steps=(1, 2, 3)):
    """Drive the oracle through the hand-worked error-feedback example; returns the list of
    (key, got, want) triples that differ, so a planted mistake can be shown to be noticed."""
    n = int(gold["n"][0])
    bad = []

    def chk(key, got, atol=0.0):
        want = gold[key]
        got = np.atleast_1d(np.asarray(got, dtype=np.float64))
        if got.shape != (len(want),) or np.any(np.abs(got - np.asarray(want)) > atol):
            bad.append((key, got.tolist(), want))

    for t in steps:
        p = "t%d." % t
        o.step(np.array([gold[p + "g0"], gold[p + "g1"]], dtype=np.float32))
        for i in range(n):
            bits, scales = o.payload(i)
            chk(p + "w%d.scale" % i, scales[0])
            chk(p + "w%d.word" % i, bits[0])
            chk(p + "w%d.delta" % i, o.state("ghat_w")[i])
        bits, scales = o.payload(-1)
        chk(p + "s.scale", scales[0])
        chk(p + "s.word", bits[0])
        chk(p + "s.delta", o.state("gtil"))
        # delta + c gives back what the server compressed: mean plus the old error
        c = decode_sign(bits, scales, np.array([0, 4]), 4)
        chk(p + "s.p", o.state("gtil") + c)
        for name in ("m", "v", "vhat"):
            chk(p + name, o.state(name))
        chk(p + "x", o.state("x"), atol=0.0 if t == 1 else 1.5e-7)   # 7 digits in the fixture
    return bad


def ef_example_oracle(gold):
    return orc.Oracle(int(gold["d"][0]), int(gold["n"][0]), orc.SIGN, beta1=gold["beta1"][0],
                      beta2=gold["beta2"][0], lr=gold["alpha"][0], eps=gold["nu"][0],
                      x0=gold["x1"], mode=orc.EF)


def test_error_feedback_worked_example_three_iterations():
    """Section 4, error feedback, both directions, scaled sign: the hand-worked run."""
    gold = read_golden("worked_example_ef.txt")
    o = ef_example_oracle(gold)
    assert run_ef_example(o, gold) == []
    assert not o.state("ghat_s").any()         # this mode keeps one error vector at the server
    # x_4 to binary32 accuracy from the exact expression (x_3 is rounded once on the way)
    r = 0.5 / math.sqrt(223 / 128)
    x3 = [0.75 - r, 1.25 + r, 0.75 - r, 1.25 + r]
    want = [a - b * r for a, b in zip(x3, gold["t3.m"])]
    np.testing.assert_allclose(o.state("x"), want, rtol=0, atol=2.5e-7)


def test_error_feedback_example_notices_a_lost_server_error():
    """The example must be able to fail on the server half: lose the server's error before
    iteration 3 (what dropping the '+ delta' term of the server's input would do) and both the
    server's scale and its sign word leave the hand-worked values; lose it before iteration 2
    and the new error does.  Same for a worker's error."""
    gold = read_golden("worked_example_ef.txt")
    o = ef_example_oracle(gold)
    assert run_ef_example(o, gold, (1, 2)) == []
    o.state("gtil")[:] = 0
    keys = {k for k, _, _ in run_ef_example(o, gold, (3,))}
    assert {"t3.s.scale", "t3.s.word", "t3.s.delta", "t3.s.p", "t3.m", "t3.x"} <= keys
    assert not any(k.startswith("t3.w") for k in keys)      # the workers are untouched by it
    o = ef_example_oracle(gold)
    assert run_ef_example(o, gold, (1,)) == []
    o.state("gtil")[:] = 0
    keys = {k for k, _, _ in run_ef_example(o, gold, (2,))}
    assert "t2.s.delta" in keys and "t2.s.p" in keys
    o = ef_example_oracle(gold)
    assert run_ef_example(o, gold, (1,)) == []
    o.state("ghat_w")[1][:] = 0
    keys = {k for k, _, _ in run_ef_example(o, gold, (2,))}
    assert {"t2.w1.scale", "t2.w1.delta"} <= keys and "t2.w0.scale" not in keys


@pytest.mark.parametrize("comp", [orc.TOPK, orc.SIGN, orc.IDENTITY])
def test_error_feedback_server_recursion(comp):
    """Server half of the error-feedback scheme (Section 4), from the messages alone:
    p = (sum_i c^(i), i ascending) / n + delta_old;  c = C(p);  delta_new = p - c;  the
    moments are driven by c, not by p or by a running estimate."""
    rng = np.random.default_rng(29)
    d, n, k = 240, 3, 9
    off = np.array([0, 70, 101, d])
    kw = dict(k=k) if comp == orc.TOPK else (dict(offsets=off) if comp == orc.SIGN else {})
    b1, b2 = np.float32(0.9), np.float32(0.999)
    o = orc.Oracle(d, n, comp, mode=orc.EF, beta1=float(b1), beta2=float(b2), **kw)
    m_prev = np.zeros(d, np.float32); v_prev = np.zeros(d, np.float32)
    for t in range(5):
        d_old = o.state("gtil").copy()
        dw_old = o.state("ghat_w").copy()
        g = (rng.standard_normal((n, d)) * (1 + 3 * (rng.random((n, d)) < 0.05))).astype(np.float32)
        o.step(g)
        acc = np.zeros(d, np.float32)
        for i in range(n):                         # decode the n messages, add them in order
            if comp == orc.TOPK:
                idx, val = o.payload(i)
                c_i = np.zeros(d, np.float32); c_i[idx] = val
            elif comp == orc.SIGN:
                c_i = decode_sign(*o.payload(i), off, d)
            else:
                c_i = g[i] + dw_old[i]
            acc = acc + c_i
        p = acc / np.float32(n) + d_old
        if comp == orc.TOPK:
            idx, val = o.payload(-1)
            order = sorted(range(d), key=lambda j: (-abs(float(p[j])), j))[:k]
            assert idx.tolist() == sorted(order)
            assert np.array_equal(val, p[idx])
            c = np.zeros(d, np.float32); c[idx] = val
            assert np.array_equal(o.state("gtil") + c, p)            # exact: c is p where kept
            assert not o.state("gtil")[idx].any()
        elif comp == orc.SIGN:
            bits, scales = o.payload(-1)
            for r in range(3):
                seg = p[off[r]:off[r + 1]]
                assert scales[r] == np.float32(math.fsum(abs(float(z)) for z in seg) / seg.size)
            c = decode_sign(bits, scales, off, d)
            assert np.array_equal(c >= 0, p >= 0)
        else:
            c = p
        assert np.array_equal(o.state("gtil"), p - c)
        m = b1 * m_prev + (np.float32(1) - b1) * c
        v = b2 * v_prev + (np.float32(1) - b2) * (c * c)
        assert np.array_equal(o.state("m"), m) and np.array_equal(o.state("v"), v)
        m_prev, v_prev = m, v
    assert not o.state("ghat_s").any()


# ------------------------------------------------------------------ scales given from outside

def forced_pair(rng, n=3, d=333, off=(0, 50, 81, 200, 333), mode=orc.MARKOV):
    off = np.array(off)
    x0 = (rng.standard_normal(d) * 0.02).astype(np.float32)
    free = orc.Oracle(d, n, orc.SIGN, offsets=off, x0=x0, mode=mode)
    given = orc.Oracle(d, n, orc.SIGN, offsets=off, x0=x0, mode=mode)
    return off, free, given


def test_given_scales_reproduce_the_computed_run():
    """An oracle handed the scales another one computed (the sampled full-size checks use this
    branch) repeats that run bit for bit: every sign word, scale and state vector, and each
    decoded coordinate is plus or minus the given scale of its segment."""
    rng = np.random.default_rng(41)
    n, d = 3, 333
    off, free, given = forced_pair(rng)
    q = off.size - 1
    for t in range(3):
        g = (rng.standard_normal((n, d)) * np.repeat([1.0, 1e-2, 30.0, 0.3], np.diff(off))).astype(np.float32)
        prev_w = given.state("ghat_w").copy(); prev_t = given.state("gtil").copy()
        free.step(g)
        ws = np.stack([free.payload(i)[1] for i in range(n)])        # n x q, row i = worker i
        ss = free.payload(-1)[1]
        given.force_scales(ws, ss)
        given.step(g)
        for who in list(range(n)) + [-1]:
            for a, b in zip(free.payload(who), given.payload(who)):
                assert np.array_equal(a, b)
        for name in orc.STATE_NAMES:
            assert np.array_equal(free.state(name), given.state(name)), name
        for i in range(n):                      # c_j = +-given[i][r] by segment, written out
            u = g[i] - prev_w[i]
            for r in range(q):
                sl = slice(off[r], off[r + 1])
                want = np.where(u[sl] >= 0, ws[i, r], -ws[i, r]).astype(np.float32)
                assert np.array_equal(prev_w[i][sl] + want, given.state("ghat_w")[i][sl])
        w = given.state("ghat_s") - prev_t
        for r in range(q):
            sl = slice(off[r], off[r + 1])
            want = np.where(w[sl] >= 0, ss[r], -ss[r]).astype(np.float32)
            assert np.array_equal(prev_t[sl] + want, given.state("gtil")[sl])
    # a sample of the coordinates with the full problem's scales follows the full run there
    pick = np.sort(rng.choice(d, 60, replace=False))
    seg_of = np.searchsorted(off, pick, side="right") - 1
    sub_off = np.concatenate([[0], np.cumsum(np.bincount(seg_of, minlength=q))])
    assert np.all(np.diff(sub_off) > 0)
    full = orc.Oracle(d, n, orc.SIGN, offsets=off)
    sub = orc.Oracle(pick.size, n, orc.SIGN, offsets=sub_off)
    for t in range(3):
        g = rng.standard_normal((n, d)).astype(np.float32)
        full.step(g)
        sub.force_scales(np.stack([full.payload(i)[1] for i in range(n)]), full.payload(-1)[1])
        sub.step(g[:, pick])
        for name in orc.STATE_NAMES:
            assert np.array_equal(full.state(name)[..., pick], sub.state(name)), name
    # back to computed scales
    sub.force_scales(None, None)
    sub.step(g[:, pick])
    assert not np.array_equal(sub.payload(-1)[1], full.payload(-1)[1])


@pytest.mark.parametrize("mistake", ["rows_swapped", "server_for_worker", "one_doubled",
                                     "segments_reversed"])
def test_given_scales_planted_mistakes_change_the_state(mistake):
    """Hand the scales over wrongly, the way a slip in that branch would use them (worker rows
    exchanged, the server's scales used for a worker, one scale doubled, segment order
    reversed): the worker states or the second Markov state must leave the computed run."""
    rng = np.random.default_rng(43)
    n, d = 3, 333
    off, free, given = forced_pair(rng)
    sig = np.repeat([1.0, 1e-2, 30.0, 0.3], np.diff(off))
    for t in range(2):
        g = (rng.standard_normal((n, d)) * sig * (1 + np.arange(n))[:, None]).astype(np.float32)
        free.step(g)
        ws = np.stack([free.payload(i)[1] for i in range(n)]); ss = free.payload(-1)[1]
        if t == 1:
            if mistake == "rows_swapped":
                ws = ws[[1, 0, 2]]
            elif mistake == "server_for_worker":
                ws = ws.copy(); ws[2] = ss
            elif mistake == "one_doubled":
                ss = ss.copy(); ss[1] *= 2
            else:
                ws = ws[:, ::-1]; ss = ss[::-1]
        given.force_scales(ws, ss)
        given.step(g)
    if mistake == "one_doubled":
        assert np.array_equal(free.state("ghat_w"), given.state("ghat_w"))
        sl = slice(off[1], off[2])
        assert not np.array_equal(free.state("gtil")[sl], given.state("gtil")[sl])
        assert np.array_equal(free.state("gtil")[:off[1]], given.state("gtil")[:off[1]])
    else:
        assert not np.array_equal(free.state("ghat_w"), given.state("ghat_w"))
        assert not np.array_equal(free.state("gtil"), given.state("gtil"))
