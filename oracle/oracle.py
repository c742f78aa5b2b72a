"""ctypes front end of the CPU oracle (test infrastructure, see ``cdadam_oracle.c``).

Argument marshalling only: every number comes from the C file.  The shared object is built
with gcc into ``oracle/_build`` on first use (``-O2 -ffp-contract=off``: one rounding per
operation, no fused multiply-add).
"""
import ctypes
import os
import subprocess

import numpy as np

SIGN, TOPK, IDENTITY, RANDK = 0, 1, 2, 3
MARKOV, EF, NAIVE = 0, 1, 2
STATE_NAMES = ("ghat_w", "ghat_s", "gtil", "m", "v", "vhat", "x")

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cdadam_oracle.c")
_OUT = os.path.join(_HERE, "_build", "libcdadam_oracle.so")
_lib = None


def build(force=False):
    """Compile the oracle with gcc; returns the path of the shared object."""
    if (not force and os.path.exists(_OUT)
            and os.path.getmtime(_OUT) >= os.path.getmtime(_SRC)):
        return _OUT
    os.makedirs(os.path.dirname(_OUT), exist_ok=True)
    tmp = _OUT + ".%d.tmp" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11",
                           "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _OUT)
    return _OUT


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c = ctypes
    fp, up, ip = c.POINTER(c.c_float), c.POINTER(c.c_uint32), c.POINTER(c.c_int64)
    lib.oracle_l1_exact.restype = c.c_double
    lib.oracle_l1_exact.argtypes = [fp, c.c_int64]
    lib.oracle_compress_sign.restype = None
    lib.oracle_compress_sign.argtypes = [fp, c.c_int64, c.c_int, ip, up, fp, fp]
    lib.oracle_compress_topk.restype = None
    lib.oracle_compress_topk.argtypes = [fp, c.c_int64, c.c_int64, up, fp, fp]
    lib.oracle_create.restype = c.c_void_p
    lib.oracle_create.argtypes = [c.c_int64, c.c_int, c.c_int, c.c_int64,
                                  c.c_float, c.c_float, c.c_float, c.c_float]
    lib.oracle_destroy.restype = None
    lib.oracle_destroy.argtypes = [c.c_void_p]
    lib.oracle_set_segments.restype = c.c_int
    lib.oracle_set_segments.argtypes = [c.c_void_p, c.c_int, ip]
    lib.oracle_set_topk_segments.restype = c.c_int
    lib.oracle_set_topk_segments.argtypes = [c.c_void_p, c.c_int, ip, ip]
    lib.oracle_set_mode.restype = c.c_int
    lib.oracle_set_mode.argtypes = [c.c_void_p, c.c_int]
    lib.oracle_set_lr.restype = c.c_int
    lib.oracle_set_lr.argtypes = [c.c_void_p, c.c_float]
    lib.oracle_set_weight_decay.restype = c.c_int
    lib.oracle_set_weight_decay.argtypes = [c.c_void_p, c.c_float]
    lib.oracle_set_lr_milestones.restype = c.c_int
    lib.oracle_set_lr_milestones.argtypes = [c.c_void_p, c.c_float, c.c_int, ip, c.c_float]
    lib.oracle_compress_randk.restype = None
    lib.oracle_compress_randk.argtypes = [fp, c.c_int64, c.c_int64, up, up, fp, fp]
    lib.oracle_set_random_sets.restype = c.c_int
    lib.oracle_set_random_sets.argtypes = [c.c_void_p, up, up]
    lib.oracle_force_scales.restype = c.c_int
    lib.oracle_force_scales.argtypes = [c.c_void_p, fp, fp]
    lib.oracle_state.restype = fp
    lib.oracle_state.argtypes = [c.c_void_p, c.c_int]
    lib.oracle_step.restype = c.c_int
    lib.oracle_step.argtypes = [c.c_void_p, fp]
    for name, res in (("bits", up), ("scales", fp), ("idx", up), ("val", fp)):
        f = getattr(lib, "oracle_payload_" + name)
        f.restype = res
        f.argtypes = [c.c_void_p, c.c_int]
    _lib = lib
    return lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _offsets(d, offsets):
    off = np.ascontiguousarray([0, d] if offsets is None else offsets, dtype=np.int64)
    return off, off.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def l1_exact(x):
    """Correctly rounded float64 value of sum |x_j| over float32 data."""
    a, p = _f32(x)
    return float(_load().oracle_l1_exact(p, a.size))


def compress_sign(x, offsets=None):
    """Scaled-sign compressor of Appendix A per segment.  Returns (bits, scales, c)."""
    a, p = _f32(x)
    d = a.size
    off, op = _offsets(d, offsets)
    q = off.size - 1
    bits = np.zeros((d + 31) // 32, dtype=np.uint32)
    scales = np.zeros(q, dtype=np.float32)
    c = np.zeros(d, dtype=np.float32)
    _load().oracle_compress_sign(p, d, q, op,
                                 bits.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)),
                                 scales.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                 c.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
    return bits, scales, c


def compress_topk(x, k):
    """Top-k compressor of Appendix A (ties: lower index).  Returns (idx, val, c)."""
    a, p = _f32(x)
    d = a.size
    idx = np.zeros(k, dtype=np.uint32)
    val = np.zeros(k, dtype=np.float32)
    c = np.zeros(d, dtype=np.float32)
    _load().oracle_compress_topk(p, d, k,
                                 idx.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)),
                                 val.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                 c.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
    return idx, val, c


def compress_randk(x, S):
    """Rand-k compressor of Appendix A on the given coordinate set S.  Returns (idx, val, c)."""
    a, p = _f32(x)
    d = a.size
    S = np.ascontiguousarray(S, dtype=np.uint32)
    k = S.size
    idx = np.zeros(k, dtype=np.uint32)
    val = np.zeros(k, dtype=np.float32)
    c = np.zeros(d, dtype=np.float32)
    up = ctypes.POINTER(ctypes.c_uint32)
    _load().oracle_compress_randk(p, d, k, S.ctypes.data_as(up), idx.ctypes.data_as(up),
                                  val.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                  c.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
    return idx, val, c


class Oracle:
    """Algorithm 1 for n workers on the CPU.  State arrays are numpy views of the C memory."""

    def __init__(self, d, n, compressor=SIGN, k=0, beta1=0.9, beta2=0.999, lr=1e-3,
                 eps=1e-8, offsets=None, mode=MARKOV, x0=None):
        self._lib = _load()
        self.d, self.n, self.compressor, self.k = int(d), int(n), int(compressor), int(k)
        self._h = self._lib.oracle_create(self.d, self.n, self.compressor, self.k,
                                          beta1, beta2, lr, eps)
        if not self._h:
            raise ValueError("oracle_create rejected its arguments")
        self.q = 1
        if offsets is not None:
            off, op = _offsets(self.d, offsets)
            if self._lib.oracle_set_segments(self._h, off.size - 1, op) != 0:
                raise ValueError("bad segment offsets")
            self.q = off.size - 1
        if mode != MARKOV and self._lib.oracle_set_mode(self._h, mode) != 0:
            raise ValueError("bad mode")
        if x0 is not None:
            self.state("x")[:] = np.asarray(x0, dtype=np.float32)

    def close(self):
        if self._h:
            self._lib.oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def set_lr(self, lr):
        self._lib.oracle_set_lr(self._h, lr)

    def set_topk_segments(self, offsets, k_per_segment):
        """Top-k on every segment on its own; the payload has sum(k_per_segment) entries."""
        off, op = _offsets(self.d, offsets)
        ks = np.ascontiguousarray(k_per_segment, dtype=np.int64)
        assert ks.size == off.size - 1
        ip = ctypes.POINTER(ctypes.c_int64)
        if self._lib.oracle_set_topk_segments(self._h, off.size - 1, op, ks.ctypes.data_as(ip)) != 0:
            raise ValueError("bad top-k segments")
        self.q = off.size - 1
        self.k = int(ks.sum())

    def set_weight_decay(self, weight_decay):
        if self._lib.oracle_set_weight_decay(self._h, weight_decay) != 0:
            raise ValueError("bad weight decay")

    def set_lr_milestones(self, base_lr, after_steps, gamma):
        """alpha_t = base_lr * gamma^(number of entries of after_steps that are <= t - 1)."""
        ms = np.ascontiguousarray(after_steps, dtype=np.int64)
        ip = ctypes.POINTER(ctypes.c_int64)
        if self._lib.oracle_set_lr_milestones(self._h, base_lr, ms.size, ms.ctypes.data_as(ip), gamma) != 0:
            raise ValueError("bad milestones")

    def set_random_sets(self, workers, server):
        """Rand-k: coordinate sets (n x k and k increasing distinct coordinates) of the next step."""
        w = np.ascontiguousarray(workers, dtype=np.uint32)
        s = np.ascontiguousarray(server, dtype=np.uint32)
        assert w.size == self.n * self.k and s.size == self.k
        up = ctypes.POINTER(ctypes.c_uint32)
        if self._lib.oracle_set_random_sets(self._h, w.ctypes.data_as(up), s.ctypes.data_as(up)) != 0:
            raise ValueError("set_random_sets applies to the rand-k compressor")

    def force_scales(self, worker_scales=None, server_scales=None):
        """Sampled checks only: use these scaled-sign scales (n x q, q) instead of computing
        them from the (sampled, hence incomplete) data.  None returns to computed scales."""
        ws = ss = None
        if worker_scales is not None:
            wa, ws = _f32(worker_scales)
            assert wa.size == self.n * self.q
        if server_scales is not None:
            sa, ss = _f32(server_scales)
            assert sa.size == self.q
        if self._lib.oracle_force_scales(self._h, ws, ss) != 0:
            raise ValueError("force_scales applies to the scaled-sign compressor")

    def state(self, name):
        """Writable numpy view of a state vector ('ghat_w' is n x d, the others d)."""
        i = STATE_NAMES.index(name)
        p = self._lib.oracle_state(self._h, i)
        shape = (self.n, self.d) if name == "ghat_w" else (self.d,)
        return np.ctypeslib.as_array(p, shape=shape)

    def step(self, grads):
        g, p = _f32(grads)
        if g.size != self.n * self.d:
            raise ValueError("grads must hold n*d values")
        if self._lib.oracle_step(self._h, p) != 0:
            raise RuntimeError("oracle_step failed")

    def payload(self, who):
        """Last payload of worker `who` (0..n-1) or of the server (who = -1).

        sign: (bits uint32[ceil(d/32)], scales float32[q]); top-k: (idx uint32[k] ascending,
        val float32[k]).  Copies."""
        words = (self.d + 31) // 32
        if self.compressor == SIGN:
            b = np.ctypeslib.as_array(self._lib.oracle_payload_bits(self._h, who), shape=(words,))
            s = np.ctypeslib.as_array(self._lib.oracle_payload_scales(self._h, who), shape=(self.q,))
            return b.copy(), s.copy()
        if self.compressor in (TOPK, RANDK):
            i = np.ctypeslib.as_array(self._lib.oracle_payload_idx(self._h, who), shape=(self.k,))
            v = np.ctypeslib.as_array(self._lib.oracle_payload_val(self._h, who), shape=(self.k,))
            return i.copy(), v.copy()
        raise ValueError("the identity compressor has no payload")
