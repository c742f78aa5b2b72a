"""ctypes binding of libcdadam.so: the same entry points as include/cdadam.h.

Argument marshalling only.  PyTorch supplies device memory and streams; every step of the
method runs in the library's CUDA kernels.  There is no CPU fallback: if the shared library
is missing, loading raises.
"""
import ctypes
import os

import torch

SIGN, TOPK, IDENTITY, RANDK = 0, 1, 2, 3
MARKOV, EF, NAIVE = 0, 1, 2
SERVER = -1
STATE_NAMES = ("ghat_w", "ghat_s", "gtil", "m", "v", "vhat", "x")
OK, ERR_ARG, ERR_ALLOC, ERR_CUDA, ERR_STATE, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcdadam.so")
_lib = None

_c = ctypes
_SIGNATURES = {
    "cdadam_create": (_c.c_void_p, [_c.c_int64, _c.c_int, _c.c_int, _c.c_int64,
                                    _c.c_float, _c.c_float, _c.c_float, _c.c_float]),
    "cdadam_destroy": (None, [_c.c_void_p]),
    "cdadam_step": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "cdadam_step_bf16": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "cdadam_step_host": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "cdadam_create_shard": (_c.c_void_p, [_c.c_int64, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int64,
                                          _c.c_float, _c.c_float, _c.c_float, _c.c_float]),
    "cdadam_step_workers": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "cdadam_step_server": (_c.c_int, [_c.c_void_p, _c.c_void_p]),
    "cdadam_step_update": (_c.c_int, [_c.c_void_p, _c.c_void_p]),
    "cdadam_exchange_buffers": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_void_p), _c.POINTER(_c.c_void_p),
                                           _c.POINTER(_c.c_void_p), _c.POINTER(_c.c_void_p),
                                           _c.POINTER(_c.c_int64), _c.POINTER(_c.c_int)]),
    "cdadam_create_range": (_c.c_void_p, [_c.c_int64, _c.c_int, _c.c_int64, _c.c_int64, _c.c_int, _c.c_int, _c.c_int,
                                          _c.c_int64, _c.c_float, _c.c_float, _c.c_float, _c.c_float]),
    "cdadam_range_workers": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "cdadam_range_server": (_c.c_int, [_c.c_void_p, _c.c_void_p]),
    "cdadam_range_update": (_c.c_int, [_c.c_void_p, _c.c_void_p]),
    "cdadam_range_buffers": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_void_p), _c.POINTER(_c.c_void_p),
                                        _c.POINTER(_c.c_int64), _c.POINTER(_c.c_int64), _c.POINTER(_c.c_int),
                                        _c.POINTER(_c.c_void_p)]),
    "cdadam_range_topk": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_void_p, _c.c_void_p]),
    "cdadam_range_topk_buffer": (_c.c_int, [_c.c_void_p, _c.c_int, _c.POINTER(_c.c_void_p), _c.POINTER(_c.c_int64)]),
    "cdadam_params": (_c.c_void_p, [_c.c_void_p]),
    "cdadam_set_params": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "cdadam_set_segments": (_c.c_int, [_c.c_void_p, _c.c_int, _c.POINTER(_c.c_int64)]),
    "cdadam_set_random_sets": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_void_p]),
    "cdadam_set_mode": (_c.c_int, [_c.c_void_p, _c.c_int]),
    "cdadam_set_tile": (_c.c_int, [_c.c_void_p, _c.c_int]),
    "cdadam_set_topk_segments": (_c.c_int, [_c.c_void_p, _c.c_int, _c.POINTER(_c.c_int64), _c.POINTER(_c.c_int64)]),
    "cdadam_set_lr": (_c.c_int, [_c.c_void_p, _c.c_float]),
    "cdadam_set_lr_milestones": (_c.c_int, [_c.c_void_p, _c.c_float, _c.c_int, _c.POINTER(_c.c_int64), _c.c_float]),
    "cdadam_set_weight_decay": (_c.c_int, [_c.c_void_p, _c.c_float]),
    "cdadam_get_state": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_void_p, _c.c_void_p]),
    "cdadam_set_state": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_void_p, _c.c_void_p]),
    "cdadam_last_payload": (_c.c_int, [_c.c_void_p, _c.c_int, _c.POINTER(_c.c_void_p),
                                       _c.POINTER(_c.c_void_p), _c.POINTER(_c.c_int64)]),
    "cdadam_step_count": (_c.c_int64, [_c.c_void_p]),
    "cdadam_set_step_count": (_c.c_int, [_c.c_void_p, _c.c_int64]),
    "cdadam_device_status": (_c.c_int, [_c.c_void_p, _c.c_void_p]),
    "cdadam_launches_per_step": (_c.c_int, [_c.c_void_p]),
    "cdadam_set_wait_limit": (_c.c_int, [_c.c_void_p, _c.c_int]),
    "cdadam_compress_sign": (_c.c_int, [_c.c_void_p, _c.c_int64, _c.c_int,
                                        _c.POINTER(_c.c_int64), _c.c_void_p, _c.c_void_p,
                                        _c.c_void_p]),
    "cdadam_compress_topk": (_c.c_int, [_c.c_void_p, _c.c_int64, _c.c_int64, _c.c_void_p,
                                        _c.c_void_p, _c.c_void_p]),
    "cdadam_compress_sign_static": (_c.c_int, [_c.c_void_p, _c.c_int64, _c.c_void_p, _c.c_void_p,
                                               _c.c_void_p]),
    "cdadam_profile_enable": (_c.c_int, [_c.c_void_p, _c.c_int]),
    "cdadam_profile_read": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_double), _c.POINTER(_c.c_int64)]),
    "cdadam_profile_name": (_c.c_char_p, [_c.c_void_p, _c.c_int]),
    "cdadam_last_error": (_c.c_char_p, []),
}


def exported_symbols():
    """Names of the C entry points this binding expects (those include/cdadam.h declares)."""
    return sorted(_SIGNATURES)


def lib():
    """Load libcdadam.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("libcdadam.so is missing: run `python -m paper_2111_00705_b200.build`"
                               " (there is no fallback path)")
        handle = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            f = getattr(handle, name)
            f.restype, f.argtypes = res, args
        _lib = handle
    return _lib


class CdadamError(RuntimeError):
    def __init__(self, code, message):
        super().__init__("cdadam error %d: %s" % (code, message))
        self.code = code


def last_error():
    return lib().cdadam_last_error().decode()


def _check(code):
    if code != OK:
        raise CdadamError(code, last_error())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dev_f32(t, count, what):
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.numel() == count):
        raise ValueError("%s must be a contiguous CUDA float32 tensor of %d elements" % (what, count))
    return ctypes.c_void_p(t.data_ptr())


class _DevView:
    """Zero-copy view of library-owned device memory for torch.as_tensor."""

    def __init__(self, ptr, count, typestr):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr,
                                         "data": (ptr, False), "version": 2}


def _view(ptr, count, dtype, device):
    typestr = {torch.float32: "<f4", torch.int32: "<i4", torch.float64: "<f8"}[dtype]
    if count == 0:
        return torch.empty(0, dtype=dtype, device=device)
    return torch.as_tensor(_DevView(ptr, count, typestr), device=device)


class CDAdam:
    """One context of the library: n simulated workers and the server on one GPU."""

    def __init__(self, d, n, compressor=SIGN, k=0, beta1=0.9, beta2=0.999, lr=1e-3, eps=1e-8,
                 offsets=None, x0=None, device=None, mode=MARKOV):
        self._h = None
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None \
            else torch.device(device)
        self.d, self.n, self.compressor, self.k = int(d), int(n), int(compressor), int(k)
        self.q = 1
        self.mode = int(mode)
        self.first_worker, self.n_local = 0, self.n
        with torch.cuda.device(self.device):
            self._h = self._create(beta1, beta2, lr, eps)
        if not self._h:
            raise CdadamError(ERR_ARG, last_error())
        if mode != MARKOV:
            _check(lib().cdadam_set_mode(self._h, int(mode)))
        if offsets is not None:
            self.set_segments(offsets)
        if x0 is not None:
            self.set_params(x0)

    def _create(self, beta1, beta2, lr, eps):
        return lib().cdadam_create(self.d, self.n, self.compressor, self.k, beta1, beta2, lr, eps)

    def close(self):
        if self._h:
            lib().cdadam_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the three calls of the hot path ------------------------------------------------
    def step(self, grads, stream=None):
        """One iteration of Algorithm 1 on the n x d device gradients."""
        _check(lib().cdadam_step(self._h, _dev_f32(grads, self.n * self.d, "grads"), _stream(stream)))

    def step_bf16(self, grads, stream=None):
        """One iteration on n x d device gradients in bfloat16."""
        if not (grads.is_cuda and grads.dtype == torch.bfloat16 and grads.is_contiguous()
                and grads.numel() == self.n * self.d):
            raise ValueError("grads must be a contiguous CUDA bfloat16 tensor of n*d elements")
        _check(lib().cdadam_step_bf16(self._h, ctypes.c_void_p(grads.data_ptr()), _stream(stream)))

    def step_host(self, grads_host, x_out_host=None, stream=None):
        """The same with host gradients (pinned or pageable) and x copied back to the host."""
        if grads_host.is_cuda or grads_host.dtype != torch.float32 or not grads_host.is_contiguous() \
                or grads_host.numel() != self.n * self.d:
            raise ValueError("grads_host must be a contiguous CPU float32 tensor of n*d elements")
        xo = None
        if x_out_host is not None:
            if x_out_host.is_cuda or x_out_host.dtype != torch.float32 or x_out_host.numel() != self.d \
                    or not x_out_host.is_contiguous():
                raise ValueError("x_out_host must be a contiguous CPU float32 tensor of d elements")
            xo = ctypes.c_void_p(x_out_host.data_ptr())
        _check(lib().cdadam_step_host(self._h, ctypes.c_void_p(grads_host.data_ptr()), xo, _stream(stream)))

    def params(self):
        """The model x as a torch view of the library's memory (no copy)."""
        return _view(lib().cdadam_params(self._h), self.d, torch.float32, self.device)

    # -- helpers ------------------------------------------------------------------------
    def set_params(self, x0, stream=None):
        _check(lib().cdadam_set_params(self._h, _dev_f32(x0, self.d, "x0"), _stream(stream)))

    def set_segments(self, offsets):
        off = (ctypes.c_int64 * len(offsets))(*[int(v) for v in offsets])
        _check(lib().cdadam_set_segments(self._h, len(offsets) - 1, off))
        self.q = len(offsets) - 1

    def set_random_sets(self, workers, server, stream=None):
        """Rand-k: CUDA int32/uint32 tensors with n*k and k increasing coordinates."""
        for t, cnt in ((workers, self.n * self.k), (server, self.k)):
            if not (t.is_cuda and t.is_contiguous() and t.element_size() == 4 and t.numel() == cnt):
                raise ValueError("sets must be contiguous CUDA 32-bit integer tensors of n*k and k elements")
        _check(lib().cdadam_set_random_sets(self._h, ctypes.c_void_p(workers.data_ptr()),
                                            ctypes.c_void_p(server.data_ptr()), _stream(stream)))

    def set_tile(self, tile):
        _check(lib().cdadam_set_tile(self._h, int(tile)))

    def set_topk_segments(self, offsets, k_per_segment):
        """Top-k on every segment on its own; the payload has sum(k_per_segment) entries."""
        off = [int(a) for a in offsets]
        ks = [int(a) for a in k_per_segment]
        if len(ks) != len(off) - 1:
            raise ValueError("one k per segment")
        _check(lib().cdadam_set_topk_segments(self._h, len(ks), (ctypes.c_int64 * len(off))(*off),
                                              (ctypes.c_int64 * len(ks))(*ks)))
        self.k = sum(ks)

    def set_lr(self, lr):
        _check(lib().cdadam_set_lr(self._h, lr))

    def set_lr_milestones(self, base_lr, after_steps, gamma):
        """alpha_t = base_lr * gamma^(number of entries of after_steps that are <= t - 1)."""
        ms = (ctypes.c_int64 * len(after_steps))(*[int(a) for a in after_steps])
        _check(lib().cdadam_set_lr_milestones(self._h, base_lr, len(after_steps), ms, gamma))

    def set_weight_decay(self, weight_decay):
        _check(lib().cdadam_set_weight_decay(self._h, weight_decay))

    def get_state(self, name, stream=None):
        count = self.n_local * self.d if name == "ghat_w" else self.d
        out = torch.empty(count, dtype=torch.float32, device=self.device)
        _check(lib().cdadam_get_state(self._h, STATE_NAMES.index(name), ctypes.c_void_p(out.data_ptr()),
                                      _stream(stream)))
        return out.view(self.n_local, self.d) if name == "ghat_w" else out

    def set_state(self, name, value, stream=None):
        count = self.n_local * self.d if name == "ghat_w" else self.d
        _check(lib().cdadam_set_state(self._h, STATE_NAMES.index(name), _dev_f32(value, count, name),
                                      _stream(stream)))

    def last_payload(self, who):
        """(bits int32[ceil(d/32)], scales float32[q]) or (idx int32[k], val float32[k]) as
        views of library memory, valid until the next step.  Integer words are returned as
        int32 tensors holding the uint32 bit patterns."""
        a, b, cnt = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_int64()
        _check(lib().cdadam_last_payload(self._h, who, ctypes.byref(a), ctypes.byref(b), ctypes.byref(cnt)))
        if self.compressor == SIGN:
            return (_view(a.value, (self.d + 31) // 32, torch.int32, self.device),
                    _view(b.value, self.q, torch.float32, self.device))
        return (_view(a.value, self.k, torch.int32, self.device),
                _view(b.value, self.k, torch.float32, self.device))

    def profile_enable(self, on=True):
        _check(lib().cdadam_profile_enable(self._h, 1 if on else 0))

    def profile_read(self):
        """({stage name: total ms}, steps) accumulated since the last read."""
        ms = (ctypes.c_double * 8)()
        steps = ctypes.c_int64()
        _check(lib().cdadam_profile_read(self._h, ms, ctypes.byref(steps)))
        out = {}
        for s in range(8):
            name = lib().cdadam_profile_name(self._h, s).decode()
            if name:
                out[name] = ms[s]
        return out, steps.value

    def device_status(self, stream=None):
        """Wait for the stream; raise if a kernel reported that a bounded wait ran out."""
        _check(lib().cdadam_device_status(self._h, _stream(stream)))

    def set_wait_limit(self, polls):
        """Polls before a kernel's wait on an asynchronous copy gives up (< 0: the default)."""
        _check(lib().cdadam_set_wait_limit(self._h, int(polls)))

    def step_count(self):
        return lib().cdadam_step_count(self._h)

    def set_step_count(self, t):
        """The iteration counter of a run resumed from saved state (see state_dict)."""
        _check(lib().cdadam_set_step_count(self._h, int(t)))

    def state_dict(self, stream=None):
        """Everything a resumed run needs: copies of the seven state vectors and the counter."""
        out = {name: self.get_state(name, stream) for name in STATE_NAMES}
        out["step_count"] = self.step_count()
        return out

    def load_state_dict(self, state, stream=None):
        """Load what state_dict returned into a context created with the same configuration."""
        for name in STATE_NAMES:
            self.set_state(name, state[name].reshape(-1), stream)
        self.set_step_count(state["step_count"])

    def launches_per_step(self):
        return lib().cdadam_launches_per_step(self._h)


class CDAdamShard(CDAdam):
    """A context for the workers [first_worker, first_worker + n_local) of n (scaled sign or
    top-k): one process of a distributed deployment.  An iteration runs in its stages with
    the messages moved by the caller in between (see ``distributed.py``)."""

    def __init__(self, d, n, first_worker, n_local, beta1=0.9, beta2=0.999, lr=1e-3, eps=1e-8,
                 offsets=None, x0=None, device=None, mode=MARKOV, compressor=SIGN, k=0):
        self._shard = (int(first_worker), int(n_local))
        super().__init__(d, n, compressor, k, beta1, beta2, lr, eps, offsets, x0, device, mode)
        self.first_worker, self.n_local = self._shard

    def _create(self, beta1, beta2, lr, eps):
        return lib().cdadam_create_shard(self.d, self.n, self._shard[0], self._shard[1], self.compressor, self.k,
                                         beta1, beta2, lr, eps)

    def step_workers(self, grads, stream=None):
        """Worker stage on the n_local x d device gradients of this context's workers."""
        g = None if self.n_local == 0 else _dev_f32(grads, self.n_local * self.d, "grads")
        _check(lib().cdadam_step_workers(self._h, g, _stream(stream)))

    def step_server(self, stream=None):
        """Server stage from the n worker messages in the exchange buffers."""
        _check(lib().cdadam_step_server(self._h, _stream(stream)))

    def step_update(self, stream=None):
        """gtil += c and the AMSGrad update from the server message in the exchange buffers."""
        _check(lib().cdadam_step_update(self._h, _stream(stream)))

    def exchange_buffers(self):
        """Torch views (no copy) of the message buffers: worker_bits int32[n, words],
        worker_scales float32[n, q], server_bits int32[words], server_scales float32[q].
        worker_scales alternates between two arrays: ask again after every step_workers.
        With top-k the same keys hold the coordinates (int32[n, k], int32[k]) and the values
        (float32[n, k], float32[k]) of the messages."""
        wb, ws, sb, ss = (ctypes.c_void_p() for _ in range(4))
        words, q = ctypes.c_int64(), ctypes.c_int()
        _check(lib().cdadam_exchange_buffers(self._h, ctypes.byref(wb), ctypes.byref(ws), ctypes.byref(sb),
                                             ctypes.byref(ss), ctypes.byref(words), ctypes.byref(q)))
        w, q = words.value, q.value
        return {"worker_bits": _view(wb.value, self.n * w, torch.int32, self.device).view(self.n, w),
                "worker_scales": _view(ws.value, self.n * q, torch.float32, self.device).view(self.n, q),
                "server_bits": _view(sb.value, w, torch.int32, self.device),
                "server_scales": _view(ss.value, q, torch.float32, self.device)}


class CDAdamRange(CDAdam):
    """A context for the coordinates [lo, hi) of a d-dimensional problem with n workers
    (scaled sign): one process of a coordinate-sharded deployment.  Every vector of the
    context has hi - lo coordinates; `offsets` are the segments of the WHOLE problem.  An
    iteration runs in three stages, the l1 sums of the ranges moved by the caller in between
    (see ``distributed.py``)."""

    def __init__(self, d, n, lo, hi, rank, ranks, beta1=0.9, beta2=0.999, lr=1e-3, eps=1e-8,
                 offsets=None, x0=None, device=None, mode=MARKOV, compressor=SIGN, k=0):
        self._range = (int(d), int(lo), int(hi), int(rank), int(ranks))
        self.dim, self.lo, self.hi, self.rank, self.ranks = self._range
        self.q_all = 1 if offsets is None else len(offsets) - 1
        self.k_all = int(k)                 # top-k: entries kept in the whole vector
        super().__init__(hi - lo, n, compressor, min(int(k), hi - lo), beta1, beta2, lr, eps, offsets, x0, device, mode)

    def _create(self, beta1, beta2, lr, eps):
        d, lo, hi, rank, ranks = self._range
        return lib().cdadam_create_range(d, self.n, lo, hi, rank, ranks, self.compressor, self.k_all,
                                         beta1, beta2, lr, eps)

    TOPK_STAGES = 10

    def range_topk(self, stage, grads=None, stream=None):
        """Stage 0..9 of a top-k iteration on the range (0..4 take the n x (hi - lo) gradients)."""
        g = None if grads is None else _dev_f32(grads, self.n * self.d, "grads")
        _check(lib().cdadam_range_topk(self._h, int(stage), g, _stream(stream)))

    def range_topk_buffer(self, stage):
        """The exchange buffer to gather after `stage` as an int32[ranks, words] view, or None."""
        buf, words = ctypes.c_void_p(), ctypes.c_int64()
        _check(lib().cdadam_range_topk_buffer(self._h, int(stage), ctypes.byref(buf), ctypes.byref(words)))
        if not buf.value:
            return None
        return _view(buf.value, self.ranks * words.value, torch.int32, self.device).view(self.ranks, words.value)

    def set_segments(self, offsets):
        super().set_segments(offsets)
        self.q_all = len(offsets) - 1
        self.q = self.range_buffers()["q_local"]

    def range_workers(self, grads, stream=None):
        """Worker pass on the n x (hi - lo) device gradients; writes this range's l1 parts."""
        _check(lib().cdadam_range_workers(self._h, _dev_f32(grads, self.n * self.d, "grads"), _stream(stream)))

    def range_server(self, stream=None):
        """Workers' scales from the gathered parts, server pass on the range, its l1 parts."""
        _check(lib().cdadam_range_server(self._h, _stream(stream)))

    def range_update(self, stream=None):
        """Server's scales from the gathered parts; gtil += c and AMSGrad on the range."""
        _check(lib().cdadam_range_update(self._h, _stream(stream)))

    def range_buffers(self):
        """Torch views (no copy) of the exchange buffers: worker_sums float64[ranks, n, q, 2],
        server_sums float64[ranks, q, 2] (value and rounding error of each range's part of the
        l1 sums; slot [rank] is this context's), q_local and segment_of_local int32[q_local]."""
        ws, ss, seg = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p()
        wd, sd, ql = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int()
        _check(lib().cdadam_range_buffers(self._h, ctypes.byref(ws), ctypes.byref(ss), ctypes.byref(wd),
                                          ctypes.byref(sd), ctypes.byref(ql), ctypes.byref(seg)))
        q = sd.value // 2
        return {"worker_sums": _view(ws.value, self.ranks * wd.value, torch.float64, self.device).view(self.ranks, self.n, q, 2),
                "server_sums": _view(ss.value, self.ranks * sd.value, torch.float64, self.device).view(self.ranks, q, 2),
                "q_local": ql.value,
                "segment_of_local": _view(seg.value, ql.value, torch.int32, self.device)}


def compress_sign(x, offsets=None, stream=None):
    """Stand-alone scaled-sign compressor on a CUDA vector: (bits int32, scales float32)."""
    d = x.numel()
    q = 1 if offsets is None else len(offsets) - 1
    off = None if offsets is None else (ctypes.c_int64 * len(offsets))(*[int(v) for v in offsets])
    bits = torch.empty((d + 31) // 32, dtype=torch.int32, device=x.device)
    scales = torch.empty(q, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        _check(lib().cdadam_compress_sign(_dev_f32(x, d, "x"), d, q, off, ctypes.c_void_p(bits.data_ptr()),
                                          ctypes.c_void_p(scales.data_ptr()), _stream(stream)))
    return bits, scales


def compress_topk(x, k, stream=None):
    """Stand-alone top-k compressor on a CUDA vector: (idx int32[k] increasing, val float32[k])."""
    d = x.numel()
    idx = torch.empty(k, dtype=torch.int32, device=x.device)
    val = torch.empty(k, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        _check(lib().cdadam_compress_topk(_dev_f32(x, d, "x"), d, k, ctypes.c_void_p(idx.data_ptr()),
                                          ctypes.c_void_p(val.data_ptr()), _stream(stream)))
    return idx, val


STATIC_MAX_D = 1 << 28


def compress_sign_static(x, bits=None, scale=None, stream=None):
    """Flat scaled-sign compressor through the entry point that allocates nothing inside the
    library (for callers that cannot allocate device memory at call time).  Pass preallocated
    `bits` (int32[ceil(d/32)]) and `scale` (float32[1]) to keep the whole call free of
    allocations; they are created here only when omitted.  Returns (bits, scale)."""
    d = x.numel()
    if bits is None:
        bits = torch.empty((d + 31) // 32, dtype=torch.int32, device=x.device)
    if scale is None:
        scale = torch.empty(1, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        _check(lib().cdadam_compress_sign_static(_dev_f32(x, d, "x"), d, ctypes.c_void_p(bits.data_ptr()),
                                                 ctypes.c_void_p(scale.data_ptr()), _stream(stream)))
    return bits, scale
