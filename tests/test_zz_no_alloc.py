"""The scaled-sign compressor entry point that allocates nothing.

Some callers cannot allocate device memory at the moment they compress a vector: they run
where cudaMalloc/cudaFree (which may synchronise the whole device) are not acceptable, or
their GPU memory is entirely owned by a framework's pool.  cdadam_compress_sign_static
keeps its scratch (the per-tile partial sums of the l1 norm) in a fixed array inside the
library, so it calls no allocator.  This test checks it, through the C interface, against
the allocating entry point cdadam_compress_sign and against the CPU oracle's scaled-sign
compressor: sign words and scale must be identical (the bar of the other compressor tests),
on two calls in a row that share the array; and the free device memory must not move while
it is called.

This file sorts last on purpose, so a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2111_00705_b200 import binding as cd

pytestmark = pytest.mark.gpu


def _same(x):
    bits_a, scale_a = cd.compress_sign(x)
    bits = torch.full(((x.numel() + 31) // 32,), -1, dtype=torch.int32, device=x.device)
    scale = torch.full((1,), float("nan"), device=x.device)
    cd.compress_sign_static(x, bits, scale)       # caller-provided outputs: no allocation at all
    torch.cuda.synchronize()
    assert torch.equal(bits, bits_a)
    assert scale.cpu().numpy().view(np.uint32)[0] == scale_a.cpu().numpy().view(np.uint32)[0]
    # and against the oracle's compressor (Appendix A, scaled sign), bit for bit
    obits, oscales, _ = orc.compress_sign(x.cpu().numpy())
    assert np.array_equal(bits.cpu().numpy().view(np.uint32), obits)
    assert scale.cpu().numpy().view(np.uint32)[0] == oscales.view(np.uint32)[0]


def test_static_scratch_matches_allocating_entry_point_twice_in_a_row():
    g = torch.Generator(device="cuda").manual_seed(5)
    # first call: several tiles and a ragged tail; the array now holds this call's sums
    x1 = torch.randn(3 * 16384 * 7 + 12345, generator=g, device="cuda") * 3.0
    _same(x1)
    # second call, shorter and with other magnitudes: stale sums beyond its tiles stay unread
    x2 = torch.randn(16384 + 3, generator=g, device="cuda") * 1e-4
    _same(x2)
    # third: unaligned start (scalar path) and a single element
    buf = torch.randn(40001, generator=g, device="cuda")
    _same(buf[1:])
    _same(buf[:1].clone())


def test_static_scratch_leaves_free_device_memory_alone():
    """What the entry point is for: once its first call on the device has looked up the
    array's address, calls with caller-provided outputs change nothing in the device's free
    memory (cudaMemGetInfo before and after)."""
    g = torch.Generator(device="cuda").manual_seed(6)
    x = torch.randn(5 * 16384 + 77, generator=g, device="cuda")
    bits = torch.empty((x.numel() + 31) // 32, dtype=torch.int32, device="cuda")
    scale = torch.empty(1, device="cuda")
    cd.compress_sign_static(x, bits, scale)            # the first call may do the one-time set-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(8):
        cd.compress_sign_static(x, bits, scale)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before


def test_static_scratch_rejects_sizes_beyond_its_array():
    x = torch.zeros(8, device="cuda")
    lib = cd.lib()
    import ctypes
    bits = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = torch.zeros(1, device="cuda")
    rc = lib.cdadam_compress_sign_static(ctypes.c_void_p(x.data_ptr()), cd.STATIC_MAX_D + 1,
                                         ctypes.c_void_p(bits.data_ptr()),
                                         ctypes.c_void_p(scale.data_ptr()), None)
    assert rc == cd.ERR_ARG and "scratch array" in cd.last_error()
    rc = lib.cdadam_compress_sign_static(ctypes.c_void_p(x.data_ptr()), 0, ctypes.c_void_p(bits.data_ptr()),
                                         ctypes.c_void_p(scale.data_ptr()), None)
    assert rc == cd.ERR_ARG
    torch.cuda.synchronize()
