"""CPU checks of the C boundary: the library builds, loads, exports every entry point the
header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

from paper_2111_00705_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cdadam.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cdadam_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    handle = ctypes.CDLL(path)
    names = declared_functions()
    assert len(names) >= 15
    for name in names:
        assert hasattr(handle, name), name
    assert names == binding.exported_symbols()


def test_bad_arguments_fail_without_a_device():
    lib = binding.lib()
    assert not lib.cdadam_create(0, 4, 0, 0, 0.9, 0.999, 1e-3, 1e-8)
    assert b"d must be" in lib.cdadam_last_error()
    assert not lib.cdadam_create(1 << 32, 4, 0, 0, 0.9, 0.999, 1e-3, 1e-8)
    assert not lib.cdadam_create(10, 0, 0, 0, 0.9, 0.999, 1e-3, 1e-8)
    assert not lib.cdadam_create(10, 70000, 0, 0, 0.9, 0.999, 1e-3, 1e-8)
    assert not lib.cdadam_create(10, 2, 1, 11, 0.9, 0.999, 1e-3, 1e-8)
    assert b"top-k" in lib.cdadam_last_error()
    assert not lib.cdadam_create(10, 2, 9, 0, 0.9, 0.999, 1e-3, 1e-8)
    assert lib.cdadam_step(None, None, None) == binding.ERR_ARG
    assert lib.cdadam_set_lr(None, 0.1) == binding.ERR_ARG
    assert lib.cdadam_params(None) is None
    assert lib.cdadam_step_count(None) == 0
    lib.cdadam_destroy(None)
    assert lib.cdadam_compress_topk(None, 10, 1, None, None, None) == binding.ERR_ARG
    assert lib.cdadam_compress_sign(None, 10, 1, None, None, None, None) == binding.ERR_ARG
