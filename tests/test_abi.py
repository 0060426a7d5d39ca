"""The C-ABI library loads without a GPU and exports every symbol the header declares."""

import ctypes
import os
import re

import pytest

from paper_2506_03700_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "adadecode.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ada_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    build.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_host_side_argument_checks_need_no_gpu():
    lib = binding.load()
    assert lib.ada_strerror(0) == b"ok" and b"CUDA" in lib.ada_strerror(-4)
    h = ctypes.c_void_p()
    bad = binding.Config(4, 250, 4, 4, 64, 688, 2048, 0, 1, 10000.0, 1e-5)       # d_model not a multiple of 8
    assert lib.ada_model_create(ctypes.byref(bad), ctypes.byref(h)) == -6
    bad = binding.Config(4, 256, 4, 3, 64, 688, 2048, 0, 1, 10000.0, 1e-5)       # q heads not a multiple of kv heads
    assert lib.ada_model_create(ctypes.byref(bad), ctypes.byref(h)) == -1
    ok = binding.Config(4, 256, 4, 4, 64, 688, 2048, 0, 1, 10000.0, 1e-5)
    assert lib.ada_model_create(ctypes.byref(ok), ctypes.byref(h)) == 0
    assert lib.ada_model_set_tensor(h, b"layers.9.wo", 4096, 256 * 256 * 4) == -1   # no such layer
    assert lib.ada_model_set_tensor(h, b"layers.0.wo", 4096, 12) == -1             # wrong size
    assert lib.ada_model_set_tensor(h, b"lm_head", 4096, 2048 * 256 * 4) == -1      # tied model has no lm_head
    assert lib.ada_model_set_exit_head(h, 4, None, 1.0) == -1                      # layer L carries no head
    assert lib.ada_model_finalize(h) == -2                                         # tensors missing
    assert lib.ada_session_scratch_bytes(h, 1, 256, 5) > 0
    assert lib.ada_kv_page_bytes(h, 64) == 4 * 2 * 4 * 64 * 64 * 4
    lib.ada_model_destroy(h)
