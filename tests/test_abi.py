"""The C ABI: the library loads without a GPU and exports every function include/compams.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2205_05632_b200 import build, load_library
    build.build()
    return load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "compams.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(compams_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_core_calls():
    names = declared_functions()
    for core in ("compams_create", "compams_step", "compams_destroy"):
        assert core in names


def test_library_exports_every_declared_symbol(lib):
    missing = [f for f in declared_functions() if not hasattr(lib, f)]
    assert not missing, missing


def test_static_strings_need_no_gpu(lib):
    assert lib.compams_error_string(0) == b"ok"
    assert lib.compams_error_string(-1) == b"invalid argument"
    assert lib.compams_kernel_name(1) == b"bs_sweep"
    assert lib.compams_kernel_name(999) == b"unknown"


def test_invalid_arguments_are_rejected_before_any_cuda_call(lib):
    h = ctypes.c_void_p()
    offs = (ctypes.c_int64 * 2)(0, 10)
    bad = (ctypes.c_int64 * 3)(0, 7, 7)
    create = lib.compams_create
    assert create(ctypes.byref(h), 0, 10, offs, 1, 0, 0.5, 1e-3, 0.9, 0.999, 1e-8) == -1   # n < 1
    assert create(ctypes.byref(h), 2, 10, offs, 1, 5, 0.5, 1e-3, 0.9, 0.999, 1e-8) == -1   # unknown compressor
    assert create(ctypes.byref(h), 2, 10, offs, 1, 0, 1.5, 1e-3, 0.9, 0.999, 1e-8) == -1   # k_ratio > 1
    assert create(ctypes.byref(h), 2, 7, bad, 2, 1, 1.0, 1e-3, 0.9, 0.999, 1e-8) == -1     # empty block
    assert create(ctypes.byref(h), 2, 11, offs, 1, 1, 1.0, 1e-3, 0.9, 0.999, 1e-8) == -1   # last offset != d
    assert create(None, 2, 10, offs, 1, 1, 1.0, 1e-3, 0.9, 0.999, 1e-8) == -1
    # d beyond what the 32-bit tile coordinates can address (they overshoot a block's end by up to two tiles)
    big = (1 << 31) - 4 * 8192 + 1
    offs_big = (ctypes.c_int64 * 2)(0, big)
    assert create(ctypes.byref(h), 1, big, offs_big, 1, 1, 1.0, 1e-3, 0.9, 0.999, 1e-8) == -1
    assert not h.value
    assert lib.compams_destroy(None) == 0
    assert lib.compams_step(None, None, None) == -1


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    import paper_2205_05632_b200.binding as B
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_HERE", str(tmp_path))
    with pytest.raises(B.CompAMSError):
        B.load_library()
