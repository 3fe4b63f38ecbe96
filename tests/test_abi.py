"""The C-ABI library loads without a GPU and exports every symbol the header declares; the
host-side argument checks answer before any CUDA call."""
import ctypes
import os
import re

import pytest

from paper_2306_00978_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "awq_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(awq_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_sizes_and_layout_version(lib):
    assert lib.awq_layout_version() == 3
    assert lib.awq_qweight_bytes(4096, 4096) == 4096 * 4096 // 2
    assert lib.awq_scales_bytes(4096, 4096, 128) == 32 * 4096 * 2
    assert lib.awq_zeros_bytes(4096, 11008, 64) == 172 * 4096 // 2
    assert lib.awq_qweight_bytes(100, 4096) == 0
    assert lib.awq_scales_bytes(4096, 4096, 32) == 0
    assert lib.awq_workspace_bytes(1, 4096, 4096, 128) > 4096
    # optional for M <= 128: split-K partial sums of the one-SM tensor-core kernel (16 splits at most)
    assert lib.awq_workspace_bytes(64, 4096, 4096, 128) == 4096 + 32 * 16 * 128 * 64 * 4
    assert lib.awq_workspace_bytes(12, 4096, 4096, 128) == 4096 + 32 * 16 * 128 * 32 * 4
    big = lib.awq_workspace_bytes(2048, 4096, 4096, 128)            # optional: stream-K partial tiles
    assert big > 4096 and (big - 4096) % (256 * 256 * 4) == 0
    assert lib.awq_workspace_bytes(2048, 4096 + 128, 4096, 128) == 0
    assert lib.awq_workspace_bytes(8, 4096, 4096, 128) == 4096 + 256 * 2 * 8 * 128 * 4


def test_argument_errors_need_no_gpu(lib):
    one = ctypes.c_void_p(16)
    assert lib.awq_quantize_pack(one, one, 1.5, 128, one, one, one, 128, 128, None) == 4
    assert lib.awq_quantize_pack(one, one, float("nan"), 128, one, one, one, 128, 128, None) == 4
    assert lib.awq_quantize_pack(one, one, 0.5, 32, one, one, one, 128, 128, None) == 3
    assert lib.awq_quantize_pack(one, one, 0.5, 128, one, one, one, 100, 128, None) == 2
    assert lib.awq_quantize_pack(None, one, 0.5, 128, one, one, one, 128, 128, None) == 1
    assert lib.awq_quantize_pack(one, None, 0.5, 128, one, one, one, 128, 128, None) == 1
    assert lib.awq_quantize_pack(ctypes.c_void_p(8), one, 0.5, 128, one, one, one, 128, 128, None) == 5
    assert lib.awq_linear(one, one, one, one, one, 0, 128, 128, 128, None) == 2
    assert lib.awq_linear(one, one, one, one, None, 1, 128, 128, 128, None) == 1
    assert lib.awq_linear(one, one, one, one, one, 1, 128, 192, 128, None) == 2
    assert lib.awq_linear_path(one, one, one, one, one, 17, 128, 128, 128, 1, None) == 2
    bad = (ctypes.c_float * 2)(1.0, 1.5)
    ok = (ctypes.c_float * 2)(1.0, 0.9)
    assert lib.awq_search_clip(one, one, 0.5, 128, 4, ctypes.cast(bad, ctypes.c_void_p), 2, one, 128, 128, None) == 10
    assert lib.awq_search_clip(one, one, 0.5, 128, 5, ctypes.cast(ok, ctypes.c_void_p), 2, one, 128, 128, None) == 10
    assert lib.awq_search_clip(one, one, 0.5, 128, 4, ctypes.cast(ok, ctypes.c_void_p), 33, one, 128, 128, None) == 10
    assert lib.awq_quantize_pack_ex(one, one, 0.5, 128, 2, 0, None, one, one, one, 128, 128, None) == 10
    assert lib.awq_quantize_pack_ex(one, one, 0.5, 128, 4, 2, None, one, one, one, 128, 128, None) == 10
    assert lib.awq_linear_path(one, one, one, one, one, 1, 128, 128, 128, 7, None) == 10
    assert lib.awq_linear_path(one, one, one, one, one, 17, 128, 128, 128, 3, None) == 2
    assert b"group" in lib.awq_status_string(3)
    assert lib.awq_launch_count() == 0


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libawq_b200.so")
    with pytest.raises(binding.AwqError):
        binding.lib()
