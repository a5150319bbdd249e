"""CPU-side checks of the C ABI: the library loads, exports every symbol the header declares, and every
argument error is reported on the host before anything is launched (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from paper_2412_01034_b200 import _lib, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return _lib.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "qil.h")).read()
    declared = set(re.findall(r"\b(qil_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(_lib.SIGNATURES), "binding and header disagree"
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.qil_version() >= 100
    for code in range(0, 9):
        assert lib.qil_status_string(code) and b"unknown" not in lib.qil_status_string(code)


A = 0x10000  # a 16-byte aligned, never dereferenced address
U = 0x10004  # misaligned


def test_quantize_validation(lib):
    f = lib.qil_quantize_rtn_w4
    assert f(None, 0, 4, 8, 8, 0, A, A, 2, A, None, None) == 1
    assert f(A, 0, 4, 8, 8, 0, A, A, 2, None, None, None) == 1      # asymmetric needs zeros
    assert f(A, 0, 0, 8, 8, 0, A, A, 2, A, None, None) == 2
    assert f(A, 0, 4, 8, 3, 0, A, A, 2, A, None, None) == 2          # group does not divide K
    assert f(A, 7, 4, 8, 8, 0, A, A, 2, A, None, None) == 4          # dtype
    assert f(A, 0, 4, 8, 8, 0, A, A, 0, A, None, None) == 4          # asymmetric scale must be fp16
    assert f(A, 0, 4, 8, 8, 1, A, A, 1, None, None, None) == 4       # bf16 scale unsupported
    assert f(U, 0, 4, 8, 8, 0, A, A, 2, A, None, None) == 3


def test_pack_validation(lib):
    assert lib.qil_pack_w4(None, 4, 8, 0, A, None) == 1
    assert lib.qil_pack_w4(A, 4, 12, 0, A, None) == 2
    assert lib.qil_pack_w4(A, 4, 8, 5, A, None) == 4
    assert lib.qil_pack_w4(A, 8, 128, 1, A, None) == 2               # TILE16 needs N % 16 == 0
    assert lib.qil_pack_w4(A, 16, 64, 1, A, None) == 2               # TILE16 needs K % 128 == 0
    assert lib.qil_pack_w4(A, 4, 8, 0, U, None) == 3
    assert lib.qil_unpack_w4(A, 4, 8, 0, 0, None, None) == 1


def test_linear_w4a16_validation(lib):
    f = lib.qil_linear_w4a16
    assert f(None, A, A, A, A, 1, 16, 128, 128, 0, None, 0, None) == 1
    assert f(A, A, A, A, A, 0, 16, 128, 128, 0, None, 0, None) == 2
    assert f(A, A, A, A, A, 1, 16, 100, 100, 0, None, 0, None) == 2  # K % 8
    assert f(A, A, A, A, A, 1, 16, 128, 48, 0, None, 0, None) == 2   # K % group
    assert f(A, A, A, A, A, 1, 16, 128, 128, 9, None, 0, None) == 4
    assert f(A, A, A, A, A, 1, 24, 128, 128, 1, None, 0, None) == 2  # TILE16 with N % 16 != 0
    assert f(A, U, A, A, A, 1, 16, 128, 128, 0, None, 0, None) == 3
    assert f(A, A, A, A, A, 1, 16, 64, 32, 1, None, 0, None) == 2    # TILE16 needs K % 128
    # a shape that needs a K split must be given a workspace
    need = lib.qil_linear_w4a16_workspace_size(1, 4096, 4096, 128)
    if need:
        assert f(A, A, A, A, A, 1, 4096, 4096, 128, 0, None, 0, None) == 5
        assert f(A, A, A, A, A, 1, 4096, 4096, 128, 0, A, 1024, None) == 5
    assert lib.qil_linear_w4a16_workspace_size(0, 1, 1, 1) == 0


def test_linear_w4a16_swiglu_validation(lib):
    f = lib.qil_linear_w4a16_swiglu
    assert f(None, A, A, A, A, 1, 16, 128, 128, None, 0, None) == 1
    assert f(A, A, A, A, A, 0, 16, 128, 128, None, 0, None) == 2
    assert f(A, A, A, A, A, 1, 15, 128, 128, None, 0, None) == 2    # gate / up rows come in pairs
    assert f(A, A, A, A, A, 1, 16, 128, 48, None, 0, None) == 2     # K % group
    assert f(A, U, A, A, A, 1, 16, 128, 128, None, 0, None) == 3
    # the unfused shapes need the workspace (it holds the linear's bf16 output)
    assert f(A, A, A, A, A, 1, 16, 128, 128, None, 0, None) == 5
    assert lib.qil_linear_w4a16_swiglu_workspace_size(1, 16, 128, 128) >= lib.qil_linear_w4a16_workspace_size(1, 16, 128, 128) + 1 * 16 * 2
    assert lib.qil_linear_w4a16_swiglu_workspace_size(0, 16, 128, 128) == 0


def test_lora_side_validation(lib):
    f = lib.qil_lora_side_add
    assert f(None, A, A, A, 1, 16, 128, 32, 1.0, A, 4096, None) == 1
    assert f(A, A, A, A, 1, 16, 127, 32, 1.0, A, 4096, None) == 2    # K even
    assert f(A, A, A, A, 1, 16, 128, 0, 1.0, A, 4096, None) == 2
    assert f(A, A, A, A, 1, 16, 128, 33, 1.0, A, 4096, None) == 4    # rank above 32
    assert f(A, A, A, A, 4, 16, 128, 32, 1.0, A, 16, None) == 5      # workspace too small
    assert f(A, A, A, A, 4, 16, 128, 32, 1.0, None, 0, None) == 5
    assert lib.qil_lora_side_workspace_size(4) >= 4 * 32 * 4


def test_conv3x3_validation(lib):
    import ctypes as C
    f = lib.qil_conv3x3_w4a4
    one = C.c_float(1.0)
    assert f(None, one, A, A, A, None, None, one, 0, 1, 4, 4, 32, 8, A, 16, None) == 1
    assert f(A, one, A, A, None, None, None, one, 0, 1, 4, 4, 32, 8, A, 16, None) == 1      # no output
    assert f(A, one, A, A, A, None, A, one, 0, 1, 4, 4, 32, 8, A, 16, None) == 1            # two outputs
    assert f(A, one, A, A, A, None, None, one, 0, 1, 4, 4, 48, 8, A, 16, None) == 2         # C % 32
    assert f(A, one, A, A, None, None, A, one, 0, 1, 4, 4, 32, 12, A, 16, None) == 2        # packed output needs Cout % 8
    assert f(A, one, A, A, None, None, A, C.c_float(0.0), 0, 1, 4, 4, 32, 8, A, 16, None) == 4
    assert f(A, one, A, A, A, None, None, one, 0, 1, 4, 4, 32, 8, None, 0, None) == 5


def test_w4a4_and_act_validation(lib):
    assert lib.qil_quantize_act_a4(None, 1, 8, None, A, A, None) == 1
    assert lib.qil_quantize_act_a4(A, 1, 12, None, A, A, None) == 2
    assert lib.qil_quantize_act_a4(A, 1, 8, None, U, A, None) == 3
    assert lib.qil_quantize_act_a4(A, 1, 8, C.byref(C.c_float(0.0)), A, A, None) == 4
    f = lib.qil_linear_w4a4
    assert f(None, A, A, A, A, None, 1, 1, 32, None, 0, None) == 1
    assert f(A, A, A, A, A, None, 1, 1, 24, None, 0, None) == 2      # K % 32
    assert f(A, A, A, A, A, None, 1, 1, 262144, None, 0, None) == 2  # accumulator headroom
    assert f(A, A, A, A, U, None, 1, 1, 32, None, 0, None) == 3
    assert lib.qil_ref_gemv_bf16(A, None, A, 1, 8, None) == 1
    assert lib.qil_probe_hbm_read(A, 8, A, None) == 2
    assert lib.qil_device_status(None, None, None) == 1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(_lib, "_lib", None)
    monkeypatch.setattr(_lib, "LIB_PATH", str(tmp_path / "libqil.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        _lib.load()


def test_w8_validation(lib):
    f = lib.qil_linear_w8a16
    assert f(None, A, A, A, A, 1, 16, 128, 128, A, 256, None) == 1
    assert f(A, A, A, A, A, 1, 16, 120, 120, A, 256, None) == 2          # K % 16
    assert f(A, A, A, A, A, 1, 16, 128, 96, A, 256, None) == 2           # group does not divide K
    assert f(A, A, A, A, A, 1, 16, 128, 128, None, 0, None) == 5         # workspace
    assert f(U, A, A, A, A, 1, 16, 128, 128, A, 256, None) == 3
    assert lib.qil_linear_w8a16_workspace_size(1, 16, 128, 128) >= 8
    assert lib.qil_linear_w8a16_batch(None, 1, A, 256, None) == 1
    assert lib.qil_quantize_rtn_w8(A, 0, 4, 8, 3, 0, A, A, 2, A, None, None) == 2
    assert lib.qil_quantize_act_a8(A, 4, 12, None, A, A, None) == 2
    assert lib.qil_set_wait_limit_ns(0) == 0
    assert lib.qil_linear_w8a8(A, A, A, A, A, None, 4, 4, 24, A, 16, None) == 2     # K % 16
    assert lib.qil_linear_w8a8(A, A, A, A, A, None, 4, 4, 32, None, 0, None) == 5
    assert lib.qil_probe_mma_i8(0, 8, None, None, None) == 2
