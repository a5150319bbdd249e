"""ctypes wrapper around the plain-C oracle (test infrastructure only).

``build()`` compiles ``oracle/c/qil_oracle.c`` with gcc into a shared object
next to the source; ``load()`` builds on demand.  The wrapper only marshals
NumPy arrays; all arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "c", "qil_oracle.c")
_SO = os.path.join(_HERE, "c", "libqil_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
               "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.qo_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(load().qo_num_threads())


def quantize_rtn_w4_asym(w, group_size):
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, K = w.shape
    ng = K // group_size
    codes = np.empty((N, K), np.uint8)
    scales = np.empty((N, ng), np.uint16)
    zeros = np.empty((N, ng), np.uint16)
    rc = load().qo_quantize_rtn_w4_asym(_p(w), N, K, int(group_size), _p(codes), _p(scales), _p(zeros))
    if rc:
        raise OverflowError("scale does not fit fp16")
    return codes, scales.view(np.float16), zeros.view(np.float16)


def quantize_sym4(v, group_size=None, scale_f16=False, static_scale=None):
    v = np.ascontiguousarray(v, dtype=np.float32)
    R, K = v.shape
    G = K if group_size is None else int(group_size)
    ng = K // G
    codes = np.empty((R, K), np.int8)
    scales = np.empty((R, ng), np.uint16 if scale_f16 else np.float32)
    ss = None if static_scale is None else C.byref(C.c_float(static_scale))
    rc = load().qo_quantize_sym4(_p(v), R, K, G, int(bool(scale_f16)), ss, _p(codes), _p(scales))
    if rc:
        raise OverflowError("scale does not fit fp16")
    return codes, (scales.view(np.float16) if scale_f16 else scales)


def pack_w4(codes):
    c = np.ascontiguousarray(codes).view(np.uint8)
    R, K = c.shape
    out = np.empty((R, K // 8), np.uint32)
    load().qo_pack_w4(_p(c), R, K, _p(out))
    return out


def unpack_w4(packed, signed=False):
    p = np.ascontiguousarray(packed, dtype=np.uint32)
    R, W = p.shape
    out = np.empty((R, W * 8), np.uint8)
    load().qo_unpack_w4(_p(p), R, W * 8, int(bool(signed)), _p(out))
    return out.view(np.int8) if signed else out


def to_tile16(packed):
    p = np.ascontiguousarray(packed, dtype=np.uint32)
    N, W = p.shape
    out = np.empty(N * W, np.uint32)
    load().qo_to_tile16(_p(p), N, W * 8, _p(out))
    return out


def linear_w4a16(x_bf16_bits, codes, scales, zeros, group_size):
    x = np.ascontiguousarray(x_bf16_bits, dtype=np.uint16)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    s = np.ascontiguousarray(scales).view(np.uint16)
    z = np.ascontiguousarray(zeros).view(np.uint16)
    M, K = x.shape
    N = codes.shape[0]
    y = np.empty((M, N), np.float64)
    load().qo_linear_w4a16(_p(x), _p(codes), _p(s), _p(z), M, N, K, int(group_size), _p(y))
    return y


def linear_w4a4(qx, sx, qw, sw, want_y=True):
    qx = np.ascontiguousarray(qx, dtype=np.int8)
    qw = np.ascontiguousarray(qw, dtype=np.int8)
    sx = np.ascontiguousarray(sx, dtype=np.float32).reshape(-1)
    sw = np.ascontiguousarray(sw, dtype=np.float32).reshape(-1)
    M, K = qx.shape
    N = qw.shape[0]
    acc = np.empty((M, N), np.int64)
    y = np.empty((M, N), np.float64) if want_y else None
    load().qo_linear_w4a4(_p(qx), _p(sx), _p(qw), _p(sw), M, N, K, _p(acc), _p(y) if want_y else None)
    return acc, y


# ---- 8-bit variants (the C loops of the two linears do not depend on the code width) ----
def quantize_rtn_asym(w, group_size, bits):
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, K = w.shape
    ng = K // group_size
    codes = np.empty((N, K), np.uint8)
    scales = np.empty((N, ng), np.uint16)
    zeros = np.empty((N, ng), np.uint16)
    rc = load().qo_quantize_rtn_asym(_p(w), N, K, int(group_size), int(bits), _p(codes), _p(scales), _p(zeros))
    if rc:
        raise OverflowError("scale does not fit fp16")
    return codes, scales.view(np.float16), zeros.view(np.float16)


def quantize_rtn_w8_asym(w, group_size):
    return quantize_rtn_asym(w, group_size, 8)


def quantize_sym(v, bits, group_size=None, static_scale=None):
    v = np.ascontiguousarray(v, dtype=np.float32)
    R, K = v.shape
    G = K if group_size is None else int(group_size)
    codes = np.empty((R, K), np.int8)
    scales = np.empty((R, K // G), np.float32)
    ss = None if static_scale is None else C.byref(C.c_float(static_scale))
    load().qo_quantize_sym(_p(v), R, K, G, int(bits), ss, _p(codes), _p(scales))
    return codes, scales


def quantize_sym8(v, group_size=None, static_scale=None):
    return quantize_sym(v, 8, group_size, static_scale)


def linear_w8a16(x_bf16_bits, codes, scales, zeros, group_size):
    return linear_w4a16(x_bf16_bits, codes, scales, zeros, group_size)


def linear_w8a8(qx, sx, qw, sw, want_y=True):
    return linear_w4a4(qx, sx, qw, sw, want_y)


def linear_w4a4_requant(qx, sx, qw, sw, out_scale, relu):
    qx = np.ascontiguousarray(qx, dtype=np.int8)
    qw = np.ascontiguousarray(qw, dtype=np.int8)
    sx = np.ascontiguousarray(sx, dtype=np.float32).reshape(-1)
    sw = np.ascontiguousarray(sw, dtype=np.float32).reshape(-1)
    M, K = qx.shape
    N = qw.shape[0]
    q = np.empty((M, N), np.int8)
    load().qo_linear_w4a4_requant(_p(qx), _p(sx), _p(qw), _p(sw), M, N, K, C.c_float(out_scale), int(bool(relu)), _p(q))
    return q
