"""Loads ``libqil.so`` and declares the C ABI of ``include/qil.h`` for ctypes."""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqil.so")

# name -> (restype, argtypes); mirrors include/qil.h one to one
_vp, _i, _sz = C.c_void_p, C.c_int, C.c_size_t
SIGNATURES = {
    "qil_quantize_rtn_w4": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _vp, _i, _vp, _vp, _vp]),
    "qil_pack_w4": (_i, [_vp, _i, _i, _i, _vp, _vp]),
    "qil_unpack_w4": (_i, [_vp, _i, _i, _i, _i, _vp, _vp]),
    "qil_stream128_w4_bytes": (_sz, [_i, _i]),
    "qil_pack_stream128_w4": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _vp]),
    "qil_linear_w4a16_workspace_size": (_sz, [_i, _i, _i, _i]),
    "qil_linear_w4a16": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _sz, _vp]),
    "qil_lora_side_workspace_size": (_sz, [_i]),
    "qil_lora_side_add": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, C.c_float, _vp, _sz, _vp]),
    "qil_linear_w4a16_swiglu_workspace_size": (_sz, [_i, _i, _i, _i]),
    "qil_linear_w4a16_swiglu": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _sz, _vp]),
    "qil_linear_w4a16_static_ws": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]),
    "qil_linear_w4a16_static_ws_need": (_sz, [_i, _i, _i, _i]),
    "qil_set_wait_limit_ns": (_i, [C.c_ulonglong]),
    "qil_linear_w4a16_batch": (_i, [_vp, _i, _vp, _sz, _vp]),
    "qil_linear_w4a16_batch_host": (_i, [_vp, _i, _vp, _vp, _sz, _vp, _vp, _sz, _vp, _sz, _vp]),
    "qil_quantize_rtn_w8": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _vp, _i, _vp, _vp, _vp]),
    "qil_linear_w8a16_workspace_size": (_sz, [_i, _i, _i, _i]),
    "qil_linear_w8a16": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _sz, _vp]),
    "qil_linear_w8a16_batch": (_i, [_vp, _i, _vp, _sz, _vp]),
    "qil_quantize_act_a8": (_i, [_vp, _i, _i, C.POINTER(C.c_float), _vp, _vp, _vp]),
    "qil_quantize_act_a4": (_i, [_vp, _i, _i, C.POINTER(C.c_float), _vp, _vp, _vp]),
    "qil_linear_w4a4_workspace_size": (_sz, [_i, _i, _i]),
    "qil_linear_w4a4": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "qil_conv3x3_w4a4": (_i, [_vp, C.c_float, _vp, _vp, _vp, _vp, _vp, C.c_float, _i, _i, _i, _i, _i, _i, _vp, _sz, _vp]),
    "qil_linear_w4a4_requant": (_i, [_vp, _vp, _vp, _vp, _vp, C.c_float, _i, _i, _i, _i, _vp, _sz, _vp]),
    "qil_linear_w8a8": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp, _sz, _vp]),
    "qil_linear_int_batch": (_i, [_vp, _i, _vp, _sz, _vp]),
    "qil_status_string": (C.c_char_p, [_i]),
    "qil_version": (_i, []),
    "qil_device_status": (_i, [_vp, C.POINTER(C.c_int), _vp]),
    "qil_ref_gemv_bf16": (_i, [_vp, _vp, _vp, _i, _i, _vp]),
    "qil_probe_hbm_read": (_i, [_vp, _sz, _vp, _vp]),
    "qil_probe_mma_i8": (_i, [_i, _i, C.POINTER(C.c_double), _vp, _vp]),
    "qil_probe_mma_bf16": (_i, [_i, _i, C.POINTER(C.c_double), _vp, _vp]),
}



class LinearDesc(C.Structure):
    """ctypes mirror of ``qil_linear_desc``."""
    _fields_ = [("x", _vp), ("qweight", _vp), ("scales", _vp), ("zeros", _vp), ("y", _vp),
                ("M", _i), ("N", _i), ("K", _i), ("group_size", _i), ("layout", _i), ("flags", _i)]


class IGemmDesc(C.Structure):
    """ctypes mirror of ``qil_igemm_desc``."""
    _fields_ = [("qx", _vp), ("sx", _vp), ("qw", _vp), ("sw", _vp), ("y", _vp), ("acc_out", _vp),
                ("M", _i), ("N", _i), ("K", _i), ("bits", _i)]


_lib = None


def load() -> C.CDLL:
    """Returns the loaded library; raises if it was never built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2412_01034_b200.build` "
                "(the library has no CPU or PyTorch fallback)")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib
