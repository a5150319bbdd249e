"""Thin Python binding of the qil C ABI (same names as ``include/qil.h``).

Only argument marshalling happens here: tensors are allocated with torch, their
device pointers and sizes are passed to ``libqil.so`` and the status code is
turned into an exception.  All arithmetic runs in the CUDA kernels.
"""
from __future__ import annotations

import ctypes as C

import torch

from . import _lib

OK = 0
F32, BF16, F16 = 0, 1, 2
LAYOUT_CANONICAL, LAYOUT_TILE16, LAYOUT_STREAM128 = 0, 1, 3
DEP_PREVIOUS = 1
DEP_NEVER = 2
ERR_RANGE = 8

_DT = {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16}


class QilError(RuntimeError):
    def __init__(self, code: int):
        self.code = int(code)
        msg = _lib.load().qil_status_string(self.code).decode()
        super().__init__(f"qil status {self.code}: {msg}")


def _check(code: int) -> None:
    if code != OK:
        raise QilError(code)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _need_cuda(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("qil needs contiguous CUDA tensors")


def version() -> int:
    return int(_lib.load().qil_version())


def quantize_rtn_w4(w, group_size: int, symmetric: bool = False, scale_dtype=None, stream=None):
    """Round-to-nearest 4-bit weight quantiser.  Returns (codes, scales, zeros) ; zeros is None when symmetric.

    codes: uint8 [N][K] (asymmetric, 0..15) or int8 [N][K] (symmetric, -8..7)."""
    lib = _lib.load()
    _need_cuda(w)
    N, K = w.shape
    if scale_dtype is None:
        scale_dtype = torch.float32 if symmetric else torch.float16
    if group_size <= 0 or K % group_size != 0:
        _check(2)
    ng = K // group_size
    codes = torch.empty((N, K), dtype=torch.int8 if symmetric else torch.uint8, device=w.device)
    scales = torch.empty((N, ng), dtype=scale_dtype, device=w.device)
    zeros = None if symmetric else torch.empty((N, ng), dtype=torch.float16, device=w.device)
    status = torch.zeros(1, dtype=torch.int32, device=w.device)
    _check(lib.qil_quantize_rtn_w4(_ptr(w), _DT[w.dtype], N, K, int(group_size), int(bool(symmetric)), _ptr(codes),
                                   _ptr(scales), _DT[scale_dtype], _ptr(zeros), _ptr(status), _stream(stream)))
    out = C.c_int(0)
    _check(lib.qil_device_status(_ptr(status), C.byref(out), _stream(stream)))
    if out.value:
        raise QilError(ERR_RANGE if out.value & ERR_RANGE else out.value)
    return codes, scales, zeros


def quantize_rtn_w8(w, group_size: int, symmetric: bool = False, scale_dtype=None, stream=None):
    """Round-to-nearest 8-bit weight quantiser: (codes uint8 0..255 / int8 -128..127, scales, zeros or None)."""
    lib = _lib.load()
    _need_cuda(w)
    N, K = w.shape
    if scale_dtype is None:
        scale_dtype = torch.float32 if symmetric else torch.float16
    if group_size <= 0 or K % group_size != 0:
        _check(2)
    ng = K // group_size
    codes = torch.empty((N, K), dtype=torch.int8 if symmetric else torch.uint8, device=w.device)
    scales = torch.empty((N, ng), dtype=scale_dtype, device=w.device)
    zeros = None if symmetric else torch.empty((N, ng), dtype=torch.float16, device=w.device)
    status = torch.zeros(1, dtype=torch.int32, device=w.device)
    _check(lib.qil_quantize_rtn_w8(_ptr(w), _DT[w.dtype], N, K, int(group_size), int(bool(symmetric)), _ptr(codes),
                                   _ptr(scales), _DT[scale_dtype], _ptr(zeros), _ptr(status), _stream(stream)))
    out = C.c_int(0)
    _check(lib.qil_device_status(_ptr(status), C.byref(out), _stream(stream)))
    if out.value:
        raise QilError(ERR_RANGE if out.value & ERR_RANGE else out.value)
    return codes, scales, zeros


def linear_w8a16(x, codes, scales, zeros, group_size: int, out=None, workspace=None, stream=None):
    """y[M][N] (bf16) = x[M][K] (bf16) . dequant(W)^T with 8-bit group-quantised W (codes uint8 [N][K])."""
    _need_cuda(x, codes, scales, zeros, out, workspace)
    M, K = x.shape
    N = codes.shape[0]
    lib = _lib.load()
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    if workspace is None:
        workspace = new_workspace(int(lib.qil_linear_w8a16_workspace_size(M, N, K, int(group_size))), x.device)
    _check(lib.qil_linear_w8a16(_ptr(x), _ptr(codes), _ptr(scales), _ptr(zeros), _ptr(out), M, N, K, int(group_size),
                                _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))
    return out


def quantize_act_a8(x, static_scale: float | None = None, stream=None):
    """bf16 x [M][K] -> (int8 codes [M][K], scales [M] fp32)."""
    _need_cuda(x)
    M, K = x.shape
    qx = torch.empty((M, K), dtype=torch.int8, device=x.device)
    scales = torch.empty((M,), dtype=torch.float32, device=x.device)
    ss = None if static_scale is None else C.byref(C.c_float(static_scale))
    _check(_lib.load().qil_quantize_act_a8(_ptr(x), M, K, ss, _ptr(qx), _ptr(scales), _stream(stream)))
    return qx, scales


def pack_w4(codes, layout: int = LAYOUT_CANONICAL, stream=None):
    """codes [N][K] (uint8 or int8) -> packed words: [N][K/8] (canonical) or flat [N*K/8] (TILE16)."""
    _need_cuda(codes)
    N, K = codes.shape
    shape = (N, max(K // 8, 0)) if layout == LAYOUT_CANONICAL else (N * max(K // 8, 0),)
    packed = torch.empty(shape, dtype=torch.int32, device=codes.device)
    _check(_lib.load().qil_pack_w4(_ptr(codes), N, K, int(layout), _ptr(packed), _stream(stream)))
    return packed


def pack_stream128_w4(codes, scales, zeros, group_size: int, stream=None):
    """codes uint8 [N][K] + fp16 scales/zeros [N][K/G] -> the STREAM128 buffer of the tcgen05 decode kernel."""
    _need_cuda(codes, scales, zeros)
    N, K = codes.shape
    lib = _lib.load()
    nbytes = int(lib.qil_stream128_w4_bytes(N, K))
    out = torch.empty((max(nbytes, 16),), dtype=torch.uint8, device=codes.device)
    _check(lib.qil_pack_stream128_w4(_ptr(codes), _ptr(scales), _ptr(zeros), N, K, int(group_size), _ptr(out),
                                     _stream(stream)))
    return out


def unpack_w4(packed, N: int, K: int, layout: int = LAYOUT_CANONICAL, signed: bool = False, stream=None):
    _need_cuda(packed)
    codes = torch.empty((N, K), dtype=torch.int8 if signed else torch.uint8, device=packed.device)
    _check(_lib.load().qil_unpack_w4(_ptr(packed), N, K, int(layout), int(bool(signed)), _ptr(codes), _stream(stream)))
    return codes


def linear_w4a16_workspace_size(M: int, N: int, K: int, group_size: int) -> int:
    return int(_lib.load().qil_linear_w4a16_workspace_size(M, N, K, group_size))


def new_workspace(nbytes: int, device="cuda"):
    """A zero-filled workspace of at least ``nbytes`` bytes (zero-filling is required once)."""
    return torch.zeros(max(int(nbytes), 16), dtype=torch.uint8, device=device)


def linear_w4a16(x, qweight, scales, zeros, N: int, group_size: int, layout: int = LAYOUT_CANONICAL, out=None,
                 workspace=None, stream=None):
    """y[M][N] (bf16) = x[M][K] (bf16) . dequant(W)^T with 4-bit group-quantised W."""
    _need_cuda(x, qweight, scales, zeros, out, workspace)
    M, K = x.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    if workspace is None:
        need = linear_w4a16_workspace_size(M, N, K, group_size)
        workspace = new_workspace(need, x.device) if need else None
    _check(_lib.load().qil_linear_w4a16(_ptr(x), _ptr(qweight), _ptr(scales), _ptr(zeros), _ptr(out), M, N, K,
                                        int(group_size), int(layout), _ptr(workspace),
                                        0 if workspace is None else workspace.numel() * workspace.element_size(),
                                        _stream(stream)))
    return out


def lora_side_workspace_size(M: int) -> int:
    return int(_lib.load().qil_lora_side_workspace_size(M))


def lora_side_add(x, a, b, y, scale: float = 1.0, workspace=None, stream=None):
    """y[M][N] (bf16, in place) += scale * (x[M][K] . a[r][K]^T) . b[N][r]^T: an unmerged low-rank adapter, r <= 32."""
    _need_cuda(x, a, b, y, workspace)
    M, K = x.shape
    r = a.shape[0]
    N = b.shape[0]
    assert a.shape == (r, K) and b.shape == (N, r) and y.shape == (M, N)
    if workspace is None:
        workspace = torch.empty(max(int(_lib.load().qil_lora_side_workspace_size(M)), 16), dtype=torch.uint8, device=x.device)
    _check(_lib.load().qil_lora_side_add(_ptr(x), _ptr(a), _ptr(b), _ptr(y), M, N, K, r, float(scale), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)))
    return y


def interleave_rows(gate, up):
    """Rows 2i = gate[i], 2i + 1 = up[i] (codes, scales or zeros of the two projections of a gated MLP): the weight
    layout `linear_w4a16_swiglu` expects.  A layout step done once, offline."""
    assert gate.shape == up.shape
    return torch.stack((gate, up), dim=1).reshape(2 * gate.shape[0], *gate.shape[1:]).contiguous()


def linear_w4a16_swiglu_workspace_size(M: int, N: int, K: int, group_size: int) -> int:
    return int(_lib.load().qil_linear_w4a16_swiglu_workspace_size(M, N, K, group_size))


def linear_w4a16_swiglu(x, qweight, scales, zeros, N: int, group_size: int, out=None, workspace=None, stream=None):
    """y[M][N/2] (bf16) = silu(x . dequant(W[0::2])^T) * (x . dequant(W[1::2])^T): gate and up rows interleaved in W."""
    _need_cuda(x, qweight, scales, zeros, out, workspace)
    M, K = x.shape
    if out is None:
        out = torch.empty((M, N // 2), dtype=torch.bfloat16, device=x.device)
    if workspace is None:
        workspace = new_workspace(linear_w4a16_swiglu_workspace_size(M, N, K, group_size), x.device)
    _check(_lib.load().qil_linear_w4a16_swiglu(_ptr(x), _ptr(qweight), _ptr(scales), _ptr(zeros), _ptr(out), M, N, K,
                                               int(group_size), _ptr(workspace),
                                               workspace.numel() * workspace.element_size(), _stream(stream)))
    return out


def quantize_act_a4(x, static_scale: float | None = None, stream=None):
    """bf16 x [M][K] -> (packed int4 codes [M][K/8] int32, scales [M] fp32)."""
    _need_cuda(x)
    M, K = x.shape
    qx = torch.empty((M, max(K // 8, 0)), dtype=torch.int32, device=x.device)
    scales = torch.empty((M,), dtype=torch.float32, device=x.device)
    ss = None if static_scale is None else C.byref(C.c_float(static_scale))
    _check(_lib.load().qil_quantize_act_a4(_ptr(x), M, K, ss, _ptr(qx), _ptr(scales), _stream(stream)))
    return qx, scales


def linear_w4a4_workspace_size(M: int, N: int, K: int) -> int:
    return int(_lib.load().qil_linear_w4a4_workspace_size(M, N, K))


def linear_w4a4(qx, sx, qw, sw, want_acc: bool = False, out=None, workspace=None, stream=None):
    """Integer GEMM of packed int4 operands; returns y (bf16) or (y, acc int32)."""
    _need_cuda(qx, sx, qw, sw, out, workspace)
    M, K = qx.shape[0], qx.shape[1] * 8
    N = qw.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=qx.device)
    acc = torch.empty((M, N), dtype=torch.int32, device=qx.device) if want_acc else None
    if workspace is None:
        need = linear_w4a4_workspace_size(M, N, K)
        workspace = new_workspace(need, qx.device) if need else None
    _check(_lib.load().qil_linear_w4a4(_ptr(qx), _ptr(sx), _ptr(qw), _ptr(sw), _ptr(out), _ptr(acc), M, N, K,
                                       _ptr(workspace),
                                       0 if workspace is None else workspace.numel() * workspace.element_size(),
                                       _stream(stream)))
    return (out, acc) if want_acc else out


def linear_w4a4_requant(qx, sx, qw, sw, out_scale: float, relu: bool = False, workspace=None, stream=None):
    """W4A4 GEMM whose epilogue quantises the output for the next layer: returns packed int4 codes [M][N/8]."""
    _need_cuda(qx, sx, qw, sw, workspace)
    M, K = qx.shape[0], qx.shape[1] * 8
    N = qw.shape[0]
    qy = torch.empty((M, max(N // 8, 1)), dtype=torch.int32, device=qx.device)
    if workspace is None:
        workspace = new_workspace(linear_w4a4_workspace_size(M, N, K), qx.device)
    _check(_lib.load().qil_linear_w4a4_requant(_ptr(qx), _ptr(sx), _ptr(qw), _ptr(sw), _ptr(qy), C.c_float(out_scale),
                                               int(bool(relu)), M, N, K, _ptr(workspace),
                                               workspace.numel() * workspace.element_size(), _stream(stream)))
    return qy


def conv3x3_w4a4(qx, x_scale: float, qw, sw, out_scale: float | None = None, relu: bool = False, want_acc: bool = False,
                 workspace=None, stream=None):
    """3 x 3 convolution (stride 1, zero padding 1) on an int4 feature map qx [B][H][W][C/8] with filters qw
    [Cout][9C/8] (column (3 kh + kw) C + c).  out_scale None: returns bf16 y [B][H][W][Cout] (and the int32
    accumulators if want_acc); else the next layer's packed int4 feature map [B][H][W][Cout/8]."""
    _need_cuda(qx, qw, sw, workspace)
    B, H, W = qx.shape[0], qx.shape[1], qx.shape[2]
    Cin, Cout = qx.shape[3] * 8, qw.shape[0]
    assert qw.shape[1] * 8 == 9 * Cin
    y = acc = qy = None
    if out_scale is None:
        y = torch.empty((B, H, W, Cout), dtype=torch.bfloat16, device=qx.device)
        if want_acc:
            acc = torch.empty((B, H, W, Cout), dtype=torch.int32, device=qx.device)
    else:
        qy = torch.empty((B, H, W, max(Cout // 8, 1)), dtype=torch.int32, device=qx.device)
    if workspace is None:
        workspace = new_workspace(linear_w4a4_workspace_size(B * H * W, Cout, 9 * Cin), qx.device)
    _check(_lib.load().qil_conv3x3_w4a4(_ptr(qx), C.c_float(x_scale), _ptr(qw), _ptr(sw), _ptr(y), _ptr(acc), _ptr(qy),
                                        C.c_float(out_scale if out_scale is not None else 1.0), int(bool(relu)), B, H, W, Cin,
                                        Cout, _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))
    if out_scale is not None:
        return qy
    return (y, acc) if want_acc else y


def linear_int_batch(entries, workspace=None, stream=None):
    """A list of independent integer GEMMs in one launch.  entries: [(qx, sx, qw, sw, y, acc or None, bits)] with the
    operands of linear_w4a4 (bits 4) or linear_w8a8 (bits 8); outputs are written into y (and acc)."""
    descs = (_lib.IGemmDesc * len(entries))()
    dev = None
    for d, (qx, sx, qw, sw, y, acc, bits) in zip(descs, entries):
        _need_cuda(qx, sx, qw, sw, y, acc)
        dev = qx.device
        d.qx, d.sx, d.qw, d.sw, d.y = qx.data_ptr(), sx.data_ptr(), qw.data_ptr(), sw.data_ptr(), y.data_ptr()
        d.acc_out = None if acc is None else acc.data_ptr()
        d.M, d.N = y.shape
        d.K = qx.shape[1] * (8 if bits == 4 else 1)
        d.bits = bits
    if workspace is None:
        workspace = new_workspace(16, dev)
    _check(_lib.load().qil_linear_int_batch(descs, len(entries), _ptr(workspace),
                                            workspace.numel() * workspace.element_size(), _stream(stream)))


def linear_w8a8(qx, sx, qw, sw, want_acc: bool = False, out=None, workspace=None, stream=None):
    """Integer GEMM of int8 operands (qx [M][K], qw [N][K]); returns y (bf16) or (y, acc int32)."""
    _need_cuda(qx, sx, qw, sw, out, workspace)
    M, K = qx.shape
    N = qw.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=qx.device)
    acc = torch.empty((M, N), dtype=torch.int32, device=qx.device) if want_acc else None
    if workspace is None:
        workspace = new_workspace(linear_w4a4_workspace_size(M, N, K), qx.device)
    _check(_lib.load().qil_linear_w8a8(_ptr(qx), _ptr(sx), _ptr(qw), _ptr(sw), _ptr(out), _ptr(acc), M, N, K,
                                       _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))
    return (out, acc) if want_acc else out


def ref_gemv_bf16(x, w, out=None, stream=None):
    _need_cuda(x, w, out)
    N, K = w.shape
    if out is None:
        out = torch.empty((N,), dtype=torch.bfloat16, device=w.device)
    _check(_lib.load().qil_ref_gemv_bf16(_ptr(x), _ptr(w), _ptr(out), N, K, _stream(stream)))
    return out


def probe_hbm_read(buf, sink, stream=None):
    _need_cuda(buf, sink)
    _check(_lib.load().qil_probe_hbm_read(_ptr(buf), buf.numel() * buf.element_size(), _ptr(sink), _stream(stream)))


def probe_mma(kind: str, iters: int, commit_every: int = 8, status=None, stream=None) -> float:
    """Launches the tensor-core probe ("i8" or "bf16"); returns the operations of the launch (the caller times it)."""
    lib = _lib.load()
    ops = C.c_double(0.0)
    fn = lib.qil_probe_mma_i8 if kind == "i8" else lib.qil_probe_mma_bf16
    _check(fn(int(iters), int(commit_every), C.byref(ops), _ptr(status), _stream(stream)))
    return float(ops.value)
