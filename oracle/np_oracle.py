"""NumPy oracle of the quantised linear layer (test infrastructure only).

What the paper fixes: weights and/or activations of a GEMM are mapped to a
low-bit uniform grid by round-to-nearest (Sec. 2.1, "Quantization for Efficient
DNN Inference"); OpenVLA runs 4-bit weight-only linears whose decode stage is
memory bound (Sec. 5.4 "Implementation", App. A.4.2); CILRS runs 4-bit weights
and 4-bit activations (Sec. 5.1, App. A.1.2).  The paper prints no formula for
the quantiser, so the operation sequence below is this library's reading of
"round-to-nearest uniform quantiser", written step by step so that a CPU and
a GPU can agree bit for bit:

  * fp32 arithmetic, IEEE round-to-nearest-even for every +, -, / ;
  * "round" means round-half-to-even (numpy.rint);
  * true division (never multiply by a reciprocal).

Conventions: W is [N][K] (output features x input features), groups of
``group_size`` consecutive k share a scale (and a zero point), x is [M][K],
y[m][n] = sum_k x[m][k] * W_hat[n][k].

bf16 tensors are carried as uint16 bit patterns; ``bf16_to_f32`` widens them.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32


# ----------------------------------------------------------------------------
# bf16 widening (exact): a bf16 value is the upper 16 bits of an fp32.
# ----------------------------------------------------------------------------
def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# Asymmetric uint4 group quantiser (weights of the weight-only linear).
# Reading of Sec. 2.1 (round-to-nearest) with an integer zero point; the group
# range always contains 0 so that 0 is exactly representable.
# ----------------------------------------------------------------------------
def quantize_rtn_w4_asym(w: np.ndarray, group_size: int):
    """w fp32 [N][K] -> (codes u8 [N][K] in 0..15, scales f16 [N][K/G], zeros f16 [N][K/G]).

    Per (row n, group g):
      lo = min(0, min w), hi = max(0, max w)
      s32 = (hi - lo) / 15            (fp32)
      s16 = fp16(s32); 0 -> 1.0; inf -> error
      z   = clamp(rint(-lo / s16), 0, 15)
      q_k = clamp(rint(w_k / s16) + z, 0, 15)
    """
    w = np.ascontiguousarray(w, dtype=F32)
    N, K = w.shape
    G = int(group_size)
    if G <= 0 or K % G != 0:
        raise ValueError("group_size must divide K")
    ng = K // G
    wg = w.reshape(N, ng, G)
    lo = np.minimum(F32(0), wg.min(axis=2)).astype(F32)
    hi = np.maximum(F32(0), wg.max(axis=2)).astype(F32)
    r = (hi - lo).astype(F32)
    s32 = (r / F32(15.0)).astype(F32)
    with np.errstate(over="ignore"):
        s16 = s32.astype(np.float16)
    if np.isinf(s16).any():
        raise OverflowError("scale does not fit fp16")
    s16 = np.where(s16 == np.float16(0), np.float16(1.0), s16).astype(np.float16)
    s = s16.astype(F32)
    z = np.clip(np.rint((-lo / s).astype(F32)), F32(0), F32(15)).astype(F32)
    u = (np.rint((wg / s[:, :, None]).astype(F32)) + z[:, :, None]).astype(F32)
    q = np.clip(u, F32(0), F32(15))
    codes = q.astype(np.uint8).reshape(N, K)
    # the zero point is an integer: store it as fp16(int(z)) (never a negative zero)
    return codes, s16, z.astype(np.uint8).astype(np.float16)


def unclamped_levels_asym(w: np.ndarray, group_size: int):
    """rint(w/s)+z before the final clamp; used only by the error-bound pins."""
    w = np.ascontiguousarray(w, dtype=F32)
    N, K = w.shape
    G = int(group_size)
    _, s16, z16 = quantize_rtn_w4_asym(w, G)
    s = s16.astype(F32)
    z = z16.astype(F32)
    wg = w.reshape(N, K // G, G)
    u = np.rint((wg / s[:, :, None]).astype(F32)) + z[:, :, None]
    return u.reshape(N, K)


# ----------------------------------------------------------------------------
# Symmetric int4 quantiser (per-channel weights and per-token activations of
# the W4A4 path; Sec. 5.1 / App. A.1.2 use 4-bit weights and activations).
# ----------------------------------------------------------------------------
def quantize_sym4(v: np.ndarray, group_size: int | None = None, scale_f16: bool = False,
                  static_scale: float | None = None):
    """v fp32 [R][K] -> (codes int8 [R][K] in -8..7, scales [R][K/G]).

    Per (row, group): a = max|v|; s = a / 7 (fp32); a == 0 -> s = 1.
    With ``scale_f16`` the scale is rounded to fp16 first (0 -> 1, inf -> error)
    and the codes are computed with the rounded value.  With ``static_scale``
    every group uses that fp32 value.  q = clamp(rint(v / s), -8, 7).
    """
    v = np.ascontiguousarray(v, dtype=F32)
    R, K = v.shape
    G = K if group_size is None else int(group_size)
    if G <= 0 or K % G != 0:
        raise ValueError("group_size must divide K")
    ng = K // G
    vg = v.reshape(R, ng, G)
    if static_scale is not None:
        s = np.full((R, ng), F32(static_scale), dtype=F32)
    else:
        a = np.abs(vg).max(axis=2).astype(F32)
        s = (a / F32(7.0)).astype(F32)
        s = np.where(a == F32(0), F32(1.0), s).astype(F32)
    if scale_f16:
        with np.errstate(over="ignore"):
            s16 = s.astype(np.float16)
        if np.isinf(s16).any():
            raise OverflowError("scale does not fit fp16")
        s16 = np.where(s16 == np.float16(0), np.float16(1.0), s16).astype(np.float16)
        s = s16.astype(F32)
        s_out = s16
    else:
        s_out = s
    q = np.clip(np.rint((vg / s[:, :, None]).astype(F32)), F32(-8), F32(7))
    return q.astype(np.int8).reshape(R, K), s_out


# ----------------------------------------------------------------------------
# Packing: 8 four-bit codes per uint32, element k of a row in word k//8 at bits
# [4*(k%8), 4*(k%8)+3] (little-nibble first).  Signed codes keep their two's
# complement low nibble.
# ----------------------------------------------------------------------------
LAYOUT_CANONICAL = 0
LAYOUT_TILE16 = 1


def pack_w4(codes: np.ndarray) -> np.ndarray:
    """codes [R][K] (u8 0..15 or int8 -8..7) -> uint32 [R][K/8], canonical layout."""
    c = np.asarray(codes)
    R, K = c.shape
    if K % 8 != 0:
        raise ValueError("K must be a multiple of 8")
    nib = (c.astype(np.int64) & 0xF).astype(np.uint32).reshape(R, K // 8, 8)
    out = np.zeros((R, K // 8), dtype=np.uint32)
    for j in range(8):
        out |= nib[:, :, j] << np.uint32(4 * j)
    return out


def unpack_w4(packed: np.ndarray, signed: bool = False) -> np.ndarray:
    p = np.asarray(packed, dtype=np.uint32)
    R, Wd = p.shape
    out = np.zeros((R, Wd, 8), dtype=np.int16)
    for j in range(8):
        out[:, :, j] = ((p >> np.uint32(4 * j)) & np.uint32(0xF)).astype(np.int16)
    out = out.reshape(R, Wd * 8)
    if signed:
        out = np.where(out >= 8, out - 16, out)
        return out.astype(np.int8)
    return out.astype(np.uint8)


def to_layout(packed: np.ndarray, layout: int) -> np.ndarray:
    """Rearrange canonical packed words [N][K/8] into a kernel-private layout (flat uint32).

    LAYOUT_TILE16: the matrix is cut into tiles of 16 rows x 128 columns
    (16 words per row).  Tiles are stored one after another, all column tiles
    of row-tile 0 first; inside a tile the 16 rows follow each other, 16 words
    each.  Word (n, i) lands at
        ((n // 16) * (K // 128) + i // 16) * 256 + (n % 16) * 16 + i % 16.
    Needs N % 16 == 0 and K % 128 == 0.
    """
    p = np.asarray(packed, dtype=np.uint32)
    if layout == LAYOUT_CANONICAL:
        return p.reshape(-1).copy()
    if layout == LAYOUT_TILE16:
        N, Wd = p.shape
        if N % 16 != 0 or Wd % 16 != 0:
            raise ValueError("TILE16 layout needs N % 16 == 0 and K % 128 == 0")
        out = np.zeros(N * Wd, dtype=np.uint32)
        kt = Wd // 16
        for n in range(N):
            for i in range(Wd):
                out[((n // 16) * kt + i // 16) * 256 + (n % 16) * 16 + i % 16] = p[n, i]
        return out
    raise ValueError("unknown layout")


def from_layout(flat: np.ndarray, N: int, K: int, layout: int) -> np.ndarray:
    """Inverse of ``to_layout`` (flat uint32 -> canonical [N][K/8])."""
    f = np.asarray(flat, dtype=np.uint32).reshape(-1)
    Wd = K // 8
    if layout == LAYOUT_CANONICAL:
        return f.reshape(N, Wd).copy()
    if layout == LAYOUT_TILE16:
        out = np.zeros((N, Wd), dtype=np.uint32)
        kt = Wd // 16
        for n in range(N):
            for i in range(Wd):
                out[n, i] = f[((n // 16) * kt + i // 16) * 256 + (n % 16) * 16 + i % 16]
        return out
    raise ValueError("unknown layout")


def to_stream128(codes: np.ndarray, scales, zeros, group_size: int) -> np.ndarray:
    """Codes uint8 [N][K] + fp16 scales/zeros [N][K/G] -> the STREAM128 byte buffer.

    Unit u = (n // 128) * (K // 128) + kb starts at byte 8704 * u.  Its first 8192 bytes are 4 chunks
    (32 columns each) x 128 rows x 16 bytes: byte 4*m + b of (chunk j, row r) holds column 32*j + 8*m + b
    of the block in its low nibble and column 32*j + 8*m + 4 + b in its high nibble.  Then, for each of
    the 128 rows, the fp16 scale followed by the fp16 zero of the group containing block kb.  Rows
    beyond N are all zero.
    """
    c = np.asarray(codes, dtype=np.uint8)
    N, K = c.shape
    G = int(group_size)
    if K % 128 or G % 128 or K % G:
        raise ValueError("STREAM128 layout needs K % 128 == 0 and G % 128 == 0")
    s16 = np.ascontiguousarray(scales, dtype=np.float16).view(np.uint16)
    z16 = np.ascontiguousarray(zeros, dtype=np.float16).view(np.uint16)
    KB, RT = K // 128, (N + 127) // 128
    out = np.zeros(RT * KB * 8704, dtype=np.uint8)
    for rt in range(RT):
        rows = min(128, N - rt * 128)
        for kb in range(KB):
            base = (rt * KB + kb) * 8704
            blk = c[rt * 128:rt * 128 + rows, kb * 128:(kb + 1) * 128]
            for j in range(4):
                for m in range(4):
                    for b in range(4):
                        lo = blk[:, 32 * j + 8 * m + b] & 0xF
                        hi = blk[:, 32 * j + 8 * m + 4 + b] & 0xF
                        off = base + j * 128 * 16 + np.arange(rows) * 16 + 4 * m + b
                        out[off] = lo | (hi << 4)
            meta = np.empty((rows, 2), dtype=np.uint16)
            meta[:, 0] = s16[rt * 128:rt * 128 + rows, (kb * 128) // G]
            meta[:, 1] = z16[rt * 128:rt * 128 + rows, (kb * 128) // G]
            out[base + 8192:base + 8192 + rows * 4] = meta.view(np.uint8).reshape(-1)
    return out


# ----------------------------------------------------------------------------
# Dequantisation and the two linears, in fp64 / int64.
# ----------------------------------------------------------------------------
def dequant_w4_asym(codes, scales, zeros, group_size: int) -> np.ndarray:
    """W_hat[n][k] = (q - z) * s  in fp64."""
    codes = np.asarray(codes)
    N, K = codes.shape
    G = int(group_size)
    q = codes.astype(np.float64).reshape(N, K // G, G)
    s = np.asarray(scales).astype(np.float64)[:, :, None]
    z = np.asarray(zeros).astype(np.float64)[:, :, None]
    return ((q - z) * s).reshape(N, K)


def linear_w4a16(x_bf16_bits, codes, scales, zeros, group_size: int) -> np.ndarray:
    """y[m][n] = sum_k x[m][k] * (q[n][k] - z[n][k/G]) * s[n][k/G], fp64 throughout."""
    x = bf16_to_f32(x_bf16_bits).astype(np.float64)
    w_hat = dequant_w4_asym(codes, scales, zeros, group_size)
    return np.matmul(x, w_hat.T)


def conv3x3_w4a4(q_fmap, x_scale: float, qw, sw):
    """3 x 3 convolution, stride 1, zero padding 1, on integer codes (the W4A4 conv layers of the CILRS-style encoder,
    Sec. 5.1, App. A.1.2; one static activation scale for the tensor):
        acc[b][h][w][n] = sum_{kh, kw, c} q[b][h + kh - 1][w + kw - 1][c] * qw[n][(3 kh + kw) C + c]   (0 outside the image)
        y = acc * x_scale * sw[n]
    q_fmap [B][H][W][C], qw [Cout][9 C] integers; returns (acc int64, y fp64), both [B][H][W][Cout].  Written tap by tap
    from the definition (no im2col matrix)."""
    q = np.asarray(q_fmap).astype(np.int64)
    w = np.asarray(qw).astype(np.int64)
    B, H, W, Cc = q.shape
    Cout = w.shape[0]
    assert w.shape[1] == 9 * Cc
    acc = np.zeros((B, H, W, Cout), dtype=np.int64)
    for kh in range(3):
        for kw in range(3):
            tap = w[:, (3 * kh + kw) * Cc:(3 * kh + kw + 1) * Cc]          # [Cout][C]
            # output pixels (h, w) whose input pixel (h + kh - 1, w + kw - 1) lies inside the image
            h0, h1 = max(0, 1 - kh), min(H, H + 1 - kh)
            w0, w1 = max(0, 1 - kw), min(W, W + 1 - kw)
            if h0 >= h1 or w0 >= w1:
                continue
            src = q[:, h0 + kh - 1:h1 + kh - 1, w0 + kw - 1:w1 + kw - 1, :]
            acc[:, h0:h1, w0:w1, :] += np.matmul(src, tap.T)
    y = acc.astype(np.float64) * float(x_scale) * np.asarray(sw, dtype=np.float64).reshape(1, 1, 1, -1)
    return acc, y


def lora_side(x_bf16_bits, a_bf16_bits, b_bf16_bits, scale: float) -> np.ndarray:
    """The term an unmerged low-rank adapter adds to a linear's output (the paper fine-tunes OpenVLA with QLoRA
    adapters of rank 32 over the frozen quantised base, App. A.1.2): scale * (x . A^T) . B^T, fp64 throughout.
    x [M][K], A [r][K], B [N][r], all given as bf16 bit patterns."""
    x = bf16_to_f32(x_bf16_bits).astype(np.float64)
    a = bf16_to_f32(a_bf16_bits).astype(np.float64)
    b = bf16_to_f32(b_bf16_bits).astype(np.float64)
    return float(scale) * np.matmul(np.matmul(x, a.T), b.T)


def silu(g: np.ndarray) -> np.ndarray:
    """silu(g) = g / (1 + exp(-g)), fp64 (the activation of the Llama-2 gated MLP, the backbone of the paper's OpenVLA
    deployment, App. A.4.2).  Written so that large |g| neither overflows nor loses the small side."""
    g = np.asarray(g, dtype=np.float64)
    e = np.exp(-np.abs(g))                       # in (0, 1]
    return np.where(g >= 0, g / (1.0 + e), g * e / (1.0 + e))


def linear_w4a16_swiglu(x_bf16_bits, codes, scales, zeros, group_size: int) -> np.ndarray:
    """Gate and up projections with rows interleaved (row 2i = gate i, row 2i + 1 = up i) and the gated activation:
    y[m][i] = silu(t[m][2i]) * t[m][2i + 1], t = the plain dequantise-then-matmul, fp64 throughout."""
    t = linear_w4a16(x_bf16_bits, codes, scales, zeros, group_size)
    return silu(t[:, 0::2]) * t[:, 1::2]


def linear_w4a4(qx, sx, qw, sw):
    """acc[m][n] = sum_k qx[m][k]*qw[n][k] (int64); y = acc * sx[m] * sw[n] (fp64)."""
    a = np.asarray(qx).astype(np.int64)
    b = np.asarray(qw).astype(np.int64)
    acc = np.matmul(a, b.T)
    y = acc.astype(np.float64) * np.asarray(sx, dtype=np.float64).reshape(-1, 1) \
        * np.asarray(sw, dtype=np.float64).reshape(1, -1)
    return acc, y


# ----------------------------------------------------------------------------
# 8-bit variants: the paper's other two deployment points (Table "OpenVLA
# performance", INT8 weight-only row; Table "CILRS performance", W8A8 row;
# Sec. 5.4 "Implementation").  Same round-to-nearest uniform quantiser (Sec. 2.1)
# on a grid of 2^8 levels; the operation list is the 4-bit one with 15 -> 255
# and (-8, 7, divisor 7) -> (-128, 127, divisor 127).
# ----------------------------------------------------------------------------
def quantize_rtn_asym(w: np.ndarray, group_size: int, bits: int):
    """w fp32 [N][K] -> (codes u8 [N][K] in 0..L, scales f16 [N][K/G], zeros f16 [N][K/G]), L = 2^bits - 1.

    Per (row n, group g):
      lo = min(0, min w), hi = max(0, max w)
      s32 = (hi - lo) / L             (fp32)
      s16 = fp16(s32); 0 -> 1.0; inf -> error
      z   = clamp(rint(-lo / s16), 0, L)
      q_k = clamp(rint(w_k / s16) + z, 0, L)
    """
    if bits not in (4, 8):
        raise ValueError("bits must be 4 or 8")
    L = F32(2 ** bits - 1)
    w = np.ascontiguousarray(w, dtype=F32)
    N, K = w.shape
    G = int(group_size)
    if G <= 0 or K % G != 0:
        raise ValueError("group_size must divide K")
    ng = K // G
    wg = w.reshape(N, ng, G)
    lo = np.minimum(F32(0), wg.min(axis=2)).astype(F32)
    hi = np.maximum(F32(0), wg.max(axis=2)).astype(F32)
    r = (hi - lo).astype(F32)
    s32 = (r / L).astype(F32)
    with np.errstate(over="ignore"):
        s16 = s32.astype(np.float16)
    if np.isinf(s16).any():
        raise OverflowError("scale does not fit fp16")
    s16 = np.where(s16 == np.float16(0), np.float16(1.0), s16).astype(np.float16)
    s = s16.astype(F32)
    z = np.clip(np.rint((-lo / s).astype(F32)), F32(0), L).astype(F32)
    u = (np.rint((wg / s[:, :, None]).astype(F32)) + z[:, :, None]).astype(F32)
    q = np.clip(u, F32(0), L)
    return q.astype(np.uint8).reshape(N, K), s16, z.astype(np.uint8).astype(np.float16)


def quantize_rtn_w8_asym(w: np.ndarray, group_size: int):
    return quantize_rtn_asym(w, group_size, 8)


def quantize_sym(v: np.ndarray, bits: int, group_size: int | None = None, static_scale: float | None = None):
    """v fp32 [R][K] -> (codes int8 [R][K] in -2^(b-1) .. 2^(b-1)-1, fp32 scales [R][K/G]).

    Per (row, group): a = max|v|; s = a / (2^(b-1) - 1) (fp32); a == 0 -> s = 1; with ``static_scale`` every group
    uses that value.  q = clamp(rint(v / s), -2^(b-1), 2^(b-1) - 1).
    """
    if bits not in (4, 8):
        raise ValueError("bits must be 4 or 8")
    qmax = F32(2 ** (bits - 1) - 1)
    qmin = F32(-(2 ** (bits - 1)))
    v = np.ascontiguousarray(v, dtype=F32)
    R, K = v.shape
    G = K if group_size is None else int(group_size)
    if G <= 0 or K % G != 0:
        raise ValueError("group_size must divide K")
    ng = K // G
    vg = v.reshape(R, ng, G)
    if static_scale is not None:
        s = np.full((R, ng), F32(static_scale), dtype=F32)
    else:
        a = np.abs(vg).max(axis=2).astype(F32)
        s = (a / qmax).astype(F32)
        s = np.where(a == F32(0), F32(1.0), s).astype(F32)
    q = np.clip(np.rint((vg / s[:, :, None]).astype(F32)), qmin, qmax)
    return q.astype(np.int8).reshape(R, K), s


def quantize_sym8(v: np.ndarray, group_size: int | None = None, static_scale: float | None = None):
    return quantize_sym(v, 8, group_size, static_scale)


def dequant_asym(codes, scales, zeros, group_size: int) -> np.ndarray:
    """W_hat[n][k] = (q - z) * s in fp64, for codes of any width."""
    return dequant_w4_asym(codes, scales, zeros, group_size)


def linear_w8a16(x_bf16_bits, codes, scales, zeros, group_size: int) -> np.ndarray:
    """y[m][n] = sum_k x[m][k] * (q[n][k] - z[n][k/G]) * s[n][k/G] with 8-bit codes, fp64 throughout."""
    x = bf16_to_f32(x_bf16_bits).astype(np.float64)
    w_hat = dequant_asym(codes, scales, zeros, group_size)
    return np.matmul(x, w_hat.T)


def linear_w8a8(qx, sx, qw, sw):
    """acc[m][n] = sum_k qx[m][k]*qw[n][k] (int64, |acc| <= 2^14 K); y = acc * sx[m] * sw[n] (fp64)."""
    return linear_w4a4(qx, sx, qw, sw)


# ----------------------------------------------------------------------------
# W4A4 linear whose output is quantised again for the next layer (tensor-wise static activation scale, the paper's
# W4A4 setting: App. A.1.2 uses one learned step size per activation tensor).  The next layer's quantiser is applied to
# the fp32 output of the rescale, before any rounding to bf16:
#   acc = sum_k qx qw                     (integer, exact)
#   y32 = fl32(fl32(acc) * fl32(sx[m] * sw[n]))          two fp32 multiplications
#   y32 = max(y32, 0)                     when relu is set
#   q   = clamp(rint(y32 / out_scale), -8, 7)            fp32 division, ties to even
# ----------------------------------------------------------------------------
def linear_w4a4_requant(qx, sx, qw, sw, out_scale: float, relu: bool):
    acc, _ = linear_w4a4(qx, sx, qw, sw)
    if np.abs(acc).max() >= 2 ** 24:
        raise OverflowError("accumulator is not exact in fp32")
    scale = (np.asarray(sx, dtype=F32).reshape(-1, 1) * np.asarray(sw, dtype=F32).reshape(1, -1)).astype(F32)
    y32 = (acc.astype(F32) * scale).astype(F32)
    if relu:
        y32 = np.maximum(y32, F32(0))
    q = np.clip(np.rint((y32 / F32(out_scale)).astype(F32)), F32(-8), F32(7))
    return q.astype(np.int8)
