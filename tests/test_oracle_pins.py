"""Pins of the CPU oracle to things other than itself.

The paper (Sec. 2.1) names round-to-nearest uniform quantisation and prints no
numbers, so the oracle is pinned by: hand-worked fixtures (tests/golden),
closed-form error bounds, invariants, reductions to library routines
(numpy.matmul in fp64 / int64), brute force, and agreement of two independent
writings (NumPy and plain C).  Each test names the mistake it would catch.
"""
import json
import os

import numpy as np
import pytest

from oracle import c_oracle, np_oracle
from paper_2412_01034_b200 import workloads as wl

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")))
IMPLS = [pytest.param(np_oracle, id="numpy"), pytest.param(c_oracle, id="c")]


def bf16_bits(a):
    return wl.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


# --------------------------------------------------------------------------
# hand cases
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("case", ["asym_2x2", "asym_4x8_g8", "asym_4x8_g4"])
def test_hand_cases_asym(impl, case):
    c = GOLD[case]
    w = np.array(c["w"], dtype=np.float32)
    G = c["group"]
    codes, scales, zeros = impl.quantize_rtn_w4_asym(w, G)
    assert codes.dtype == np.uint8
    np.testing.assert_array_equal(codes, np.array(c["codes"], dtype=np.uint8))
    np.testing.assert_array_equal(scales.astype(np.float64), np.array(c["scales"]))
    np.testing.assert_array_equal(zeros.astype(np.float64), np.array(c["zeros"], dtype=np.float64))
    if "scale_bits" in c:
        bits = np.array([[int(b, 16) for b in row] for row in c["scale_bits"]], dtype=np.uint16)
        np.testing.assert_array_equal(np.ascontiguousarray(scales).view(np.uint16), bits)
    w_hat = np_oracle.dequant_w4_asym(codes, scales, zeros, G)
    np.testing.assert_array_equal(w_hat, np.array(c["w_hat"], dtype=np.float64))
    x = np.array(c["x"] if "x" in c else GOLD["x_rows_8"], dtype=np.float32)
    y = impl.linear_w4a16(bf16_bits(x), codes, scales, zeros, G)
    # all hand products are exactly representable in fp64 and every partial sum is too
    np.testing.assert_array_equal(y, np.array(c["y"], dtype=np.float64))


@pytest.mark.parametrize("impl", IMPLS)
def test_hand_case_sym(impl):
    c = GOLD["sym_row"]
    q, s = impl.quantize_sym4(np.array(c["v"], dtype=np.float32))
    np.testing.assert_array_equal(q, np.array(c["codes"], dtype=np.int8))
    np.testing.assert_array_equal(np.asarray(s, dtype=np.float64).reshape(-1), np.array(c["scale"]))
    q2, s2 = impl.quantize_sym4(np.array(c["v_static"], dtype=np.float32), static_scale=c["static_scale"])
    np.testing.assert_array_equal(q2, np.array(c["codes_static"], dtype=np.int8))
    assert float(np.asarray(s2).reshape(-1)[0]) == c["static_scale"]


@pytest.mark.parametrize("impl", IMPLS)
def test_hand_case_pack(impl):
    c = GOLD["pack_words"]
    u = impl.pack_w4(np.array(c["unsigned_codes"], dtype=np.uint8))
    assert int(u[0, 0]) == int(c["unsigned_word"][0], 16)
    s = impl.pack_w4(np.array(c["signed_codes"], dtype=np.int8))
    assert int(s[0, 0]) == int(c["signed_word"][0], 16)
    np.testing.assert_array_equal(impl.unpack_w4(s, signed=True), np.array(c["signed_codes"], dtype=np.int8))
    np.testing.assert_array_equal(impl.unpack_w4(u), np.array(c["unsigned_codes"], dtype=np.uint8))


@pytest.mark.parametrize("impl", IMPLS)
def test_hand_case_w4a4(impl):
    c = GOLD["w4a4_small"]
    acc, y = impl.linear_w4a4(np.array(c["qx"], np.int8), np.array(c["sx"], np.float32),
                              np.array(c["qw"], np.int8), np.array(c["sw"], np.float32))
    np.testing.assert_array_equal(acc, np.array(c["acc"], dtype=np.int64))
    np.testing.assert_array_equal(y, np.array(c["y"], dtype=np.float64))


# --------------------------------------------------------------------------
# closed forms and invariants of the asymmetric quantiser
# --------------------------------------------------------------------------
def _weights(seed, N=64, K=1024, sigma=0.02):
    return wl.normal_weights(100, seed, N, K, sigma)


@pytest.mark.parametrize("impl", IMPLS)
def test_asym_ranges_and_error_bound(impl):
    """codes in [0,15]; integer zero in [0,15]; |w_hat - w| <= s/2 wherever the unclamped level is
    inside the grid; the only clamp that can occur is level 16 -> 15 (scale rounded down to fp16),
    with error <= s*(0.5 + 15*2^-11).  Catches: wrong divisor, zero point sign, missing clamp,
    scale not rounded before use."""
    G = 128
    w = _weights(1, 256, 1024)
    codes, scales, zeros = impl.quantize_rtn_w4_asym(w, G)
    assert codes.min() >= 0 and codes.max() <= 15
    z = zeros.astype(np.float64)
    assert np.all(z == np.rint(z)) and z.min() >= 0 and z.max() <= 15
    s = np.repeat(scales.astype(np.float64), G, axis=1)
    w_hat = np_oracle.dequant_w4_asym(codes, scales, zeros, G)
    err = np.abs(w_hat - w.astype(np.float64))
    u = np_oracle.unclamped_levels_asym(w, G).astype(np.float64)
    assert u.min() >= 0 and u.max() <= 16
    inside = u <= 15
    assert np.all(err[inside] <= 0.5 * s[inside] * (1 + 2.0 ** -20))
    assert np.all(err[~inside] <= s[~inside] * (0.5 + 15 * 2.0 ** -11))
    groups_with_clamp = (~inside).reshape(w.shape[0], -1, G).any(axis=2).mean()
    assert groups_with_clamp < 0.01


@pytest.mark.parametrize("impl", IMPLS)
def test_asym_extremes_and_zero(impl):
    """q(lo) == 0, q(hi) in {14, 15}, and an exact 0.0 weight dequantises to exactly 0."""
    G = 128
    w = _weights(2, 128, 1024)
    w[:, ::G] = 0.0  # plant an exact zero in every group
    codes, scales, zeros = impl.quantize_rtn_w4_asym(w, G)
    wg = w.reshape(128, -1, G)
    cg = codes.reshape(128, -1, G)
    imin = wg.argmin(axis=2)
    imax = wg.argmax(axis=2)
    cmin = np.take_along_axis(cg, imin[:, :, None], axis=2)[:, :, 0]
    cmax = np.take_along_axis(cg, imax[:, :, None], axis=2)[:, :, 0]
    assert np.all(cmin == 0)
    assert np.all((cmax == 15) | (cmax == 14))
    assert (cmax == 15).mean() > 0.5
    w_hat = np_oracle.dequant_w4_asym(codes, scales, zeros, G)
    assert np.all(w_hat[:, ::G] == 0.0)
    np.testing.assert_array_equal(cg[:, :, 0].astype(np.float64), zeros.astype(np.float64))


@pytest.mark.parametrize("impl", IMPLS)
def test_asym_grid_fixpoint(impl):
    """Weights built on a grid (q - z) * s with codes 0 and 15 present come back as (q, s, z)."""
    rng = np.random.default_rng(5)
    N, K, G = 32, 256, 32
    q = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    qg = q.reshape(N, K // G, G)
    qg[:, :, 0] = 0
    qg[:, :, 1] = 15
    z = rng.integers(0, 16, size=(N, K // G)).astype(np.float64)
    e = rng.integers(-12, 3, size=(N, K // G))
    s = 2.0 ** e
    w = ((qg.astype(np.float64) - z[:, :, None]) * s[:, :, None]).reshape(N, K).astype(np.float32)
    codes, scales, zeros = impl.quantize_rtn_w4_asym(w, G)
    np.testing.assert_array_equal(codes, q)
    np.testing.assert_array_equal(scales.astype(np.float64), s)
    np.testing.assert_array_equal(zeros.astype(np.float64), z)


@pytest.mark.parametrize("impl", IMPLS)
def test_asym_degenerate_groups(impl):
    """all-zero group -> (s=1, z=0, q=0); all-equal group -> a single code and w_hat close to c."""
    G = 16
    w = np.zeros((3, 32), dtype=np.float32)
    w[1, :16] = 0.37
    w[1, 16:] = -2.5
    w[2, :] = 1e-9  # scale underflows fp16 -> treated like a zero scale
    codes, scales, zeros = impl.quantize_rtn_w4_asym(w, G)
    assert np.all(codes[0] == 0) and np.all(scales[0] == 1.0) and np.all(zeros[0] == 0)
    assert len(set(codes[1, :16].tolist())) == 1 and len(set(codes[1, 16:].tolist())) == 1
    w_hat = np_oracle.dequant_w4_asym(codes, scales, zeros, G)
    assert np.all(np.abs(w_hat[1] - w[1]) <= 0.51 * np.repeat(scales[1].astype(np.float64), G))
    assert codes[1, 0] == 15 and zeros[1, 0] == 0
    assert codes[1, 16] == 0 and zeros[1, 1] == 15
    assert np.all(scales[2] == 1.0) and np.all(codes[2] == 0)


@pytest.mark.parametrize("impl", IMPLS)
def test_asym_scale_overflow_is_an_error(impl):
    w = np.zeros((1, 16), dtype=np.float32)
    w[0, 0] = 2.0e6  # (2e6)/15 > 65504
    with pytest.raises(OverflowError):
        impl.quantize_rtn_w4_asym(w, 16)


def test_asym_brute_force_nearest_level():
    """Brute force on small groups: the chosen code is the nearest grid level to w (among 0..15),
    up to the tie / fp16-rounding slack.  Catches an off-by-one zero point or a transposed sign."""
    w = _weights(3, 16, 256)
    G = 32
    codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, G)
    s = np.repeat(scales.astype(np.float64), G, axis=1)
    z = np.repeat(zeros.astype(np.float64), G, axis=1)
    levels = np.arange(16, dtype=np.float64)
    cand = (levels[None, None, :] - z[:, :, None]) * s[:, :, None]
    d = np.abs(cand - w.astype(np.float64)[:, :, None])
    best = d.min(axis=2)
    chosen = np.take_along_axis(d, codes.astype(np.int64)[:, :, None], axis=2)[:, :, 0]
    assert np.all(chosen <= best + 1e-6 * s)


# --------------------------------------------------------------------------
# symmetric quantiser
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
def test_sym_bounds(impl):
    """|v - q s| <= s/2, codes in [-7, 7] under dynamic absmax, the absmax element maps to +-7,
    an all-zero row gives s = 1 and q = 0.  Catches divisor 8 vs 7, missing abs, wrong rounding."""
    v = wl.normal_weights(101, 0, 64, 576, 1.0)
    v[5] = 0.0
    q, s = impl.quantize_sym4(v)
    s = np.asarray(s, dtype=np.float64).reshape(-1, 1)
    assert q.min() >= -7 and q.max() <= 7
    err = np.abs(v.astype(np.float64) - q.astype(np.float64) * s)
    assert np.all(err <= 0.5 * s * (1 + 2.0 ** -20))
    imax = np.abs(v).argmax(axis=1)
    top = np.abs(q[np.arange(64), imax])
    assert np.all(np.delete(top, 5) == 7)
    assert s[5, 0] == 1.0 and np.all(q[5] == 0)
    a = np.abs(v).max(axis=1).astype(np.float32)
    np.testing.assert_array_equal(np.delete(s.reshape(-1), 5),
                                  np.delete((a / np.float32(7)).astype(np.float64), 5))


@pytest.mark.parametrize("impl", IMPLS)
def test_sym_groups_and_f16_scale(impl):
    v = wl.normal_weights(101, 1, 8, 256, 0.05)
    q, s = impl.quantize_sym4(v, group_size=64, scale_f16=True)
    assert s.dtype == np.float16 and s.shape == (8, 4)
    sr = np.repeat(s.astype(np.float64), 64, axis=1)
    err = np.abs(v.astype(np.float64) - q.astype(np.float64) * sr)
    # the scale may have been rounded down by fp16: |v/s| <= 7*(1+2^-11) still rounds to 7
    assert q.min() >= -7 and q.max() <= 7
    assert np.all(err <= sr * (0.5 + 7 * 2.0 ** -11))


# --------------------------------------------------------------------------
# packing
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
def test_pack_bijection(impl):
    rng = np.random.default_rng(7)
    c = rng.integers(0, 16, size=(33, 264)).astype(np.uint8)
    p = impl.pack_w4(c)
    assert p.shape == (33, 33) and p.dtype == np.uint32
    np.testing.assert_array_equal(impl.unpack_w4(p), c)
    # bit position of one element, stated directly: element k -> word k//8, bits 4*(k%8)
    n, k = 17, 203
    assert (int(p[n, k // 8]) >> (4 * (k % 8))) & 0xF == int(c[n, k])
    sc = rng.integers(-8, 8, size=(5, 64)).astype(np.int8)
    np.testing.assert_array_equal(impl.unpack_w4(impl.pack_w4(sc), signed=True), sc)


def test_tile16_layout_is_a_documented_permutation():
    rng = np.random.default_rng(8)
    N, K = 48, 384
    p = rng.integers(0, 2 ** 32, size=(N, K // 8), dtype=np.uint64).astype(np.uint32)
    flat = np_oracle.to_layout(p, np_oracle.LAYOUT_TILE16)
    assert sorted(flat.tolist()) == sorted(p.reshape(-1).tolist())
    np.testing.assert_array_equal(np_oracle.from_layout(flat, N, K, np_oracle.LAYOUT_TILE16), p)
    np.testing.assert_array_equal(c_oracle.to_tile16(p), flat)
    # spot value from the written rule: word (n=21, i=37) of a K=384 matrix (3 column tiles):
    # tile index (21//16)*3 + 37//16 = 5; inside: (21%16)*16 + 37%16 = 85  ->  5*256 + 85
    assert flat[5 * 256 + 85] == p[21, 37]
    # and the first 16 words are row 0's first 16 words, then row 1's first 16 words
    np.testing.assert_array_equal(flat[:16], p[0, :16])
    np.testing.assert_array_equal(flat[16:32], p[1, :16])


def test_stream128_layout_follows_its_written_rule():
    rng = np.random.default_rng(13)
    N, K, G = 200, 384, 128      # two row tiles (the second one ragged), three column blocks
    codes = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    scales = (rng.random((N, K // G)) + 0.5).astype(np.float16)
    zeros = rng.integers(0, 16, size=(N, K // G)).astype(np.float16)
    buf = np_oracle.to_stream128(codes, scales, zeros, G)
    assert buf.size == 2 * 3 * 8704
    # element (n=150, k=300): row tile 1, block 2 -> unit 1*3+2 = 5; row 22; column 44 of the block ->
    # chunk 1, column 12 of the chunk -> word 1, 12 = 8*1 + 4 + 0 -> byte 0 of word 1, high nibble
    off = 5 * 8704 + (1 * 128 + 22) * 16 + 4 * 1 + 0
    assert buf[off] >> 4 == codes[150, 300]
    assert buf[off] & 0xF == codes[150, 296]       # column 40 = 32 + 8*1 + 0 -> same byte, low nibble
    m = 5 * 8704 + 8192 + 22 * 4
    assert buf[m:m + 2].view(np.float16)[0] == scales[150, 2]
    assert buf[m + 2:m + 4].view(np.float16)[0] == zeros[150, 2]
    # rows 200..255 of the second row tile are padding
    pad = buf[3 * 8704:4 * 8704]
    assert np.all(pad[:8192].reshape(4, 128, 16)[:, 72:, :] == 0) and np.all(pad[8192 + 72 * 4:] == 0)
    # every code appears exactly once: undo the rule for unit 0
    u0 = buf[:8192].reshape(4, 128, 4, 4)
    rec = np.zeros((128, 128), dtype=np.uint8)
    for j in range(4):
        for mm in range(4):
            for b in range(4):
                rec[:, 32 * j + 8 * mm + b] = u0[j, :, mm, b] & 0xF
                rec[:, 32 * j + 8 * mm + 4 + b] = u0[j, :, mm, b] >> 4
    np.testing.assert_array_equal(rec, codes[:128, :128])


# --------------------------------------------------------------------------
# linears
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
def test_w4a16_reduces_to_library_matmul(impl):
    """y == x @ W_hat^T with W_hat built elementwise; integer special case equals exact integer matmul.
    Catches transposed operands, group index errors, zero-point sign."""
    rng = np.random.default_rng(9)
    M, N, K, G = 5, 24, 256, 64
    codes = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    scales = (2.0 ** rng.integers(-8, 0, size=(N, K // G))).astype(np.float16)
    zeros = rng.integers(0, 16, size=(N, K // G)).astype(np.float16)
    xi = rng.integers(-4, 5, size=(M, K)).astype(np.float32)
    y = impl.linear_w4a16(bf16_bits(xi), codes, scales, zeros, G)
    # independent elementwise construction
    W = np.zeros((N, K))
    for n in range(N):
        for k in range(K):
            W[n, k] = (float(codes[n, k]) - float(zeros[n, k // G])) * float(scales[n, k // G])
    ref = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            ref[m, n] = sum(float(xi[m, k]) * W[n, k] for k in range(K))
    np.testing.assert_array_equal(y, ref)  # all terms are dyadic and small: exact in fp64
    ones = np.ones((N, K // G), dtype=np.float16)
    y_int = impl.linear_w4a16(bf16_bits(xi), codes, ones, 0 * ones, G)
    np.testing.assert_array_equal(y_int, (xi.astype(np.int64) @ codes.astype(np.int64).T).astype(np.float64))


@pytest.mark.parametrize("impl", IMPLS)
def test_w4a16_rows_are_independent_gemvs(impl):
    w = _weights(4, 32, 512)
    codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, 128)
    x = wl.normal_activations_bf16(102, 0, 4, 512)
    y = impl.linear_w4a16(x, codes, scales, zeros, 128)
    for m in range(4):
        ym = impl.linear_w4a16(x[m:m + 1], codes, scales, zeros, 128)
        np.testing.assert_array_equal(ym[0], y[m])
    # fp64 result is within a few ulp of the fp32-weight product up to quantisation error: sanity of scale
    y_fp = wl.bf16_bits_to_f32(x).astype(np.float64) @ w.astype(np.float64).T
    assert np.abs(y - y_fp).max() < 0.15 * np.abs(y_fp).max()


@pytest.mark.parametrize("impl", IMPLS)
def test_w4a4_reduces_to_integer_matmul(impl):
    rng = np.random.default_rng(11)
    M, N, K = 9, 7, 576
    qx = rng.integers(-8, 8, size=(M, K)).astype(np.int8)
    qw = rng.integers(-8, 8, size=(N, K)).astype(np.int8)
    qx[0] = -8
    qw[0] = -8
    sx = rng.random(M).astype(np.float32)
    sw = rng.random(N).astype(np.float32)
    acc, y = impl.linear_w4a4(qx, sx, qw, sw)
    ref = qx.astype(np.int64) @ qw.astype(np.int64).T
    np.testing.assert_array_equal(acc, ref)
    assert acc[0, 0] == 64 * K and np.abs(acc).max() <= 64 * K
    np.testing.assert_allclose(y, ref * sx.astype(np.float64)[:, None] * sw.astype(np.float64)[None, :], rtol=1e-15)


# --------------------------------------------------------------------------
# the two writings agree
# --------------------------------------------------------------------------
def test_numpy_and_c_oracles_agree():
    w = wl.normal_weights(103, 0, 96, 1024, 0.02, outlier_prob=0.001)
    a = np_oracle.quantize_rtn_w4_asym(w, 128)
    b = c_oracle.quantize_rtn_w4_asym(w, 128)
    for u, v in zip(a, b):
        np.testing.assert_array_equal(np.ascontiguousarray(u).view(np.uint8), np.ascontiguousarray(v).view(np.uint8))
    x = wl.normal_activations_bf16(103, 1, 3, 1024)
    ya = np_oracle.linear_w4a16(x, *a, 128)
    yb = c_oracle.linear_w4a16(x, *b, 128)
    np.testing.assert_allclose(ya, yb, rtol=0, atol=1e-12 * np.abs(ya).max())
    xs, wsym = wl.conv_stage(3, batch=1)
    qa, sa = np_oracle.quantize_sym4(wl.bf16_bits_to_f32(xs))
    qb, sb = c_oracle.quantize_sym4(wl.bf16_bits_to_f32(xs))
    np.testing.assert_array_equal(qa, qb)
    np.testing.assert_array_equal(np.asarray(sa).reshape(-1), np.asarray(sb).reshape(-1))
    qwa, swa = np_oracle.quantize_sym4(wsym)
    qwb, swb = c_oracle.quantize_sym4(wsym)
    np.testing.assert_array_equal(qwa, qwb)
    acc_a, y_a = np_oracle.linear_w4a4(qa, sa, qwa, swa)
    acc_b, y_b = c_oracle.linear_w4a4(qb, sb, qwb, swb)
    np.testing.assert_array_equal(acc_a, acc_b)
    np.testing.assert_allclose(y_a, y_b, rtol=1e-14)


# --------------------------------------------------------------------------
# input generators (not part of the method, but both sides rely on them)
# --------------------------------------------------------------------------
def test_bf16_rounding_of_inputs():
    x = np.array([1.0, 1.00390625, 1.01171875, -3.140625, 0.0, 1e-40], dtype=np.float32)
    # 1.00390625 = 1 + 2^-8 is a tie between 1.0 and 1.0078125 -> even (1.0);
    # 1.01171875 = 1 + 3*2^-8 is a tie between 1.0078125 and 1.015625 -> even (1.015625)
    b = wl.f32_to_bf16_bits(x)
    back = np_oracle.bf16_to_f32(b)
    np.testing.assert_array_equal(back[:5], np.array([1.0, 1.0, 1.015625, -3.140625, 0.0], dtype=np.float32))
    np.testing.assert_array_equal(wl.bf16_bits_to_f32(b), back)


def test_im2col_shapes_and_border():
    x, w = wl.conv_stage(3, batch=2)
    M, K, N = wl.conv_gemm_shape(3, batch=2)
    assert x.shape == (M, K) == (2 * 3 * 7, 4608) and w.shape == (N, K) == (512, 4608)
    # top-left output pixel: the kh=0 and kw=0 taps fall in the zero padding
    assert np.all(x[0, :3 * 512] == 0) and np.all(x[0, 3 * 512:4 * 512] == 0)
    # centre tap of pixel (h=1, w=2) equals the feature map value itself, which is >= 0 (ReLU)
    vals = wl.bf16_bits_to_f32(x)
    assert vals.min() >= 0.0
    assert wl.cfg1_bytes_per_step() == 3440377856
