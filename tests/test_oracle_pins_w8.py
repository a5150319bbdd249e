"""Pins of the 8-bit oracle functions (INT8 weight-only and W8A8, the paper's other two deployment points:
Table "OpenVLA performance" INT8 row, Table "CILRS performance" W8A8 row, Sec. 5.4) to things other than
themselves: hand-worked cases, closed forms, invariants, brute force and library reductions.  No GPU needed.

The hand cases are worked out in the comments from the operation list alone (fp32, one IEEE operation per step,
ties to even); none of their expected values was produced by running an implementation.
"""
import numpy as np
import pytest

from oracle import c_oracle, np_oracle
from paper_2412_01034_b200 import workloads as wl

IMPLS = [np_oracle, c_oracle]


def bf16_bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


# --------------------------------------------------------------------------
# hand cases of the asymmetric 8-bit quantiser
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
def test_asym8_exact_grid_hand_case(impl):
    """One group of 8 on the grid s = 2^-8, z = 100: w_k = (q_k - 100) / 256.
    lo = -100/256, hi = 155/256, hi - lo = 255/256, s32 = (255/256)/255 = 2^-8 exactly (the quotient is
    representable, so the IEEE division returns it), fp16(2^-8) = 2^-8 = 0x1C00.  z = rint(100) = 100.
    Every w_k / s is the integer q_k - 100, so the codes come back as chosen.  Catches: a divisor of 256 or 254,
    a zero point of the wrong sign, clamping to 15 or 127."""
    q = np.array([[0, 255, 100, 37, 200, 101, 99, 1]], dtype=np.int64)
    w = ((q - 100) / 256.0).astype(np.float32)
    codes, scales, zeros = impl.quantize_rtn_w8_asym(w, 8)
    np.testing.assert_array_equal(codes, q.astype(np.uint8))
    assert np.ascontiguousarray(scales).view(np.uint16).tolist() == [[0x1C00]]
    assert zeros.astype(np.float64).tolist() == [[100.0]]
    # dequantised values are the inputs again, exactly
    np.testing.assert_array_equal(np_oracle.dequant_asym(codes, scales, zeros, 8), w.astype(np.float64))


@pytest.mark.parametrize("impl", IMPLS)
def test_asym8_ties_go_to_even(impl):
    """Same grid; two more weights sit half-way between levels: (2.5 - 100 + 100) -> w = 2.5/256 and 3.5/256 with
    z = 100 give rint(2.5) + 100 = 102 and rint(3.5) + 100 = 104 (ties to even), not 103 / 104 (half away) or
    102 / 103 (truncation)."""
    w = np.array([[-100 / 256.0, 155 / 256.0, 2.5 / 256.0, 3.5 / 256.0, 0.0, 0.0, 0.0, 0.0]], dtype=np.float32)
    codes, _, zeros = impl.quantize_rtn_w8_asym(w, 8)
    assert zeros.astype(np.float64).tolist() == [[100.0]]
    assert codes.tolist() == [[0, 255, 102, 104, 100, 100, 100, 100]]


@pytest.mark.parametrize("impl", IMPLS)
def test_asym8_scale_is_rounded_to_fp16_before_use(impl):
    """Group {0, 1.0, 0.7f, ...}: lo = 0, hi = 1, s32 = 1/255 = 0.00392156886...  In fp16 the neighbours of that
    value are 2^-8 (1 + 4/1024) = 0.00392150878906 (0x1C04) and 2^-8 (1 + 5/1024) = 0.00392532348633; the first
    is nearer, so s16 = 0x1C04.  0.7f is 0.699999988079071; divided by s32 it is 178.499997 -> 178, divided by
    s16 it is 178.5027 -> 179.  The stored code must be 179: the scale is rounded first.  z = rint(0) = 0,
    q(1.0) = rint(255.0039) = 255."""
    w = np.array([[0.0, 1.0, 0.7, 0.0, 0.0, 0.0, 0.0, 0.0]], dtype=np.float32)
    codes, scales, zeros = impl.quantize_rtn_w8_asym(w, 8)
    assert np.ascontiguousarray(scales).view(np.uint16).tolist() == [[0x1C04]]
    assert zeros.astype(np.float64).tolist() == [[0.0]]
    assert codes.tolist() == [[0, 255, 179, 0, 0, 0, 0, 0]]


@pytest.mark.parametrize("impl", IMPLS)
def test_asym8_degenerate_groups(impl):
    """All-zero group -> (s, z, q) = (1, 0, 0); an all-equal negative group c: lo = c, hi = 0, the single code is
    q(c) = rint(c / s) + rint(-c / s) = 0 and z = 255 (c sits at the bottom of the grid); one-signed positive
    group: z = 0."""
    w = np.zeros((3, 8), dtype=np.float32)
    w[1] = -0.25
    w[2] = [0.5, 0.25, 0.125, 1.0, 0.75, 0.0625, 0.3, 0.9]
    codes, scales, zeros = impl.quantize_rtn_w8_asym(w, 8)
    assert codes[0].tolist() == [0] * 8 and float(scales[0, 0]) == 1.0 and float(zeros[0, 0]) == 0.0
    assert codes[1].tolist() == [0] * 8 and float(zeros[1, 0]) == 255.0
    assert float(zeros[2, 0]) == 0.0 and codes[2].max() == 255


# --------------------------------------------------------------------------
# closed forms and invariants
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
def test_asym8_ranges_and_error_bound(impl):
    """codes and zero points in [0, 255]; |w_hat - w| <= s/2 wherever the unclamped level rint(w/s) + z is on the
    grid.  The only clamp that can occur is level 256 -> 255: the span over the fp16-rounded scale is at most
    255 (1 + 2^-11), the two roundings add at most 1, so the unclamped level is at most 256, and its error is at
    most s (1/2 + 255 * 2^-11)."""
    G = 128
    w = wl.normal_weights(110, 1, 128, 1024, 0.02, outlier_prob=0.001)
    codes, scales, zeros = impl.quantize_rtn_w8_asym(w, G)
    z = zeros.astype(np.float64)
    assert np.all(z == np.rint(z)) and z.min() >= 0 and z.max() <= 255
    s = np.repeat(scales.astype(np.float64), G, axis=1)
    zz = np.repeat(z, G, axis=1)
    w_hat = np_oracle.dequant_asym(codes, scales, zeros, G)
    err = np.abs(w_hat - w.astype(np.float64))
    u = np.rint((w / s.astype(np.float32)).astype(np.float32)).astype(np.float64) + zz
    assert u.min() >= 0 and u.max() <= 256
    inside = u <= 255
    # (the fp32 quotient w / s, at most 256, is off by at most 2^-24 of itself = 2^-16 levels)
    assert np.all(err[inside] <= 0.5 * s[inside] * (1 + 2.0 ** -14))
    assert np.all(err[~inside] <= s[~inside] * (0.5 + 255 * 2.0 ** -11))
    # the 8-bit grid is 17 times finer than the 4-bit one on the same data
    c4 = impl.quantize_rtn_w4_asym(w, G)
    err4 = np.abs(np_oracle.dequant_w4_asym(*c4, G) - w.astype(np.float64))
    assert 14.0 < err4.mean() / err.mean() < 20.0


@pytest.mark.parametrize("impl", IMPLS)
def test_asym8_extremes_zero_and_fixpoint(impl):
    """q(lo) = 0 exactly; q(hi) is 254 or 255 (a clamped 256 included); a weight that is exactly 0 dequantises
    to exactly 0; quantising the dequantised weights of a group that uses codes 0 and 255 returns the same
    triple (the grid is a fix-point)."""
    G = 128
    w = wl.normal_weights(110, 2, 64, 1024, 0.02)
    w[:, ::G] = 0.0
    codes, scales, zeros = impl.quantize_rtn_w8_asym(w, G)
    wg, cg = w.reshape(64, -1, G), codes.reshape(64, -1, G)
    cmin = np.take_along_axis(cg, wg.argmin(axis=2)[:, :, None], axis=2)[:, :, 0]
    cmax = np.take_along_axis(cg, wg.argmax(axis=2)[:, :, None], axis=2)[:, :, 0]
    assert np.all(cmin == 0) and np.all(cmax >= 254)
    w_hat = np_oracle.dequant_asym(codes, scales, zeros, G)
    assert np.all(w_hat[:, ::G] == 0.0)
    both = (cg.min(axis=2) == 0) & (cg.max(axis=2) == 255)
    again = impl.quantize_rtn_w8_asym(w_hat.astype(np.float32), G)
    np.testing.assert_array_equal(again[0].reshape(64, -1, G)[both], cg[both])
    np.testing.assert_array_equal(again[1][both], scales[both])
    np.testing.assert_array_equal(again[2][both], zeros[both])


def test_asym8_code_is_the_nearest_level_brute_force():
    """For every weight the stored code is a nearest grid point among all 256 (brute force over the levels)."""
    G = 64
    w = wl.normal_weights(110, 3, 8, 256, 0.05)
    codes, scales, zeros = np_oracle.quantize_rtn_w8_asym(w, G)
    s = np.repeat(scales.astype(np.float64), G, axis=1)[:, :, None]
    z = np.repeat(zeros.astype(np.float64), G, axis=1)[:, :, None]
    levels = (np.arange(256, dtype=np.float64)[None, None, :] - z) * s
    dist = np.abs(levels - w.astype(np.float64)[:, :, None])
    chosen = np.take_along_axis(dist, codes.astype(np.int64)[:, :, None], axis=2)[:, :, 0]
    assert np.all(chosen <= dist.min(axis=2) * (1 + 1e-6) + 1e-12)


def test_generic_quantiser_with_four_bits_is_the_four_bit_quantiser():
    """The generic routine at bits = 4 returns what the separately written 4-bit routines return (asymmetric and
    symmetric), in both writings."""
    w = wl.normal_weights(110, 4, 32, 512, 0.02, outlier_prob=0.002)
    for impl in IMPLS:
        a, b = impl.quantize_rtn_asym(w, 128, 4), impl.quantize_rtn_w4_asym(w, 128)
        for u, v in zip(a, b):
            np.testing.assert_array_equal(np.ascontiguousarray(u).view(np.uint8), np.ascontiguousarray(v).view(np.uint8))
        qs, ss = impl.quantize_sym(w, 4)
        q4, s4 = impl.quantize_sym4(w)
        np.testing.assert_array_equal(qs, q4)
        np.testing.assert_array_equal(np.asarray(ss).reshape(-1), np.asarray(s4).reshape(-1))


def test_two_writings_agree_bit_for_bit():
    w = wl.normal_weights(110, 5, 48, 768, 0.02, outlier_prob=0.001)
    w[0, :128] = 0
    a, b = np_oracle.quantize_rtn_w8_asym(w, 128), c_oracle.quantize_rtn_w8_asym(w, 128)
    for u, v in zip(a, b):
        np.testing.assert_array_equal(np.ascontiguousarray(u).view(np.uint8), np.ascontiguousarray(v).view(np.uint8))
    x = wl.bf16_bits_to_f32(wl.normal_activations_bf16(110, 6, 20, 768))
    qa, sa = np_oracle.quantize_sym8(x)
    qb, sb = c_oracle.quantize_sym8(x)
    np.testing.assert_array_equal(qa, qb)
    np.testing.assert_array_equal(sa.view(np.uint32), sb.view(np.uint32))


# --------------------------------------------------------------------------
# symmetric int8
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
def test_sym8_hand_row(impl):
    """Row with absmax 127/64: s = (127/64)/127 = 2^-6 exactly, so q = rint(64 v): 64 * 1.984375 = 127,
    64 * -0.5 = -32, 64 * 0.0390625 = 2.5 -> 2 (tie to even), 64 * 0.0546875 = 3.5 -> 4, 64 * -1.984375 = -127.
    With the static scale 2^-7, 128 * 1.984375 = 254 -> clamp 127 and 128 * -1.984375 = -254 -> clamp -128."""
    v = np.array([[127 / 64.0, -0.5, 0.0390625, 0.0546875, -127 / 64.0, 0.0, 0.015625, -0.015625]], dtype=np.float32)
    q, s = impl.quantize_sym8(v)
    assert np.asarray(s, dtype=np.float64).reshape(-1).tolist() == [2.0 ** -6]
    assert q.tolist() == [[127, -32, 2, 4, -127, 0, 1, -1]]
    q2, s2 = impl.quantize_sym8(v, static_scale=2.0 ** -7)
    assert q2.tolist() == [[127, -64, 5, 7, -128, 0, 2, -2]]
    assert float(np.asarray(s2).reshape(-1)[0]) == 2.0 ** -7


@pytest.mark.parametrize("impl", IMPLS)
def test_sym8_invariants(impl):
    """|v - q s| <= s/2 everywhere (no clamp can trigger with a dynamic scale), the row's largest magnitude maps
    to +-127, an all-zero row gives scale 1 and codes 0, -128 never appears with a dynamic scale."""
    v = wl.bf16_bits_to_f32(wl.normal_activations_bf16(110, 7, 40, 1152))
    v[3] = 0.0
    q, s = impl.quantize_sym8(v)
    s = np.asarray(s, dtype=np.float64).reshape(-1, 1)
    # (the fp32 quotient v / s, at most 127, is off by at most 2^-24 of itself < 2^-17 levels)
    assert np.all(np.abs(v.astype(np.float64) - q.astype(np.float64) * s) <= 0.5 * s * (1 + 2.0 ** -14))
    assert q.min() >= -127 and q.max() <= 127
    big = np.abs(v).argmax(axis=1)
    got = np.abs(q[np.arange(40), big])
    assert np.all(got[np.arange(40) != 3] == 127) and np.all(q[3] == 0) and s[3, 0] == 1.0


# --------------------------------------------------------------------------
# the two linears
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
def test_linear_w8a16_hand_and_library(impl):
    """Hand product: two output features on the grid s = 1/256, z = 100 resp. s = 1/128, z = 0, x = (1, -2, 0.5, 4):
    y0 = ((0-100) - 2 (255-100) + 0.5 (100-100) + 4 (102-100)) / 256 = (-100 - 310 + 0 + 8) / 256 = -402/256,
    y1 = (1*10 - 2*20 + 0.5*30 + 4*255) / 128 = (10 - 40 + 15 + 1020) / 128 = 1005/128.
    Then: equals numpy.matmul with the elementwise dequantised matrix, and a triple loop on a small case."""
    codes = np.array([[0, 255, 100, 102], [10, 20, 30, 255]], dtype=np.uint8)
    scales = np.array([[1 / 256.0], [1 / 128.0]], dtype=np.float16)
    zeros = np.array([[100.0], [0.0]], dtype=np.float16)
    x = bf16_bits([[1.0, -2.0, 0.5, 4.0]])
    y = impl.linear_w8a16(x, codes, scales, zeros, 4)
    np.testing.assert_array_equal(y, np.array([[-402 / 256.0, 1005 / 128.0]]))
    w = wl.normal_weights(110, 8, 24, 256, 0.02)
    q = np_oracle.quantize_rtn_w8_asym(w, 64)
    xb = wl.normal_activations_bf16(110, 9, 3, 256)
    got = impl.linear_w8a16(xb, *q, 64)
    xf = wl.bf16_bits_to_f32(xb).astype(np.float64)
    want = np.zeros((3, 24))
    for m in range(3):
        for n in range(24):
            for k in range(256):
                want[m, n] += xf[m, k] * ((float(q[0][n, k]) - float(q[2][n, k // 64])) * float(q[1][n, k // 64]))
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("impl", IMPLS)
def test_linear_w8a8_exact_integers(impl):
    """acc is the exact integer matmul; the all-(-128) row against an all-(-128) row gives 2^14 K, against an
    all-127 row -128 * 127 K; y = acc * sx * sw with hand values."""
    rng = np.random.default_rng(3)
    qx = rng.integers(-128, 128, size=(5, 96)).astype(np.int8)
    qw = rng.integers(-128, 128, size=(7, 96)).astype(np.int8)
    qx[0] = -128
    qw[0] = -128
    qw[1] = 127
    sx = np.array([0.5, 0.25, 1.0, 2.0, 0.125], dtype=np.float32)
    sw = np.array([1.0, 0.5, 0.25, 2.0, 4.0, 0.125, 1.0], dtype=np.float32)
    acc, y = impl.linear_w8a8(qx, sx, qw, sw)
    np.testing.assert_array_equal(acc, qx.astype(np.int64) @ qw.astype(np.int64).T)
    assert acc[0, 0] == 16384 * 96 and acc[0, 1] == -128 * 127 * 96
    assert y[0, 0] == 16384 * 96 * 0.5 and y[0, 1] == -128 * 127 * 96 * 0.5 * 0.5
    assert np.abs(acc).max() <= 16384 * 96


# --------------------------------------------------------------------------
# W4A4 linear with the next layer's static-scale quantiser applied to its output
# --------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
def test_w4a4_requant_hand_case(impl):
    """qx = (1, -2, 3, 0), sx = 0.5; three weight rows with sw = (0.25, 1, 2):
    acc = (1*4 - 2*1 + 3*2, 1*7 - 2*7 + 3*7, -1 - 2*(-8) + 3*(-8)) = (8, 14, -9);
    y = acc * sx * sw = (8 * 0.125, 14 * 0.5, -9 * 1.0) = (1, 7, -9); with out_scale = 0.5: y / 0.5 = (2, 14, -18)
    -> codes (2, 7 (clamped), -8 (clamped)); with relu the last becomes 0.  A tie: acc 5 with scale 0.25 * 0.5 ... see
    second row: y = 1.25 / 0.5 = 2.5 -> 2 (ties to even)."""
    qx = np.array([[1, -2, 3, 0], [5, 0, 0, 0]], dtype=np.int8)
    qw = np.array([[4, 1, 2, 0], [7, 7, 7, 0], [-1, -8, -8, 0]], dtype=np.int8)
    sx = np.array([0.5, 0.5], dtype=np.float32)
    sw = np.array([0.25, 1.0, 2.0], dtype=np.float32)
    # row 1: acc = (20, 35, -5); y = (2.5, 17.5, -5); / 0.5 = (5, 35, -10) -> (5, 7, -8)
    q = impl.linear_w4a4_requant(qx, sx, qw, sw, 0.5, False)
    assert q.tolist() == [[2, 7, -8], [5, 7, -8]]
    q = impl.linear_w4a4_requant(qx, sx, qw, sw, 0.5, True)
    assert q.tolist() == [[2, 7, 0], [5, 7, 0]]
    # ties to even: acc = 5, scale 0.5 * 0.25 -> y = 0.625; out_scale 0.25 -> 2.5 -> 2
    q = impl.linear_w4a4_requant(np.array([[5, 0, 0, 0]], np.int8), np.array([0.5], np.float32),
                                 np.array([[1, 0, 0, 0]], np.int8), np.array([0.25], np.float32), 0.25, False)
    assert q.tolist() == [[2]]


def test_w4a4_requant_is_the_static_quantiser_of_the_fp32_output():
    """Reduces to the pinned pieces: integer matmul, two fp32 multiplications, then quantize_sym4 with a static scale;
    the two writings agree bit for bit."""
    rng = np.random.default_rng(9)
    qx = rng.integers(-8, 8, size=(37, 96)).astype(np.int8)
    qw = rng.integers(-8, 8, size=(40, 96)).astype(np.int8)
    sx = (rng.random(37) * 0.1 + 0.01).astype(np.float32)
    sw = (rng.random(40) * 0.1 + 0.01).astype(np.float32)
    acc = qx.astype(np.int64) @ qw.astype(np.int64).T
    y32 = acc.astype(np.float32) * (sx[:, None] * sw[None, :]).astype(np.float32)
    for relu in (False, True):
        want, _ = np_oracle.quantize_sym4(np.maximum(y32, 0) if relu else y32, static_scale=0.05)
        a = np_oracle.linear_w4a4_requant(qx, sx, qw, sw, 0.05, relu)
        b = c_oracle.linear_w4a4_requant(qx, sx, qw, sw, 0.05, relu)
        np.testing.assert_array_equal(a, want)
        np.testing.assert_array_equal(b, want)
        assert a.min() >= -8 and a.max() <= 7
