"""Pins of the oracle's gated-MLP linear (`np_oracle.silu`, `np_oracle.linear_w4a16_swiglu`) against what the
mathematics fixes: closed forms and identities of silu, a hand-computed case, and the reduction to two plain
(already pinned) linears.  A dropped factor, a swapped gate / up, a wrong sign in the exponent or an off-by-one in the
row interleave fails one of them.
"""
import math

import numpy as np

from oracle import np_oracle
from paper_2412_01034_b200 import workloads as wl


def test_silu_closed_forms():
    s = np_oracle.silu
    assert s(np.array([0.0]))[0] == 0.0
    # silu(x) - silu(-x) = x  (sigmoid(x) + sigmoid(-x) = 1)
    x = np.linspace(-30, 30, 241)
    np.testing.assert_allclose(s(x) - s(-x), x, rtol=0, atol=1e-12)
    # silu(ln 3) = ln 3 * 3/4, silu(-ln 3) = -ln 3 / 4
    l3 = math.log(3.0)
    np.testing.assert_allclose(s(np.array([l3, -l3])), [0.75 * l3, -0.25 * l3], rtol=1e-15)
    # limits: x for large x, x e^x for very negative x; nothing overflows on the way (e^-800 flushing to 0 is meant)
    with np.errstate(over="raise", invalid="raise", divide="raise"):
        big = s(np.array([800.0, -800.0, 40.0]))
    assert big[0] == 800.0 and big[1] == 0.0 and abs(big[2] - 40.0) < 1e-15
    np.testing.assert_allclose(s(np.array([-20.0]))[0], -20.0 * math.exp(-20.0), rtol=1e-8)
    # the minimum of silu is at the root of 1 + e^-x (1 + x) ... = 0: x = -1.2784645..., value -0.2784645...
    grid = np.linspace(-3, 0, 300001)
    v = s(grid)
    i = int(np.argmin(v))
    assert abs(grid[i] + 1.2784645427610738) < 2e-5 and abs(v[i] + 0.2784645427610738) < 1e-10


def test_silu_derivative_matches_the_formula():
    # d/dx silu = sigma (1 + x (1 - sigma)): a central difference of the oracle must agree
    x = np.linspace(-6, 6, 49)
    h = 1e-6
    num = (np_oracle.silu(x + h) - np_oracle.silu(x - h)) / (2 * h)
    sig = 1.0 / (1.0 + np.exp(-x))
    np.testing.assert_allclose(num, sig * (1 + x * (1 - sig)), rtol=0, atol=1e-8)


def test_swiglu_hand_case():
    # one token, K = 8, one group; gate row (code - z) * s = [1, 1, 0, ...] * 0.5, up row = [2, 0, ...] * 0.25
    G = 8
    codes = np.array([[9, 9, 8, 8, 8, 8, 8, 8], [10, 8, 8, 8, 8, 8, 8, 8]], dtype=np.uint8)
    scales = np.array([[0.5], [0.25]], dtype=np.float16)
    zeros = np.array([[8.0], [8.0]], dtype=np.float16)
    x = wl.f32_to_bf16_bits(np.array([[2.0, 1.0, 5.0, 0, 0, 0, 0, 0]], dtype=np.float32))
    # gate = 0.5 * (2 + 1) = 1.5, up = 0.25 * 2 * 2 = 1.0
    y = np_oracle.linear_w4a16_swiglu(x, codes, scales, zeros, G)
    assert y.shape == (1, 1)
    assert abs(y[0, 0] - 1.5 / (1.0 + math.exp(-1.5)) * 1.0) < 1e-15
    # swapping the two rows swaps the roles: silu(1.0) * 1.5
    y2 = np_oracle.linear_w4a16_swiglu(x, codes[::-1], scales[::-1], zeros[::-1], G)
    assert abs(y2[0, 0] - 1.0 / (1.0 + math.exp(-1.0)) * 1.5) < 1e-15


def test_swiglu_is_two_plain_linears_and_the_activation():
    rng = wl.generator(77, 0)
    N2, K, G, M = 24, 64, 32, 5
    gate = rng.normal(0, 0.3, (N2, K)).astype(np.float32)
    up = rng.normal(0, 0.3, (N2, K)).astype(np.float32)
    x = wl.normal_activations_bf16(77, 1, M, K)
    qg = np_oracle.quantize_rtn_w4_asym(gate, G)
    qu = np_oracle.quantize_rtn_w4_asym(up, G)
    inter = [np.stack((a, b), axis=1).reshape(2 * N2, -1) for a, b in zip(qg, qu)]
    # interleaving rows before or after quantising is the same thing (the quantiser works row by row)
    both = np.stack((gate, up), axis=1).reshape(2 * N2, K)
    for a, b in zip(np_oracle.quantize_rtn_w4_asym(both, G), inter):
        np.testing.assert_array_equal(a, b)
    y = np_oracle.linear_w4a16_swiglu(x, *inter, G)
    yg = np_oracle.linear_w4a16(x, *qg, G)
    yu = np_oracle.linear_w4a16(x, *qu, G)
    expect = yg / (1.0 + np.exp(-yg)) * yu
    np.testing.assert_allclose(y, expect, rtol=1e-13, atol=1e-15)
    # a zero up projection gives zero; a zero gate gives zero as well (silu(0) = 0)
    z_up = [inter[0].copy(), inter[1], inter[2]]
    z_up[0][1::2] = inter[2][1::2].astype(np.uint8).repeat(G, axis=1)   # code = zero point: dequantises to 0
    assert np.all(np_oracle.linear_w4a16_swiglu(x, *z_up, G) == 0.0)
    z_gate = [inter[0].copy(), inter[1], inter[2]]
    z_gate[0][0::2] = inter[2][0::2].astype(np.uint8).repeat(G, axis=1)
    assert np.all(np_oracle.linear_w4a16_swiglu(x, *z_gate, G) == 0.0)


# ---- the low-rank side path (np_oracle.lora_side) ----
def test_lora_side_hand_case_and_identities():
    f = wl.f32_to_bf16_bits
    # rank 1: A = [1, 2, 0, 0], B = [[3], [-1]], x = [[1, 1, 5, 7]]: x . A^T = 3, times B = [9, -3], times scale 0.5
    x = f(np.array([[1.0, 1.0, 5.0, 7.0]], dtype=np.float32))
    a = f(np.array([[1.0, 2.0, 0.0, 0.0]], dtype=np.float32))
    b = f(np.array([[3.0], [-1.0]], dtype=np.float32))
    np.testing.assert_array_equal(np_oracle.lora_side(x, a, b, 0.5), [[4.5, -1.5]])
    # it is the dense linear with W = B A (exactly representable operands -> exact)
    rng = wl.generator(78, 0)
    M, K, r, N = 5, 16, 3, 7
    xi = rng.integers(-4, 5, (M, K)).astype(np.float32)
    ai = rng.integers(-3, 4, (r, K)).astype(np.float32)
    bi = rng.integers(-3, 4, (N, r)).astype(np.float32)
    got = np_oracle.lora_side(f(xi), f(ai), f(bi), 2.0)
    np.testing.assert_array_equal(got, 2.0 * xi.astype(np.float64) @ (bi.astype(np.float64) @ ai.astype(np.float64)).T)
    # linear in the scale, zero for a zero factor, and transposing the roles of A and B is a different thing
    np.testing.assert_array_equal(np_oracle.lora_side(f(xi), f(ai), f(bi), -1.0), -0.5 * got)
    assert np.all(np_oracle.lora_side(f(xi), f(0 * ai), f(bi), 1.0) == 0)
    assert np.all(np_oracle.lora_side(f(xi), f(ai), f(0 * bi), 1.0) == 0)
    # a rank-r identity embedding: A picks the first r inputs, B puts them on the first r outputs
    a_id = np.zeros((r, K), dtype=np.float32); a_id[np.arange(r), np.arange(r)] = 1
    b_id = np.zeros((N, r), dtype=np.float32); b_id[np.arange(r), np.arange(r)] = 1
    out = np_oracle.lora_side(f(xi), f(a_id), f(b_id), 1.0)
    np.testing.assert_array_equal(out[:, :r], xi[:, :r])
    assert np.all(out[:, r:] == 0)


# ---- the 3 x 3 convolution on integer codes (np_oracle.conv3x3_w4a4) ----
def test_conv3x3_hand_cases():
    # one channel, one filter, 3 x 3 image 1..9, all-ones filter: the sum of each pixel's neighbourhood inside the image
    q = np.arange(1, 10, dtype=np.int8).reshape(1, 3, 3, 1)
    ones = np.ones((1, 9), dtype=np.int8)
    acc, y = np_oracle.conv3x3_w4a4(q, 0.5, ones, np.array([2.0]))
    np.testing.assert_array_equal(acc[0, :, :, 0], [[12, 21, 16], [27, 45, 33], [24, 39, 28]])
    np.testing.assert_array_equal(y, acc.astype(np.float64))          # 0.5 * 2
    # a delta filter at tap (kh, kw) shifts the image by (kh - 1, kw - 1), zeros coming in at the border
    for kh in range(3):
        for kw in range(3):
            d = np.zeros((1, 9), dtype=np.int8)
            d[0, 3 * kh + kw] = 1
            a, _ = np_oracle.conv3x3_w4a4(q, 1.0, d, np.array([1.0]))
            want = np.zeros((3, 3), dtype=np.int64)
            for h in range(3):
                for w in range(3):
                    hh, ww = h + kh - 1, w + kw - 1
                    if 0 <= hh < 3 and 0 <= ww < 3:
                        want[h, w] = q[0, hh, ww, 0]
            np.testing.assert_array_equal(a[0, :, :, 0], want)


def test_conv3x3_is_im2col_then_the_integer_gemm_and_brute_force():
    rng = np.random.default_rng(5)
    B, H, W, Cc, Cout = 2, 4, 5, 8, 3
    q = rng.integers(-8, 8, (B, H, W, Cc)).astype(np.int8)
    w = rng.integers(-8, 8, (Cout, 9 * Cc)).astype(np.int8)
    sw = rng.random(Cout) + 0.1
    acc, y = np_oracle.conv3x3_w4a4(q, 0.25, w, sw)
    # the input generator's im2col followed by the (pinned) integer GEMM
    cols = wl.im2col_3x3(q)
    acc2, y2 = np_oracle.linear_w4a4(cols, np.full(B * H * W, 0.25), w, sw)
    np.testing.assert_array_equal(acc.reshape(B * H * W, Cout), acc2)
    np.testing.assert_allclose(y.reshape(B * H * W, Cout), y2, rtol=1e-15)
    # brute force, six nested loops
    for b in range(B):
        for h in range(H):
            for x in range(W):
                for n in range(Cout):
                    t = 0
                    for kh in range(3):
                        for kw in range(3):
                            hh, ww = h + kh - 1, x + kw - 1
                            if 0 <= hh < H and 0 <= ww < W:
                                t += int(np.dot(q[b, hh, ww].astype(np.int64), w[n, (3 * kh + kw) * Cc:(3 * kh + kw + 1) * Cc].astype(np.int64)))
                    assert acc[b, h, x, n] == t
    # one-pixel images: only the centre tap sees anything
    a1, _ = np_oracle.conv3x3_w4a4(q[:, :1, :1], 1.0, w, sw)
    np.testing.assert_array_equal(a1[:, 0, 0], q[:, 0, 0].astype(np.int64) @ w[:, 4 * Cc:5 * Cc].astype(np.int64).T)
