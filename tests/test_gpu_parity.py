"""GPU parity: every entry point of the C ABI against the CPU oracle on the same seeded inputs.

Integer results (codes, scales, zero points, packed words, int32 accumulators) must be bit-exact;
bf16 outputs are judged per output row (see tests/util.py).
"""
import json
import os

import numpy as np
import pytest

from oracle import c_oracle, np_oracle
from paper_2412_01034_b200 import workloads as wl
from tests.util import CONTRACT_REL, DERIVED_REL, assert_rows_close, bf16_to_f64, bits_of, cuda, to_bf16_cuda

pytestmark = pytest.mark.gpu

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")))


@pytest.fixture(scope="module")
def api():
    import torch
    assert torch.cuda.is_available()
    from paper_2412_01034_b200 import api as a
    return a


def f16_bits(a):
    return np.ascontiguousarray(a).view(np.uint8)


# ----------------------------------------------------------------------------
# quantisers
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("case", ["asym_4x8_g8", "asym_4x8_g4"])
def test_quantize_hand_cases(api, case):
    c = GOLD[case]
    w = np.array(c["w"], dtype=np.float32)
    codes, scales, zeros = api.quantize_rtn_w4(cuda(w), c["group"])
    np.testing.assert_array_equal(codes.cpu().numpy(), np.array(c["codes"], dtype=np.uint8))
    np.testing.assert_array_equal(scales.cpu().numpy().astype(np.float64), np.array(c["scales"]))
    np.testing.assert_array_equal(zeros.cpu().numpy().astype(np.float64), np.array(c["zeros"], dtype=np.float64))


@pytest.mark.parametrize("N,K,G", [(96, 1024, 128), (33, 384, 128), (7, 4096, 4096), (64, 256, 32), (5, 40, 8)])
def test_quantize_asym_bit_exact(api, N, K, G):
    w = wl.normal_weights(200, N * 7 + K, N, K, 0.02, outlier_prob=0.001)
    w[0, :G] = 0.0            # all-zero group
    w[1 % N, :G] = -0.3       # all-equal group
    w[2 % N, 0] = 1e-9
    ref = np_oracle.quantize_rtn_w4_asym(w, G)
    got = api.quantize_rtn_w4(cuda(w), G)
    np.testing.assert_array_equal(got[0].cpu().numpy(), ref[0])
    np.testing.assert_array_equal(bits_of(got[1]), f16_bits(ref[1]).reshape(-1))
    np.testing.assert_array_equal(bits_of(got[2]), f16_bits(ref[2]).reshape(-1))


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
def test_quantize_asym_16bit_inputs(api, dtype):
    import torch
    w32 = wl.normal_weights(201, 0, 48, 512, 0.02)
    wt = cuda(w32).to(torch.bfloat16 if dtype == "bf16" else torch.float16)
    w_widened = wt.to(torch.float32).cpu().numpy()  # exact widening
    ref = np_oracle.quantize_rtn_w4_asym(w_widened, 128)
    got = api.quantize_rtn_w4(wt, 128)
    np.testing.assert_array_equal(got[0].cpu().numpy(), ref[0])
    np.testing.assert_array_equal(bits_of(got[1]), f16_bits(ref[1]).reshape(-1))
    np.testing.assert_array_equal(bits_of(got[2]), f16_bits(ref[2]).reshape(-1))


def test_quantize_scale_overflow_sets_error(api):
    w = np.zeros((2, 128), dtype=np.float32)
    w[1, 5] = 2.0e6
    with pytest.raises(api.QilError) as e:
        api.quantize_rtn_w4(cuda(w), 128)
    assert e.value.code == api.ERR_RANGE


@pytest.mark.parametrize("stage", [0, 3])
def test_quantize_sym_per_channel(api, stage):
    _, w = wl.conv_stage(stage, batch=1)
    w[3] = 0.0
    ref_q, ref_s = np_oracle.quantize_sym4(w)
    q, s, z = api.quantize_rtn_w4(cuda(w), w.shape[1], symmetric=True)
    assert z is None
    np.testing.assert_array_equal(q.cpu().numpy(), ref_q)
    np.testing.assert_array_equal(bits_of(s), np.ascontiguousarray(ref_s).view(np.uint8).reshape(-1))


def test_quantize_sym_groups_f16_scale(api):
    import torch
    w = wl.normal_weights(202, 0, 24, 512, 0.05)
    ref_q, ref_s = np_oracle.quantize_sym4(w, group_size=64, scale_f16=True)
    q, s, _ = api.quantize_rtn_w4(cuda(w), 64, symmetric=True, scale_dtype=torch.float16)
    np.testing.assert_array_equal(q.cpu().numpy(), ref_q)
    np.testing.assert_array_equal(bits_of(s), f16_bits(ref_s).reshape(-1))


def test_quantize_act_matches_oracle(api):
    c = GOLD["sym_row"]
    v = np.array(c["v"], dtype=np.float32)
    qx, sx = api.quantize_act_a4(to_bf16_cuda(wl.f32_to_bf16_bits(v)))
    got = np_oracle.unpack_w4(qx.cpu().numpy().view(np.uint32), signed=True)
    np.testing.assert_array_equal(got, np.array(c["codes"], dtype=np.int8))
    assert float(sx[0]) == c["scale"][0]
    vs = np.array(c["v_static"], dtype=np.float32)
    qx, sx = api.quantize_act_a4(to_bf16_cuda(wl.f32_to_bf16_bits(vs)), static_scale=c["static_scale"])
    np.testing.assert_array_equal(np_oracle.unpack_w4(qx.cpu().numpy().view(np.uint32), signed=True),
                                  np.array(c["codes_static"], dtype=np.int8))
    assert float(sx[0]) == c["static_scale"]


@pytest.mark.parametrize("stage,batch", [(3, 2), (2, 1), (0, 1)])
def test_quantize_act_conv_inputs(api, stage, batch):
    x, _ = wl.conv_stage(stage, batch=batch)
    x[1] = 0  # an all-zero row
    ref_q, ref_s = np_oracle.quantize_sym4(wl.bf16_bits_to_f32(x))
    qx, sx = api.quantize_act_a4(to_bf16_cuda(x))
    np.testing.assert_array_equal(qx.cpu().numpy().view(np.uint32), np_oracle.pack_w4(ref_q))
    np.testing.assert_array_equal(bits_of(sx), np.ascontiguousarray(ref_s).view(np.uint8).reshape(-1))


def test_quantize_act_ragged_k_and_static(api):
    x = wl.normal_activations_bf16(203, 0, 37, 40)
    ref_q, ref_s = np_oracle.quantize_sym4(wl.bf16_bits_to_f32(x), static_scale=0.3)
    qx, sx = api.quantize_act_a4(to_bf16_cuda(x), static_scale=0.3)
    np.testing.assert_array_equal(qx.cpu().numpy().view(np.uint32), np_oracle.pack_w4(ref_q))
    assert ref_q.min() == -8 and ref_q.max() == 7
    np.testing.assert_array_equal(sx.cpu().numpy(), np.full(37, np.float32(0.3)))


# ----------------------------------------------------------------------------
# packing
# ----------------------------------------------------------------------------
def test_pack_hand_words(api):
    c = GOLD["pack_words"]
    u = api.pack_w4(cuda(np.array(c["unsigned_codes"], dtype=np.uint8)))
    assert int(u.cpu().numpy().view(np.uint32)[0, 0]) == int(c["unsigned_word"][0], 16)
    s = api.pack_w4(cuda(np.array(c["signed_codes"], dtype=np.int8)))
    assert int(s.cpu().numpy().view(np.uint32)[0, 0]) == int(c["signed_word"][0], 16)


@pytest.mark.parametrize("N,K", [(48, 384), (16, 128), (33, 264)])
def test_pack_unpack_layouts(api, N, K):
    rng = np.random.default_rng(N + K)
    codes = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    ref = np_oracle.pack_w4(codes)
    p = api.pack_w4(cuda(codes), api.LAYOUT_CANONICAL)
    np.testing.assert_array_equal(p.cpu().numpy().view(np.uint32), ref)
    np.testing.assert_array_equal(api.unpack_w4(p, N, K).cpu().numpy(), codes)
    if N % 16 == 0 and K % 128 == 0:
        pt = api.pack_w4(cuda(codes), api.LAYOUT_TILE16)
        np.testing.assert_array_equal(pt.cpu().numpy().view(np.uint32), np_oracle.to_layout(ref, np_oracle.LAYOUT_TILE16))
        np.testing.assert_array_equal(api.unpack_w4(pt, N, K, api.LAYOUT_TILE16).cpu().numpy(), codes)
    sc = rng.integers(-8, 8, size=(N, K)).astype(np.int8)
    ps = api.pack_w4(cuda(sc))
    np.testing.assert_array_equal(api.unpack_w4(ps, N, K, signed=True).cpu().numpy(), sc)


# ----------------------------------------------------------------------------
# W4A16
# ----------------------------------------------------------------------------
def _prefill_path(M, K, G, layout):
    """Shapes that qil_linear_w4a16 serves with the tensor-core prefill GEMM: it rounds every dequantised weight and
    every group scale to bf16 (each within 2^-9, independent signs), so its error is a random sum that the tests
    hold to the contract's 1e-2 of the row maximum instead of the tighter figure derived for fp32 dequantisation."""
    return layout == 0 and M > 8 and K % 64 == 0 and G % 64 == 0


def _w4a16_case(api, M, N, K, G, layout, seed, outliers=True):
    w = wl.normal_weights(300, seed, N, K, 0.02, outlier_prob=0.001 if outliers else 0.0)
    x = wl.normal_activations_bf16(300, seed + 1, M, K)
    codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, G)
    y_ref = c_oracle.linear_w4a16(x, codes, scales, zeros, G)
    packed = api.pack_w4(cuda(codes), layout)
    y = api.linear_w4a16(to_bf16_cuda(x), packed, cuda(scales), cuda(zeros), N, G, layout)
    assert tuple(y.shape) == (M, N)
    assert_rows_close(bf16_to_f64(y), y_ref, rel=CONTRACT_REL if _prefill_path(M, K, G, layout) else DERIVED_REL)
    return y


@pytest.mark.parametrize("case", ["asym_4x8_g8", "asym_4x8_g4"])
def test_w4a16_hand_cases(api, case):
    c = GOLD[case]
    codes = np.array(c["codes"], dtype=np.uint8)
    scales = np.array(c["scales"], dtype=np.float16)
    zeros = np.array(c["zeros"], dtype=np.float16)
    x = wl.f32_to_bf16_bits(np.array(GOLD["x_rows_8"], dtype=np.float32))
    packed = api.pack_w4(cuda(codes))
    y = api.linear_w4a16(to_bf16_cuda(x), packed, cuda(scales), cuda(zeros), 4, c["group"])
    assert_rows_close(bf16_to_f64(y), np.array(c["y"]))


@pytest.mark.parametrize("M", [1, 2, 3, 7, 8, 9, 16, 17, 33, 64, 65, 130])
@pytest.mark.parametrize("layout", [0, 1])
def test_w4a16_skinny_m_sweep(api, M, layout):
    _w4a16_case(api, M, 208, 1024, 128, layout, seed=M)


@pytest.mark.parametrize("N,K,G,layout", [
    (16, 128, 128, 1), (16, 128, 128, 0), (100, 384, 128, 0), (1000, 2176, 128, 0), (48, 1024, 256, 1),
    (48, 1024, 1024, 1), (4096, 4096, 128, 1), (256, 11008, 128, 1), (11008, 512, 128, 0),
])
def test_w4a16_skinny_shapes(api, N, K, G, layout):
    for M in (1, 5):
        _w4a16_case(api, M, N, K, G, layout, seed=N + K + G)


@pytest.mark.parametrize("M,N,K,G", [
    (280, 512, 1024, 128), (130, 200, 256, 64), (65, 1000, 2176, 128), (129, 136, 128, 128), (300, 77, 192, 192),
    # two tiles shared by eight CTAs each (all parts written, second kernel), tiles shared by two CTAs (completed in the
    # kernel), three token tiles, tiles of up to 64 / 144 tokens (four / two accumulators per output)
    (280, 256, 4096, 128), (280, 2048, 1024, 128), (600, 384, 1024, 128), (40, 640, 2048, 128), (100, 1280, 1024, 64),
])
def test_w4a16_prefill_shapes(api, M, N, K, G):
    """The tcgen05 prefill GEMM (M > 8, canonical layout): ragged M and N, one to many K steps, groups of one or
    several steps, every way its persistent launch shares tiles between CTAs; run twice: the result must not depend
    on what the previous launch left behind."""
    y1 = _w4a16_case(api, M, N, K, G, 0, seed=M + N + K)
    y2 = _w4a16_case(api, M, N, K, G, 0, seed=M + N + K)
    np.testing.assert_array_equal(bits_of(y1), bits_of(y2))


@pytest.mark.parametrize("N,K", [(wl.HIDDEN, wl.HIDDEN), (wl.FFN, wl.HIDDEN), (wl.HIDDEN, wl.FFN)])
def test_cfg2_prefill_shapes(api, N, K):
    """Config 2: the Llama-2-7B linear shapes at prefill length 280; the oracle runs on 256 sampled output
    features (the kernel computes all N)."""
    M, G = wl.PREFILL_M, wl.GROUP_SIZE
    w = wl.normal_weights(2, N + K, N, K, 0.02, outlier_prob=0.001)
    x = wl.normal_activations_bf16(2, N + K + 1, M, K)
    got = api.quantize_rtn_w4(cuda(w), G)
    rows = np.sort(np.random.default_rng(N + K).choice(N, 256, replace=False))
    codes, scales, zeros = got[0].cpu().numpy()[rows], got[1].cpu().numpy()[rows], got[2].cpu().numpy()[rows]
    ref = np_oracle.quantize_rtn_w4_asym(w[rows], G)
    np.testing.assert_array_equal(codes, ref[0])
    y = api.linear_w4a16(to_bf16_cuda(x), api.pack_w4(got[0]), got[1], got[2], N, G)
    y_ref = c_oracle.linear_w4a16(x, *ref, G)
    # the row maximum over the sampled features lower-bounds the true row maximum: the check is stricter
    assert_rows_close(bf16_to_f64(y)[:, rows], y_ref, rel=CONTRACT_REL)


def test_w4a16_prefill_workspace_is_reusable_across_shapes(api):
    """One workspace serves prefill GEMMs of different shapes in turn (its tile counters return to zero after every
    launch), and every repetition gives the same bits."""
    shapes = [(280, 2048, 1024), (280, 256, 4096), (64, 1536, 512), (280, 2048, 1024), (280, 256, 4096)]
    G = 128
    size = max(api.linear_w4a16_workspace_size(M, N, K, G) for (M, N, K) in shapes)
    ws = api.new_workspace(size)
    seen = {}
    for rep in range(2):
        for (M, N, K) in shapes:
            w = wl.normal_weights(310, N + K, N, K, 0.02)
            x = wl.normal_activations_bf16(310, N + K + 1, M, K)
            codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, G)
            y = api.linear_w4a16(to_bf16_cuda(x), api.pack_w4(cuda(codes)), cuda(scales), cuda(zeros), N, G, workspace=ws)
            if (M, N, K) in seen:
                np.testing.assert_array_equal(bits_of(y), seen[(M, N, K)])
            else:
                y_ref = c_oracle.linear_w4a16(x, codes, scales, zeros, G)
                assert_rows_close(bf16_to_f64(y), y_ref, rel=CONTRACT_REL)
                seen[(M, N, K)] = bits_of(y).copy()
    import torch
    assert int(ws[:4].view(torch.int32).cpu()[0]) == 0   # the status word: no wait ran out


@pytest.mark.parametrize("M,N,K,G", [
    (280, 512, 1024, 128),   # the GEMM with the fused epilogue, tiles shared by two CTAs
    (280, 256, 4096, 128),   # tiles shared by many CTAs: the epilogue runs in the kernel that adds the parts
    (130, 154, 256, 64),     # ragged M and N (N / 2 odd)
    (600, 384, 512, 128),    # three token tiles
    (40, 640, 2048, 128),    # four accumulators per output
    (4, 64, 256, 128), (280, 48, 200, 40),   # shapes the GEMM does not take: linear into the workspace, then the activation
])
def test_w4a16_swiglu(api, M, N, K, G):
    """Gate and up rows interleaved, silu(gate) * up in the epilogue (the gated MLP of the Llama-2 backbone,
    App. A.4.2) against the oracle.  Tolerance, per token row, from the linear's own contract REL (row-relative on gate
    and on up): |d silu| <= 1.1 |d gate|, so |dy| <= REL (1.1 + 1) max|gate| max|up|, plus the output's bf16 rounding."""
    w = wl.normal_weights(320, N + K, N, K, 0.05)
    x = wl.normal_activations_bf16(320, N + K + 1, M, K)
    codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, G)
    y = api.linear_w4a16_swiglu(to_bf16_cuda(x), api.pack_w4(cuda(codes)), cuda(scales), cuda(zeros), N, G)
    assert tuple(y.shape) == (M, N // 2)
    t = c_oracle.linear_w4a16(x, codes, scales, zeros, G)
    y_ref = np_oracle.silu(t[:, 0::2]) * t[:, 1::2]
    np.testing.assert_allclose(y_ref, np_oracle.linear_w4a16_swiglu(x, codes, scales, zeros, G), rtol=1e-9, atol=1e-12)
    gmax, umax = np.abs(t[:, 0::2]).max(axis=1, keepdims=True), np.abs(t[:, 1::2]).max(axis=1, keepdims=True)
    tol = (2.1 * CONTRACT_REL + 2.0 ** -8) * gmax * umax
    got = bf16_to_f64(y)
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got - y_ref) <= tol + 1e-30), float((np.abs(got - y_ref) / tol).max())
    # and the same bits on a second call
    y2 = api.linear_w4a16_swiglu(to_bf16_cuda(x), api.pack_w4(cuda(codes)), cuda(scales), cuda(zeros), N, G)
    np.testing.assert_array_equal(bits_of(y), bits_of(y2))


def test_cfg2_gate_up_swiglu_full_size(api):
    """The fused gate_up projection of config 2 at full size (22016 x 4096, 280 tokens), the oracle on 192 sampled
    (gate, up) pairs; same tolerance as test_w4a16_swiglu."""
    M, K, G = wl.PREFILL_M, wl.HIDDEN, wl.GROUP_SIZE
    N = 2 * wl.FFN
    w = wl.normal_weights(2, 9001, N, K, 0.02, outlier_prob=0.001)
    x = wl.normal_activations_bf16(2, 9002, M, K)
    got = api.quantize_rtn_w4(cuda(w), G)
    pairs = np.sort(np.random.default_rng(11).choice(N // 2, 192, replace=False))
    rows = np.stack((2 * pairs, 2 * pairs + 1), axis=1).reshape(-1)
    ref = np_oracle.quantize_rtn_w4_asym(w[rows], G)
    np.testing.assert_array_equal(got[0].cpu().numpy()[rows], ref[0])
    y = api.linear_w4a16_swiglu(to_bf16_cuda(x), api.pack_w4(got[0]), got[1], got[2], N, G)
    t = c_oracle.linear_w4a16(x, *ref, G)
    y_ref = np_oracle.silu(t[:, 0::2]) * t[:, 1::2]
    gmax, umax = np.abs(t[:, 0::2]).max(axis=1, keepdims=True), np.abs(t[:, 1::2]).max(axis=1, keepdims=True)
    tol = (2.1 * CONTRACT_REL + 2.0 ** -8) * gmax * umax   # (sampled maxima lower-bound the row's: the check is stricter)
    err = np.abs(bf16_to_f64(y)[:, pairs] - y_ref)
    assert np.all(err <= tol), float((err / tol).max())


@pytest.mark.parametrize("M,N,K,r", [(1, 4096, 4096, 32), (7, 1000, 2176, 32), (280, 513, 1024, 16), (9, 64, 34, 5), (33, 2, 64, 1)])
def test_lora_side_add(api, M, N, K, r):
    """The unmerged low-rank adapter beside a quantised linear (QLoRA rank 32, App. A.1.2): y += scale (x A^T) B^T on
    top of an existing bf16 y.  fp32 accumulation over K and over the rank, one bf16 rounding of the sum: the error is
    bounded by the output's half ulp plus fp32 round-off of the two inner products."""
    import torch
    rng = wl.generator(330, N + K)
    x = wl.normal_activations_bf16(330, 1, M, K)
    a = wl.f32_to_bf16_bits(rng.normal(0, 0.05, (r, K)).astype(np.float32))
    b = wl.f32_to_bf16_bits(rng.normal(0, 0.05, (N, r)).astype(np.float32))
    y0 = wl.f32_to_bf16_bits(rng.normal(0, 1.0, (M, N)).astype(np.float32))
    scale = 2.0
    side = np_oracle.lora_side(x, a, b, scale)
    want = np_oracle.bf16_to_f32(y0).astype(np.float64) + side
    y = to_bf16_cuda(y0).clone()
    api.lora_side_add(to_bf16_cuda(x), to_bf16_cuda(a), to_bf16_cuda(b), y, scale)
    got = bf16_to_f64(y)
    # |x A^T| terms: K products, fp32; the rank sum: r products
    absside = scale * np.abs(np_oracle.bf16_to_f32(x).astype(np.float64)) @ np.abs(np_oracle.bf16_to_f32(a).astype(np.float64)).T \
        @ np.abs(np_oracle.bf16_to_f32(b).astype(np.float64)).T
    tol = 2.0 ** -8 * np.abs(want) + (K + r + 4) * 2.0 ** -24 * absside + 1e-30
    assert np.all(np.abs(got - want) <= tol), float((np.abs(got - want) / tol).max())
    # untouched when the scale is zero
    y1 = to_bf16_cuda(y0).clone()
    api.lora_side_add(to_bf16_cuda(x), to_bf16_cuda(a), to_bf16_cuda(b), y1, 0.0)
    np.testing.assert_array_equal(bits_of(y1), bits_of(to_bf16_cuda(y0)))


@pytest.mark.parametrize("N,K,G", [(24, 256, 32), (9, 40, 8), (17, 192, 64), (8, 320, 320)])
def test_w4a16_general_shapes(api, N, K, G):
    for M in (1, 6):
        _w4a16_case(api, M, N, K, G, 0, seed=N * K)


def test_w4a16_is_deterministic_and_workspace_is_reusable(api):
    import torch
    N, K, G, M = 512, 4096, 128, 4
    w = wl.normal_weights(301, 0, N, K, 0.02)
    x = wl.normal_activations_bf16(301, 1, M, K)
    codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, G)
    y_ref = c_oracle.linear_w4a16(x, codes, scales, zeros, G)
    packed = api.pack_w4(cuda(codes), 1)
    ws = api.new_workspace(api.linear_w4a16_workspace_size(M, N, K, G))
    xs, sc, zr = to_bf16_cuda(x), cuda(scales), cuda(zeros)
    outs = [api.linear_w4a16(xs, packed, sc, zr, N, G, 1, workspace=ws).clone() for _ in range(3)]
    torch.cuda.synchronize()
    assert_rows_close(bf16_to_f64(outs[0]), y_ref)
    for o in outs[1:]:
        np.testing.assert_array_equal(bits_of(o), bits_of(outs[0]))
    # canary: the call writes nothing outside y
    big = torch.full((M * N + 64,), 7.0, dtype=torch.bfloat16, device="cuda")
    api.linear_w4a16(xs, packed, sc, zr, N, G, 1, out=big[:M * N].view(M, N), workspace=ws)
    assert torch.all(big[M * N:] == 7.0)


def test_w4a16_large_activations_keep_precision(api):
    """|x| up to a few thousand (LLM outlier channels): the 128-offset trick must not lose the signal."""
    N, K, G, M = 64, 1024, 128, 3
    w = wl.normal_weights(302, 0, N, K, 0.02)
    xf = wl.bf16_bits_to_f32(wl.normal_activations_bf16(302, 1, M, K)).copy()
    xf[:, ::97] *= 3000.0
    x = wl.f32_to_bf16_bits(xf)
    codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, G)
    y_ref = c_oracle.linear_w4a16(x, codes, scales, zeros, G)
    y = api.linear_w4a16(to_bf16_cuda(x), api.pack_w4(cuda(codes), 1), cuda(scales), cuda(zeros), N, G, 1)
    assert_rows_close(bf16_to_f64(y), y_ref)


def test_cfg0_full(api):
    """Config 0 exactly as stated: M=1, K=N=4096, N(0, 0.02) weights, group 128, seed 0."""
    w, x = wl.cfg0()
    ref = np_oracle.quantize_rtn_w4_asym(w, 128)
    got = api.quantize_rtn_w4(cuda(w), 128)
    np.testing.assert_array_equal(got[0].cpu().numpy(), ref[0])
    np.testing.assert_array_equal(bits_of(got[1]), f16_bits(ref[1]).reshape(-1))
    np.testing.assert_array_equal(bits_of(got[2]), f16_bits(ref[2]).reshape(-1))
    for layout in (0, 1):
        packed = api.pack_w4(got[0], layout)
        np.testing.assert_array_equal(packed.cpu().numpy().view(np.uint32).reshape(-1),
                                      np_oracle.to_layout(np_oracle.pack_w4(ref[0]), layout))
        y = api.linear_w4a16(to_bf16_cuda(x), packed, got[1], got[2], 4096, 128, layout)
        assert_rows_close(bf16_to_f64(y), c_oracle.linear_w4a16(x, *ref, 128))


@pytest.mark.parametrize("N,K", [(wl.FFN, wl.HIDDEN), (wl.HIDDEN, wl.FFN)])
@pytest.mark.parametrize("M", [1, 16, 64])
def test_cfg3_shapes(api, N, K, M):
    """Config 3 shapes; the oracle runs on 512 sampled output features (the kernel computes all N)."""
    w = wl.normal_weights(3, 0 if N == wl.FFN else 1, N, K, 0.02)
    x = wl.normal_activations_bf16(3, 10 + M, M, K)
    got = api.quantize_rtn_w4(cuda(w), 128)
    packed = api.pack_w4(got[0], 1)
    y = bf16_to_f64(api.linear_w4a16(to_bf16_cuda(x), packed, got[1], got[2], N, 128, 1))
    rows = np.sort(np.random.default_rng(M).choice(N, 512, replace=False))
    ref = np_oracle.quantize_rtn_w4_asym(w[rows], 128)
    np.testing.assert_array_equal(got[0].cpu().numpy()[rows], ref[0])
    y_ref = c_oracle.linear_w4a16(x, *ref, 128)
    # the row maximum over the sampled features lower-bounds the true row maximum: the check is stricter
    assert_rows_close(y[:, rows], y_ref)


# ----------------------------------------------------------------------------
# W4A16, tensor-memory (tcgen05) decode kernel (QIL_LAYOUT_STREAM128)
# ----------------------------------------------------------------------------
def _status(api, ws):
    """The status word at the start of a workspace (0 unless a bounded device-side wait ran out)."""
    import ctypes as C
    import torch
    from paper_2412_01034_b200 import _lib
    out = C.c_int(-1)
    rc = _lib.load().qil_device_status(C.c_void_p(ws.data_ptr()), C.byref(out),
                                       C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 0
    return out.value


def _tc_inputs(api, M, N, K, G, seed, x_scale=None):
    w = wl.normal_weights(320, seed, N, K, 0.02, outlier_prob=0.001)
    x = wl.normal_activations_bf16(320, seed + 1, M, K)
    if x_scale is not None:
        xf = wl.bf16_bits_to_f32(x).copy()
        xf[:, ::61] *= x_scale
        x = wl.f32_to_bf16_bits(xf)
    codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, G)
    buf = api.pack_stream128_w4(cuda(codes), cuda(scales), cuda(zeros), G)
    return x, codes, scales, zeros, buf


@pytest.mark.parametrize("N,K,G", [(200, 384, 128), (128, 128, 128), (40, 256, 256)])
def test_pack_stream128_matches_oracle(api, N, K, G):
    _, codes, scales, zeros, buf = _tc_inputs(api, 1, N, K, G, N + K)
    ref = np_oracle.to_stream128(codes, scales, zeros, G)
    np.testing.assert_array_equal(buf.cpu().numpy()[:ref.size], ref)


@pytest.mark.parametrize("M,N,K,G", [
    (1, 128, 128, 128), (1, 256, 1024, 128), (2, 200, 384, 128), (3, 1000, 2176, 128), (4, 512, 1024, 256),
    (1, 4096, 4096, 128), (1, 4096, 11008, 128), (1, 11008, 4096, 128), (4, 4096, 4096, 128), (1, 160, 2048, 2048),
    (1, 37008, 256, 128), (2, 48, 512, 128), (4, 4096, 11008, 128), (2, 11008, 4096, 128),
])
def test_w4a16_tc_shapes(api, M, N, K, G):
    import torch
    x, codes, scales, zeros, buf = _tc_inputs(api, M, N, K, G, M + N + K)
    rows = np.arange(N) if N * K <= (1 << 24) else np.sort(np.random.default_rng(N).choice(N, 512, replace=False))
    y_ref = c_oracle.linear_w4a16(x, codes[rows], scales[rows], zeros[rows], G)
    ws = api.new_workspace(api.linear_w4a16_workspace_size(M, N, K, G))
    outs = []
    for _ in range(2):
        y = api.linear_w4a16(to_bf16_cuda(x), buf, None, None, N, G, api.LAYOUT_STREAM128, workspace=ws)
        outs.append(y.clone())
    assert _status(api, ws) == 0
    assert_rows_close(bf16_to_f64(outs[0])[:, rows], y_ref)
    np.testing.assert_array_equal(bits_of(outs[0]), bits_of(outs[1]))
    # every {value, tag} pair handed over between CTAs has been consumed (tags cleared)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    pairs = ws[256:256 + sms * 2 * 4 * 512 * 8].view(torch.int32).view(-1, 2)
    assert int(torch.count_nonzero(pairs[:, 1]).item()) == 0


def test_w4a16_tc_wide_dynamic_range(api):
    """Outlier channels 3000x larger than the rest, and a block of tiny values: the per-block fixed point
    must keep the small blocks' contribution (their scale is independent of the outlier blocks)."""
    M, N, K, G = 2, 256, 2048, 128
    x, codes, scales, zeros, buf = _tc_inputs(api, M, N, K, G, 77, x_scale=3000.0)
    xf = wl.bf16_bits_to_f32(x).copy()
    xf[:, 1024:1152] *= 1e-6
    xf[1, 1280:1408] = 0.0
    x = wl.f32_to_bf16_bits(xf)
    y_ref = c_oracle.linear_w4a16(x, codes, scales, zeros, G)
    y = api.linear_w4a16(to_bf16_cuda(x), buf, None, None, N, G, api.LAYOUT_STREAM128)
    assert_rows_close(bf16_to_f64(y), y_ref)


def test_w4a16_tc_batch_with_dependencies(api):
    import ctypes as C
    import torch
    from paper_2412_01034_b200 import _lib
    lib = _lib.load()
    G, M = 128, 2
    dims = [(512, 1024), (1024, 512), (768, 1024), (256, 768)]
    packs, refs = [], []
    for i, (N, K) in enumerate(dims):
        w = wl.normal_weights(321, i, N, K, 0.05)
        q = np_oracle.quantize_rtn_w4_asym(w, G)
        refs.append(q)
        packs.append(api.pack_stream128_w4(cuda(q[0]), cuda(q[1]), cuda(q[2]), G))
    x0 = wl.normal_activations_bf16(321, 100, M, dims[0][1])
    xd = to_bf16_cuda(x0)
    ys = [torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for (N, _) in dims]
    ins = [xd, ys[0], ys[1], ys[2]]
    descs = (_lib.LinearDesc * 4)()
    for i, (N, K) in enumerate(dims):
        d = descs[i]
        d.x, d.qweight, d.y = ins[i].data_ptr(), packs[i].data_ptr(), ys[i].data_ptr()
        d.scales = d.zeros = None
        d.M, d.N, d.K, d.group_size, d.layout, d.flags = M, N, K, G, api.LAYOUT_STREAM128, (api.DEP_PREVIOUS if i else 0)
    ws = api.new_workspace(api.linear_w4a16_workspace_size(M, 1024, 1024, G))
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    for rep in range(3):
        for y in ys:
            y.zero_()
        assert lib.qil_linear_w4a16_batch(descs, 4, C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
        torch.cuda.synchronize()
        assert _status(api, ws) == 0
        got = [y.clone() for y in ys]
        cur = xd
        for i, (N, K) in enumerate(dims):
            one = api.linear_w4a16(cur, packs[i], None, None, N, G, api.LAYOUT_STREAM128, workspace=ws)
            np.testing.assert_array_equal(bits_of(got[i]), bits_of(one))
            cur = one
    cur_bits = x0
    for i, (N, K) in enumerate(dims):
        y_ref = c_oracle.linear_w4a16(cur_bits, *refs[i], G)
        assert_rows_close(bf16_to_f64(got[i]), y_ref, rel=1e-2)
        cur_bits = wl.f32_to_bf16_bits(y_ref.astype(np.float32))


@pytest.mark.parametrize("M", [1, 2, 4])
def test_w4a16_tc_long_list_without_dependencies(api, M):
    """Six decoder layers of Llama-2-7B shaped linears in one list, no entry waiting for another: the units of the
    whole list are one stream cut into one slice per CTA (M <= 2; at M = 4 every linear is sliced by itself), CTAs and
    the roles inside a CTA drift apart by several linears, which exercises every ring (slots between CTAs, buffers
    between roles) in its blocking state.  Every output is checked against the oracle on sampled features, and a
    second and third run must reproduce the first bit for bit."""
    import ctypes as C
    import torch
    from paper_2412_01034_b200 import _lib
    lib = _lib.load()
    G = 128
    shapes = {"sq": (4096, 4096), "up": (11008, 4096), "down": (4096, 11008)}
    packs, quant = {}, {}
    for i, (name, (N, K)) in enumerate(shapes.items()):
        w = wl.normal_weights(322, i, N, K, 0.02, outlier_prob=0.001)
        q = c_oracle.quantize_rtn_w4_asym(w, G)
        quant[name] = q
        packs[name] = api.pack_stream128_w4(cuda(q[0]), cuda(q[1]), cuda(q[2]), G)
    layer = ["sq", "sq", "sq", "sq", "up", "up", "down"]
    names = layer * 6
    x_bits = {K: wl.normal_activations_bf16(322, 50 + j, M, K) for j, K in enumerate((4096, 11008))}
    xs = {K: to_bf16_cuda(b) for K, b in x_bits.items()}
    ys = [torch.zeros((M, shapes[nm][0]), dtype=torch.bfloat16, device="cuda") for nm in names]
    descs = (_lib.LinearDesc * len(names))()
    for i, nm in enumerate(names):
        N, K = shapes[nm]
        d = descs[i]
        d.x, d.qweight, d.y = xs[K].data_ptr(), packs[nm].data_ptr(), ys[i].data_ptr()
        d.scales = d.zeros = None
        d.M, d.N, d.K, d.group_size, d.layout, d.flags = M, N, K, G, api.LAYOUT_STREAM128, 0
    ws = api.new_workspace(api.linear_w4a16_workspace_size(M, 11008, 11008, G))
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    refs = {}
    for nm, (N, K) in shapes.items():
        rows = np.sort(np.random.default_rng(N + K).choice(N, 384, replace=False))
        q = quant[nm]
        refs[nm] = (rows, c_oracle.linear_w4a16(x_bits[K], q[0][rows], q[1][rows], q[2][rows], G))
    first = None
    for rep in range(3):
        assert lib.qil_linear_w4a16_batch(descs, len(names), C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
        torch.cuda.synchronize()
        assert _status(api, ws) == 0
        got = [bits_of(y) for y in ys]
        if first is None:
            first = got
            for i, nm in enumerate(names):
                rows, y_ref = refs[nm]
                assert_rows_close(bf16_to_f64(ys[i])[:, rows], y_ref)
        else:
            for a, b in zip(first, got):
                np.testing.assert_array_equal(a, b)
        for y in ys:
            y.zero_()


def test_w4a16_workspace_is_shared_by_all_layouts(api):
    """One workspace, used in turn by the streaming list kernel (with dependencies, which leaves its counters
    behind), the split-K skinny kernel on the TILE16 layout and the list kernel again: the two parts of the
    workspace do not overlap and each call finds its part as it needs it."""
    import ctypes as C
    import torch
    from paper_2412_01034_b200 import _lib
    lib = _lib.load()
    G, M = 128, 2
    N, K = 256, 4096   # 16 row tiles of the skinny kernel, split along K
    assert lib.qil_linear_w4a16_static_ws_need(M, N, K, G) > 0
    w = wl.normal_weights(323, 0, N, K, 0.02, outlier_prob=0.001)
    x = wl.normal_activations_bf16(323, 1, M, K)
    q = np_oracle.quantize_rtn_w4_asym(w, G)
    y_ref = c_oracle.linear_w4a16(x, *q, G)
    xd = to_bf16_cuda(x)
    stream_buf = api.pack_stream128_w4(cuda(q[0]), cuda(q[1]), cuda(q[2]), G)
    tile_buf = api.pack_w4(cuda(q[0]), api.LAYOUT_TILE16)
    sd, zd = cuda(q[1]), cuda(q[2])
    ws = api.new_workspace(api.linear_w4a16_workspace_size(M, N, K, G))
    y1 = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    y2 = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    descs = (_lib.LinearDesc * 2)()
    for i, y in enumerate((y1, y2)):
        d = descs[i]
        d.x, d.qweight, d.y = xd.data_ptr(), stream_buf.data_ptr(), y.data_ptr()
        d.scales = d.zeros = None
        d.M, d.N, d.K, d.group_size, d.layout, d.flags = M, N, K, G, api.LAYOUT_STREAM128, (api.DEP_PREVIOUS if i else 0)
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    for rep in range(2):
        assert lib.qil_linear_w4a16_batch(descs, 2, C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
        torch.cuda.synchronize()
        assert _status(api, ws) == 0
        assert_rows_close(bf16_to_f64(y1), y_ref)
        assert_rows_close(bf16_to_f64(y2), y_ref)
        yt = api.linear_w4a16(xd, tile_buf, sd, zd, N, G, api.LAYOUT_TILE16, workspace=ws)
        assert_rows_close(bf16_to_f64(yt), y_ref)
        y1.zero_()
        y2.zero_()


def test_cfg1_full_list_vs_oracle(api):
    """Config 1 as the benchmark runs it: all 224 Llama-2-7B decode linears (32 layers, distinct weights and
    inputs, M = 1) in one list, once without ordering constraints and once in the order a decoder layer imposes.
    Every output of layers 0, 15 and 31 and 64 random output features of every other linear are compared with the
    oracle (quantiser and linear), and the status word must stay 0."""
    import torch
    from paper_2412_01034_b200 import llama_decode
    specs = wl.llama_linear_ids()
    full_layers = (0, 15, 31)
    rng = np.random.default_rng(11)
    keep = {i: np.sort(rng.choice(s[2], 64, replace=False)) for i, s in enumerate(specs) if s[0] not in full_layers}
    model = llama_decode.QuantisedLinears(cfg=1, M=1, n_layers=32, deps="none", keep_host_rows=keep)
    expected = {}
    for i, (layer, _, N, K, tw, _) in enumerate(specs):
        x = model.input_bits(i)
        if layer in full_layers:
            q = c_oracle.quantize_rtn_w4_asym(wl.llama_weight(1, tw, N, K), wl.GROUP_SIZE)
            expected[i] = (np.arange(N), c_oracle.linear_w4a16(x, *q, wl.GROUP_SIZE))
        else:
            rows, w_rows = model.kept[i]
            q = c_oracle.quantize_rtn_w4_asym(w_rows, wl.GROUP_SIZE)
            expected[i] = (rows, c_oracle.linear_w4a16(x, *q, wl.GROUP_SIZE))
    for deps in ("none", "layer"):
        model.set_deps(deps)
        model.y_dev.zero_()
        model.run()
        torch.cuda.synchronize()
        assert _status(api, model.ws) == 0
        for i in range(len(specs)):
            rows, y_ref = expected[i]
            y = bf16_to_f64(model.output(i))
            if len(rows) == y.shape[1]:
                assert_rows_close(y, y_ref)
            else:
                # the row maximum over the sampled features lower-bounds the true row maximum: the check is stricter
                assert_rows_close(y[:, rows], y_ref)


def test_w4a16_tc_wait_that_runs_out_is_reported(api):
    """The error path of the list kernel, without a fault: the second entry carries QIL_DEP_NEVER, so its wait for
    earlier outputs can never end; with the wait limit set to a few milliseconds the launch must return on its own,
    with QIL_ERR_TIMEOUT in the status word and the place of the wait in the words after it.  The context stays
    usable: after the workspace is zeroed again the same list, without the flag, runs normally."""
    import ctypes as C
    import torch
    from paper_2412_01034_b200 import _lib
    lib = _lib.load()
    G, M = 128, 1
    dims = [(512, 1024), (384, 512)]
    packs, refs = [], []
    for i, (N, K) in enumerate(dims):
        w = wl.normal_weights(324, i, N, K, 0.05)
        q = np_oracle.quantize_rtn_w4_asym(w, G)
        refs.append(q)
        packs.append(api.pack_stream128_w4(cuda(q[0]), cuda(q[1]), cuda(q[2]), G))
    x0 = wl.normal_activations_bf16(324, 100, M, dims[0][1])
    xd = to_bf16_cuda(x0)
    ys = [torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for (N, _) in dims]
    descs = (_lib.LinearDesc * 2)()
    for i, (N, K) in enumerate(dims):
        d = descs[i]
        d.x, d.qweight, d.y = (xd if i == 0 else ys[0]).data_ptr(), packs[i].data_ptr(), ys[i].data_ptr()
        d.scales = d.zeros = None
        d.M, d.N, d.K, d.group_size, d.layout = M, N, K, G, api.LAYOUT_STREAM128
    descs[0].flags, descs[1].flags = 0, api.DEP_PREVIOUS | api.DEP_NEVER
    ws = api.new_workspace(api.linear_w4a16_workspace_size(M, 512, 1024, G))
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    try:
        assert lib.qil_set_wait_limit_ns(5_000_000) == 0
        assert lib.qil_linear_w4a16_batch(descs, 2, C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
        torch.cuda.synchronize()     # returns: every wait is bounded
    finally:
        lib.qil_set_wait_limit_ns(0)
    assert _status(api, ws) == 7     # QIL_ERR_TIMEOUT
    head = ws[:32].view(torch.int32).cpu().numpy()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert 1 <= head[2] <= sms and 0 <= head[3] < 1024
    y_ref0 = c_oracle.linear_w4a16(x0, *refs[0], G)
    assert_rows_close(bf16_to_f64(ys[0]), y_ref0)      # the entry before the wait is complete
    ws.zero_()
    descs[1].flags = api.DEP_PREVIOUS
    for y in ys:
        y.zero_()
    assert lib.qil_linear_w4a16_batch(descs, 2, C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
    torch.cuda.synchronize()
    assert _status(api, ws) == 0
    assert_rows_close(bf16_to_f64(ys[0]), y_ref0)
    y_ref1 = c_oracle.linear_w4a16(wl.f32_to_bf16_bits(y_ref0.astype(np.float32)), *refs[1], G)
    assert_rows_close(bf16_to_f64(ys[1]), y_ref1, rel=1e-2)


# ----------------------------------------------------------------------------
# W4A4
# ----------------------------------------------------------------------------
def test_w4a4_hand_case(api):
    c = GOLD["w4a4_small"]
    qx = np.zeros((2, 32), np.int8); qx[:, :8] = np.array(c["qx"], np.int8)
    qw = np.zeros((3, 32), np.int8); qw[:, :8] = np.array(c["qw"], np.int8)
    y, acc = api.linear_w4a4(api.pack_w4(cuda(qx)), cuda(np.array(c["sx"], np.float32)), api.pack_w4(cuda(qw)),
                             cuda(np.array(c["sw"], np.float32)), want_acc=True)
    np.testing.assert_array_equal(acc.cpu().numpy(), np.array(c["acc"], dtype=np.int32))
    np.testing.assert_array_equal(bf16_to_f64(y), np.array(c["y"]))


def test_w4a4_extreme_codes(api):
    M, N, K = 19, 70, 4608
    qx = np.full((M, K), -8, np.int8)
    qw = np.full((N, K), -8, np.int8)
    qw[1] = 7
    one = np.ones(max(M, N), np.float32)
    y, acc = api.linear_w4a4(api.pack_w4(cuda(qx)), cuda(one[:M]), api.pack_w4(cuda(qw)), cuda(one[:N]), want_acc=True)
    a = acc.cpu().numpy()
    assert np.all(a[:, 0] == 64 * K) and np.all(a[:, 1] == -56 * K)


@pytest.mark.parametrize("stage,batch", [(0, 32), (1, 32), (2, 32), (3, 32), (0, 2), (1, 3)])
def test_w4a4_conv_stages(api, stage, batch):
    x, w = wl.conv_stage(stage, batch=batch)
    qx_ref, sx_ref = np_oracle.quantize_sym4(wl.bf16_bits_to_f32(x))
    qw_ref, sw_ref = np_oracle.quantize_sym4(w)
    acc_ref, y_ref = c_oracle.linear_w4a4(qx_ref, sx_ref, qw_ref, sw_ref)
    qx, sx = api.quantize_act_a4(to_bf16_cuda(x))
    qw, sw, _ = api.quantize_rtn_w4(cuda(w), w.shape[1], symmetric=True)
    y, acc = api.linear_w4a4(qx, sx, api.pack_w4(qw), sw.reshape(-1), want_acc=True)
    np.testing.assert_array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert_rows_close(bf16_to_f64(y), y_ref)
    y2 = api.linear_w4a4(qx, sx, api.pack_w4(qw), sw.reshape(-1))
    np.testing.assert_array_equal(bits_of(y2), bits_of(y))


@pytest.mark.parametrize("B,H,W,Cc,Cout", [
    (2, 5, 7, 32, 24),        # ragged everything, a step spans four taps
    (1, 1, 1, 64, 8),         # one pixel: only the centre tap is inside
    (3, 22, 50, 64, 64),      # the first conv stage's geometry (a step spans two taps)
    (2, 11, 25, 128, 128), (2, 3, 7, 512, 40),
    (32, 22, 50, 64, 64), (32, 3, 7, 512, 512),   # the first and the last conv stage at the benchmark's batch
])
def test_conv3x3_w4a4_from_the_feature_map(api, B, H, W, Cc, Cout):
    """The 3 x 3 convolution read straight from the int4 feature map (no im2col matrix): accumulators bit-exact
    against the oracle's tap-by-tap definition, bf16 outputs within the integer GEMM's tolerance, and the variant
    whose epilogue writes the next layer's int4 feature map bit-exact against the oracle's requantiser."""
    rng = np.random.default_rng(B * H * W + Cc + Cout)
    q = rng.integers(-8, 8, size=(B, H, W, Cc)).astype(np.int8)
    qw = rng.integers(-8, 8, size=(Cout, 9 * Cc)).astype(np.int8)
    sw = (rng.random(Cout) * 0.05 + 0.01).astype(np.float32)
    x_scale = 0.125
    acc_ref, y_ref = np_oracle.conv3x3_w4a4(q, x_scale, qw, sw)
    q_packed = api.pack_w4(cuda(q.reshape(B * H * W, Cc))).reshape(B, H, W, Cc // 8)
    w_packed = api.pack_w4(cuda(qw))
    y, acc = api.conv3x3_w4a4(q_packed, x_scale, w_packed, cuda(sw), want_acc=True)
    np.testing.assert_array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert_rows_close(bf16_to_f64(y).reshape(B * H * W, Cout), y_ref.reshape(B * H * W, Cout))
    if Cout % 8 == 0:
        out_scale = float(np.abs(y_ref).max() / 7.0) or 1.0
        for relu in (False, True):
            cols = wl.im2col_3x3(q)    # (input generator: only feeds the oracle's requantiser its operand)
            q_next_ref = np_oracle.linear_w4a4_requant(cols, np.full(B * H * W, x_scale, dtype=np.float32), qw, sw, out_scale, relu)
            qy = api.conv3x3_w4a4(q_packed, x_scale, w_packed, cuda(sw), out_scale=out_scale, relu=relu)
            got = np_oracle.unpack_w4(qy.cpu().numpy().view(np.uint32).reshape(B * H * W, Cout // 8), signed=True)
            np.testing.assert_array_equal(got, q_next_ref)
            # ... and it is a feature map the next layer can read
            if Cout % 32 == 0:
                qw2 = rng.integers(-8, 8, size=(8, 9 * Cout)).astype(np.int8)
                acc2_ref, _ = np_oracle.conv3x3_w4a4(q_next_ref.reshape(B, H, W, Cout), out_scale, qw2, np.ones(8, dtype=np.float32))
                _, acc2 = api.conv3x3_w4a4(qy, out_scale, api.pack_w4(cuda(qw2)), cuda(np.ones(8, dtype=np.float32)), want_acc=True)
                np.testing.assert_array_equal(acc2.cpu().numpy().astype(np.int64), acc2_ref)


@pytest.mark.parametrize("M,N,K", [(1, 1, 32), (17, 9, 96), (130, 200, 160), (64, 64, 1152)])
def test_w4a4_ragged_shapes(api, M, N, K):
    rng = np.random.default_rng(M * N + K)
    qx = rng.integers(-8, 8, size=(M, K)).astype(np.int8)
    qw = rng.integers(-8, 8, size=(N, K)).astype(np.int8)
    sx = rng.random(M).astype(np.float32) + 0.1
    sw = rng.random(N).astype(np.float32) + 0.1
    acc_ref, y_ref = np_oracle.linear_w4a4(qx, sx, qw, sw)
    y, acc = api.linear_w4a4(api.pack_w4(cuda(qx)), cuda(sx), api.pack_w4(cuda(qw)), cuda(sw), want_acc=True)
    np.testing.assert_array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert_rows_close(bf16_to_f64(y), y_ref)


# ----------------------------------------------------------------------------
# measurement helpers
# ----------------------------------------------------------------------------
def test_ref_gemv_bf16(api):
    import torch
    N, K = 300, 1024
    w = wl.normal_activations_bf16(400, 0, N, K)
    x = wl.normal_activations_bf16(400, 1, 1, K)
    y = api.ref_gemv_bf16(to_bf16_cuda(x), to_bf16_cuda(w))
    ref = wl.bf16_bits_to_f32(x).astype(np.float64) @ wl.bf16_bits_to_f32(w).astype(np.float64).T
    assert_rows_close(bf16_to_f64(y).reshape(1, -1), ref)
    buf = torch.arange(1 << 16, dtype=torch.int32, device="cuda")
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.probe_hbm_read(buf, sink)
    assert int(sink.item()) & 0xFFFFFFFF == (sum(range(1 << 16))) & 0xFFFFFFFF


@pytest.mark.parametrize("stage,batch,relu", [(2, 8, True), (3, 32, False), (1, 2, True)])
def test_w4a4_requant_epilogue(api, stage, batch, relu):
    """The W4A4 GEMM that writes the next layer's int4 activations (static scale) from its epilogue: codes bit-exact
    against the oracle, and usable as the next call's packed operand."""
    x, w = wl.conv_stage(stage, batch=batch)
    qx_ref, sx_ref = np_oracle.quantize_sym4(wl.bf16_bits_to_f32(x))
    qw_ref, sw_ref = np_oracle.quantize_sym4(w)
    out_scale = 0.75
    q_ref = c_oracle.linear_w4a4_requant(qx_ref, sx_ref, qw_ref, sw_ref, out_scale, relu)
    assert q_ref.max() == 7 and (relu or q_ref.min() == -8)
    qx, sx = api.quantize_act_a4(to_bf16_cuda(x))
    qw, sw, _ = api.quantize_rtn_w4(cuda(w), w.shape[1], symmetric=True)
    qy = api.linear_w4a4_requant(qx, sx, api.pack_w4(qw), sw.reshape(-1), out_scale, relu)
    got = np_oracle.unpack_w4(qy.cpu().numpy().view(np.uint32), signed=True)
    np.testing.assert_array_equal(got, q_ref)
