"""GPU parity of the 8-bit entry points (INT8 weight-only linear, int8 quantisers) against the CPU oracle.

Codes, scales and zero points must be bit-exact; bf16 outputs are judged per output row (tests/util.py).
"""
import ctypes as C

import numpy as np
import pytest

from oracle import c_oracle, np_oracle
from paper_2412_01034_b200 import workloads as wl
from tests.util import CONTRACT_REL, DERIVED_REL, assert_rows_close, bf16_to_f64, bits_of, cuda, to_bf16_cuda

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    import torch
    assert torch.cuda.is_available()
    from paper_2412_01034_b200 import api as a
    return a


def f16_bits(a):
    return np.ascontiguousarray(a).view(np.uint8).reshape(-1)


@pytest.mark.parametrize("N,K,G", [(96, 1024, 128), (33, 384, 128), (7, 4096, 4096), (64, 256, 32), (5, 48, 8)])
def test_quantize_w8_asym_bit_exact(api, N, K, G):
    w = wl.normal_weights(600, N * 7 + K, N, K, 0.02, outlier_prob=0.001)
    w[0, :G] = 0.0
    w[1 % N, :G] = -0.3
    ref = np_oracle.quantize_rtn_w8_asym(w, G)
    got = api.quantize_rtn_w8(cuda(w), G)
    np.testing.assert_array_equal(got[0].cpu().numpy(), ref[0])
    np.testing.assert_array_equal(bits_of(got[1]), f16_bits(ref[1]))
    np.testing.assert_array_equal(bits_of(got[2]), f16_bits(ref[2]))


def test_quantize_w8_hand_cases(api):
    """The hand cases of the oracle pins (exact grid, ties, scale rounded to fp16 first)."""
    q = np.array([[0, 255, 100, 37, 200, 101, 99, 1]], dtype=np.int64)
    w = ((q - 100) / 256.0).astype(np.float32)
    codes, scales, zeros = api.quantize_rtn_w8(cuda(np.repeat(w, 2, axis=0)), 8)
    np.testing.assert_array_equal(codes.cpu().numpy()[0], q[0].astype(np.uint8))
    assert bits_of(scales).view(np.uint16)[0] == 0x1C00 and float(zeros[0, 0]) == 100.0
    w2 = np.array([[0.0, 1.0, 0.7, 0.0, 0.0, 0.0, 0.0, 0.0]] * 2, dtype=np.float32)
    codes, scales, _ = api.quantize_rtn_w8(cuda(w2), 8)
    assert bits_of(scales).view(np.uint16)[0] == 0x1C04
    assert codes.cpu().numpy()[0].tolist() == [0, 255, 179, 0, 0, 0, 0, 0]


def test_quantize_w8_sym_and_activations(api):
    import torch
    w = wl.normal_weights(601, 0, 24, 1152, 0.05)
    w[3] = 0.0
    ref_q, ref_s = np_oracle.quantize_sym8(w)
    q, s, z = api.quantize_rtn_w8(cuda(w), w.shape[1], symmetric=True)
    assert z is None
    np.testing.assert_array_equal(q.cpu().numpy(), ref_q)
    np.testing.assert_array_equal(bits_of(s), np.ascontiguousarray(ref_s).view(np.uint8).reshape(-1))
    x, _ = wl.conv_stage(2, batch=1)
    x[1] = 0
    ref_q, ref_s = np_oracle.quantize_sym8(wl.bf16_bits_to_f32(x))
    qx, sx = api.quantize_act_a8(to_bf16_cuda(x))
    np.testing.assert_array_equal(qx.cpu().numpy(), ref_q)
    np.testing.assert_array_equal(bits_of(sx), np.ascontiguousarray(ref_s).view(np.uint8).reshape(-1))
    xs = wl.normal_activations_bf16(601, 2, 9, 40)
    ref_q, _ = np_oracle.quantize_sym8(wl.bf16_bits_to_f32(xs), static_scale=0.01)
    qx, sx = api.quantize_act_a8(to_bf16_cuda(xs), static_scale=0.01)
    np.testing.assert_array_equal(qx.cpu().numpy(), ref_q)
    assert ref_q.min() == -128 and ref_q.max() == 127
    assert torch.all(sx == 0.01)


def _w8_case(api, M, N, K, G, seed, x_scale=None):
    w = wl.normal_weights(610, seed, N, K, 0.02, outlier_prob=0.001)
    x = wl.normal_activations_bf16(610, seed + 1, M, K)
    if x_scale is not None:
        xf = wl.bf16_bits_to_f32(x).copy()
        xf[:, ::61] *= x_scale
        xf[:, 128:256] *= 1e-6
        x = wl.f32_to_bf16_bits(xf)
    q = np_oracle.quantize_rtn_w8_asym(w, G)
    rows = np.arange(N) if N * K <= (1 << 24) else np.sort(np.random.default_rng(N).choice(N, 512, replace=False))
    y_ref = c_oracle.linear_w8a16(x, q[0][rows], q[1][rows], q[2][rows], G)
    y = api.linear_w8a16(to_bf16_cuda(x), cuda(q[0]), cuda(q[1]), cuda(q[2]), G)
    assert tuple(y.shape) == (M, N)
    # M > 8 runs the tensor-core GEMM, which rounds every dequantised weight to bf16: judged by the contract's bound
    gemm = M > 8 and K % 64 == 0 and G % 64 == 0
    assert_rows_close(bf16_to_f64(y)[:, rows], y_ref, rel=CONTRACT_REL if gemm else DERIVED_REL)
    return y


@pytest.mark.parametrize("M,N,K,G", [
    (1, 128, 128, 128), (1, 257, 1024, 128), (2, 200, 384, 128), (3, 1000, 2176, 128), (4, 512, 1024, 256),
    (1, 4096, 4096, 128), (1, 4096, 11008, 128), (1, 11008, 4096, 128), (4, 4096, 4096, 128), (1, 160, 2048, 2048),
    (5, 300, 1024, 128), (16, 64, 512, 128), (33, 48, 256, 128), (280, 1000, 2176, 128), (130, 4096, 4096, 128),
])
def test_w8a16_stream_shapes(api, M, N, K, G):
    y1 = _w8_case(api, M, N, K, G, M + N + K)
    y2 = _w8_case(api, M, N, K, G, M + N + K)
    np.testing.assert_array_equal(bits_of(y1), bits_of(y2))


@pytest.mark.parametrize("M,N,K,G", [(1, 24, 256, 32), (6, 9, 48, 8), (2, 17, 192, 64), (3, 8, 320, 320)])
def test_w8a16_general_shapes(api, M, N, K, G):
    _w8_case(api, M, N, K, G, N * K)


def test_w8a16_hand_case(api):
    """The hand product of the oracle pins, padded with zero weights (code = zero point) to K = 16."""
    codes = np.zeros((2, 16), dtype=np.uint8)
    codes[0, :4] = [0, 255, 100, 102]
    codes[0, 4:] = 100
    codes[1, :4] = [10, 20, 30, 255]
    scales = np.array([[1 / 256.0], [1 / 128.0]], dtype=np.float16)
    zeros = np.array([[100.0], [0.0]], dtype=np.float16)
    x = np.zeros((1, 16), dtype=np.float32)
    x[0, :4] = [1.0, -2.0, 0.5, 4.0]
    y = api.linear_w8a16(to_bf16_cuda(wl.f32_to_bf16_bits(x)), cuda(codes), cuda(scales), cuda(zeros), 16)
    assert_rows_close(bf16_to_f64(y), np.array([[-402 / 256.0, 1005 / 128.0]]))


def test_w8a16_wide_dynamic_range(api):
    _w8_case(api, 2, 256, 2048, 128, 77, x_scale=3000.0)


def test_w8a16_batch_with_and_without_dependencies(api):
    """Two decoder layers of Llama-2-7B shaped 8-bit linears in one launch, once independent and once with the
    ordering of a decoder layer, against the oracle on sampled features; then a chain of small linears in which each
    reads the previous output."""
    import torch
    from paper_2412_01034_b200 import _lib
    lib = _lib.load()
    G, M = 128, 1
    shapes = {"sq": (4096, 4096), "up": (11008, 4096), "down": (4096, 11008)}
    dev, refs = {}, {}
    x_bits = {K: wl.normal_activations_bf16(620, 50 + j, M, K) for j, K in enumerate((4096, 11008))}
    xs = {K: to_bf16_cuda(b) for K, b in x_bits.items()}
    for i, (nm, (N, K)) in enumerate(shapes.items()):
        q = c_oracle.quantize_rtn_w8_asym(wl.normal_weights(620, i, N, K, 0.02, outlier_prob=0.001), G)
        dev[nm] = tuple(cuda(a) for a in q)
        rows = np.sort(np.random.default_rng(N + K).choice(N, 384, replace=False))
        refs[nm] = (rows, c_oracle.linear_w8a16(x_bits[K], q[0][rows], q[1][rows], q[2][rows], G))
    names = ["sq", "sq", "sq", "sq", "up", "up", "down"] * 2
    ys = [torch.zeros((M, shapes[nm][0]), dtype=torch.bfloat16, device="cuda") for nm in names]
    descs = (_lib.LinearDesc * len(names))()
    ws = api.new_workspace(int(lib.qil_linear_w8a16_workspace_size(4, 11008, 11008, 128)))
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    for deps in ("none", "layer"):
        for i, nm in enumerate(names):
            N, K = shapes[nm]
            d = descs[i]
            d.x, d.qweight, d.y = xs[K].data_ptr(), dev[nm][0].data_ptr(), ys[i].data_ptr()
            d.scales, d.zeros = dev[nm][1].data_ptr(), dev[nm][2].data_ptr()
            d.M, d.N, d.K, d.group_size, d.layout = M, N, K, G, api.LAYOUT_CANONICAL
            d.flags = api.DEP_PREVIOUS if (deps == "layer" and i > 0 and i % 7 in (0, 3, 4, 6)) else 0
        assert lib.qil_linear_w8a16_batch(descs, len(names), C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
        torch.cuda.synchronize()
        assert int(ws[:4].view(torch.int32).item()) == 0
        for i, nm in enumerate(names):
            rows, y_ref = refs[nm]
            assert_rows_close(bf16_to_f64(ys[i])[:, rows], y_ref)
            ys[i].zero_()
    # a chain: each entry reads the previous entry's output
    dims = [(512, 1024), (1024, 512), (768, 1024), (256, 768)]
    M = 2
    qs = [np_oracle.quantize_rtn_w8_asym(wl.normal_weights(621, i, N, K, 0.05), G) for i, (N, K) in enumerate(dims)]
    dq = [tuple(cuda(a) for a in q) for q in qs]
    x0 = wl.normal_activations_bf16(621, 100, M, dims[0][1])
    xd = to_bf16_cuda(x0)
    outs = [torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for (N, _) in dims]
    ins = [xd, outs[0], outs[1], outs[2]]
    chain = (_lib.LinearDesc * 4)()
    for i, (N, K) in enumerate(dims):
        d = chain[i]
        d.x, d.qweight, d.y = ins[i].data_ptr(), dq[i][0].data_ptr(), outs[i].data_ptr()
        d.scales, d.zeros = dq[i][1].data_ptr(), dq[i][2].data_ptr()
        d.M, d.N, d.K, d.group_size, d.layout, d.flags = M, N, K, G, api.LAYOUT_CANONICAL, (api.DEP_PREVIOUS if i else 0)
    for rep in range(2):
        assert lib.qil_linear_w8a16_batch(chain, 4, C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
        torch.cuda.synchronize()
        assert int(ws[:4].view(torch.int32).item()) == 0
        cur = x0
        for i in range(4):
            y_ref = c_oracle.linear_w8a16(cur, *qs[i], G)
            assert_rows_close(bf16_to_f64(outs[i]), y_ref, rel=1e-2)
            cur = wl.f32_to_bf16_bits(y_ref.astype(np.float32))


def test_w8a16_wait_that_runs_out_is_reported(api):
    """The phase wait of the 8-bit list kernel with QIL_DEP_NEVER and a limit of a few milliseconds: the launch
    returns, reports QIL_ERR_TIMEOUT, and the same list without the flag then runs normally."""
    import torch
    from paper_2412_01034_b200 import _lib
    lib = _lib.load()
    G, M, N, K = 128, 1, 256, 512
    q = np_oracle.quantize_rtn_w8_asym(wl.normal_weights(622, 0, N, K, 0.05), G)
    dq = tuple(cuda(a) for a in q)
    x = wl.normal_activations_bf16(622, 1, M, K)
    xd = to_bf16_cuda(x)
    ys = [torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    descs = (_lib.LinearDesc * 2)()
    for i in range(2):
        d = descs[i]
        d.x, d.qweight, d.y = xd.data_ptr(), dq[0].data_ptr(), ys[i].data_ptr()
        d.scales, d.zeros = dq[1].data_ptr(), dq[2].data_ptr()
        d.M, d.N, d.K, d.group_size, d.layout = M, N, K, G, api.LAYOUT_CANONICAL
    descs[0].flags, descs[1].flags = 0, api.DEP_PREVIOUS | api.DEP_NEVER
    ws = api.new_workspace(int(lib.qil_linear_w8a16_workspace_size(4, 11008, 11008, 128)))
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    try:
        assert lib.qil_set_wait_limit_ns(5_000_000) == 0
        assert lib.qil_linear_w8a16_batch(descs, 2, C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
        torch.cuda.synchronize()
    finally:
        lib.qil_set_wait_limit_ns(0)
    assert int(ws[:4].view(torch.int32).item()) == 7
    y_ref = c_oracle.linear_w8a16(x, *q, G)
    assert_rows_close(bf16_to_f64(ys[0]), y_ref)
    ws.zero_()
    descs[1].flags = api.DEP_PREVIOUS
    assert lib.qil_linear_w8a16_batch(descs, 2, C.c_void_p(ws.data_ptr()), ws.numel(), st) == 0
    torch.cuda.synchronize()
    assert int(ws[:4].view(torch.int32).item()) == 0
    assert_rows_close(bf16_to_f64(ys[1]), y_ref)


# ----------------------------------------------------------------------------
# W8A8 integer GEMM
# ----------------------------------------------------------------------------
def test_w8a8_extreme_codes(api):
    """All-(-128) rows against all-(-128) and all-127 rows: 2^14 K and -128 * 127 K exactly."""
    M, N, K = 19, 70, 4608
    qx = np.full((M, K), -128, np.int8)
    qw = np.full((N, K), -128, np.int8)
    qw[1] = 127
    one = np.ones(max(M, N), np.float32)
    _, acc = api.linear_w8a8(cuda(qx), cuda(one[:M]), cuda(qw), cuda(one[:N]), want_acc=True)
    a = acc.cpu().numpy()
    assert np.all(a[:, 0] == 16384 * K) and np.all(a[:, 1] == -128 * 127 * K) and np.all(a[:, 2:] == 16384 * K)


@pytest.mark.parametrize("M,N,K", [(1, 1, 16), (17, 9, 96), (130, 200, 160), (64, 64, 1152), (300, 70, 48)])
def test_w8a8_ragged_shapes(api, M, N, K):
    rng = np.random.default_rng(M * N + K)
    qx = rng.integers(-128, 128, size=(M, K)).astype(np.int8)
    qw = rng.integers(-128, 128, size=(N, K)).astype(np.int8)
    sx = rng.random(M).astype(np.float32) + 0.1
    sw = rng.random(N).astype(np.float32) + 0.1
    acc_ref, y_ref = np_oracle.linear_w8a8(qx, sx, qw, sw)
    y, acc = api.linear_w8a8(cuda(qx), cuda(sx), cuda(qw), cuda(sw), want_acc=True)
    np.testing.assert_array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert_rows_close(bf16_to_f64(y), y_ref)


@pytest.mark.parametrize("stage,batch", [(0, 32), (1, 32), (2, 32), (3, 32), (3, 2)])
def test_w8a8_conv_stages(api, stage, batch):
    """The im2col conv GEMMs of config 4 with 8-bit operands: quantisers, accumulators (bit-exact) and outputs."""
    x, w = wl.conv_stage(stage, batch=batch)
    qx_ref, sx_ref = np_oracle.quantize_sym8(wl.bf16_bits_to_f32(x))
    qw_ref, sw_ref = np_oracle.quantize_sym8(w)
    acc_ref, y_ref = c_oracle.linear_w8a8(qx_ref, sx_ref, qw_ref, sw_ref)
    qx, sx = api.quantize_act_a8(to_bf16_cuda(x))
    qw, sw, _ = api.quantize_rtn_w8(cuda(w), w.shape[1], symmetric=True)
    np.testing.assert_array_equal(qx.cpu().numpy(), qx_ref)
    np.testing.assert_array_equal(qw.cpu().numpy(), qw_ref)
    y, acc = api.linear_w8a8(qx, sx, qw, sw.reshape(-1), want_acc=True)
    np.testing.assert_array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert_rows_close(bf16_to_f64(y), y_ref)


# ----------------------------------------------------------------------------
# lists of integer GEMMs in one persistent launch
# ----------------------------------------------------------------------------
def test_int_gemm_list_conv_stages(api):
    """The four conv GEMMs of config 4 at batch 32, as 4-bit and as 8-bit entries, all eight in one launch:
    accumulators bit-exact, outputs within tolerance; a second launch reproduces the first."""
    import torch
    entries, refs = [], []
    for stage in range(4):
        x, w = wl.conv_stage(stage, batch=32)
        xf = wl.bf16_bits_to_f32(x)
        for bits in (4, 8):
            if bits == 4:
                qx_ref, sx_ref = np_oracle.quantize_sym4(xf)
                qw_ref, sw_ref = np_oracle.quantize_sym4(w)
                qx, qw = api.pack_w4(cuda(qx_ref)), api.pack_w4(cuda(qw_ref))
            else:
                qx_ref, sx_ref = np_oracle.quantize_sym8(xf)
                qw_ref, sw_ref = np_oracle.quantize_sym8(w)
                qx, qw = cuda(qx_ref), cuda(qw_ref)
            acc_ref, y_ref = c_oracle.linear_w8a8(qx_ref, sx_ref, qw_ref, sw_ref)
            M, N = acc_ref.shape
            y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
            acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
            entries.append((qx, cuda(sx_ref.reshape(-1)), qw, cuda(sw_ref.reshape(-1)), y, acc, bits))
            refs.append((acc_ref, y_ref))
    first = None
    for rep in range(2):
        api.linear_int_batch(entries)
        torch.cuda.synchronize()
        got = [bits_of(e[4]) for e in entries]
        if first is None:
            first = got
            for e, (acc_ref, y_ref) in zip(entries, refs):
                np.testing.assert_array_equal(e[5].cpu().numpy().astype(np.int64), acc_ref)
                assert_rows_close(bf16_to_f64(e[4]), y_ref)
        else:
            for a, b in zip(first, got):
                np.testing.assert_array_equal(a, b)
        for e in entries:
            e[4].zero_()


def test_int_gemm_list_ragged(api):
    import torch
    rng = np.random.default_rng(4)
    entries, refs = [], []
    for (M, N, K, bits) in [(1, 1, 32, 4), (17, 9, 96, 4), (130, 200, 160, 8), (300, 70, 48, 8), (64, 64, 1152, 4)]:
        lo, hi = (-8, 8) if bits == 4 else (-128, 128)
        qx = rng.integers(lo, hi, size=(M, K)).astype(np.int8)
        qw = rng.integers(lo, hi, size=(N, K)).astype(np.int8)
        sx = rng.random(M).astype(np.float32) + 0.1
        sw = rng.random(N).astype(np.float32) + 0.1
        refs.append(np_oracle.linear_w8a8(qx, sx, qw, sw))
        dx, dw = (api.pack_w4(cuda(qx)), api.pack_w4(cuda(qw))) if bits == 4 else (cuda(qx), cuda(qw))
        entries.append((dx, cuda(sx), dw, cuda(sw), torch.zeros((M, N), dtype=torch.bfloat16, device="cuda"),
                        torch.zeros((M, N), dtype=torch.int32, device="cuda"), bits))
    api.linear_int_batch(entries)
    torch.cuda.synchronize()
    for e, (acc_ref, y_ref) in zip(entries, refs):
        np.testing.assert_array_equal(e[5].cpu().numpy().astype(np.int64), acc_ref)
        assert_rows_close(bf16_to_f64(e[4]), y_ref)
