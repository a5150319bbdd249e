"""qil_linear_w4a16_static_ws: the linear for callers that are not allowed to allocate.

A control loop that bans allocation after start-up, or a plug-in whose host owns all device
memory, cannot hand qil_linear_w4a16 the workspace it wants for K-split shapes.  The variant
tested here keeps that scratch in a fixed array inside the library.  It must give the same
result as the ordinary entry point, also on a second call (the array still holds the first
call's data then), and it must refuse shapes whose scratch would not fit.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes as C

import numpy as np
import pytest

from oracle import np_oracle
from paper_2412_01034_b200 import workloads as wl
from tests.util import assert_rows_close, bf16_to_f64, bits_of, cuda, to_bf16_cuda

pytestmark = pytest.mark.gpu


# (M, N, K, layout, uses the built-in scratch): split-K shapes on both layouts, one shape that needs no scratch, and one
# canonical M > 8 shape, where the ordinary entry point runs the prefill GEMM (bf16-rounded weights) and this one the
# skinny kernel, so that the two agree within the tolerance of the linear but not bit for bit.
CASES = [(1, 4096, 4096, 1, True), (4, 512, 4096, 1, True), (2, 256, 4096, 0, True), (3, 11008, 1024, 1, False),
         (24, 512, 2048, 0, True)]


@pytest.mark.parametrize("M,N,K,layout,uses_scratch", CASES)
def test_static_ws_matches_workspace_entry_point_twice(M, N, K, layout, uses_scratch):
    import torch
    from paper_2412_01034_b200 import _lib, api
    from tests.util import CONTRACT_REL
    lib = _lib.load()
    G = 128
    need = int(lib.qil_linear_w4a16_static_ws_need(M, N, K, G))
    assert (need > 0) == uses_scratch and need <= 4 * 1024 * 1024
    w = wl.normal_weights(500, N + K, N, K, 0.02, outlier_prob=0.001)
    x = wl.normal_activations_bf16(500, M, M, K)
    codes, scales, zeros = np_oracle.quantize_rtn_w4_asym(w, G)
    y_ref = np_oracle.linear_w4a16(x, codes, scales, zeros, G)
    packed = api.pack_w4(cuda(codes), layout)
    xd, sd, zd = to_bf16_cuda(x), cuda(scales), cuda(zeros)
    y_ws = api.linear_w4a16(xd, packed, sd, zd, N, G, layout)       # caller-allocated workspace
    same_kernel = not (layout == api.LAYOUT_CANONICAL and M > 8)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    for call in range(2):
        y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        rc = lib.qil_linear_w4a16_static_ws(C.c_void_p(xd.data_ptr()), C.c_void_p(packed.data_ptr()),
                                            C.c_void_p(sd.data_ptr()), C.c_void_p(zd.data_ptr()),
                                            C.c_void_p(y.data_ptr()), M, N, K, G, layout, stream)
        assert rc == 0, lib.qil_status_string(rc)
        torch.cuda.synchronize()
        assert_rows_close(bf16_to_f64(y), y_ref)                 # same tolerance as the parity tests
        if same_kernel:
            np.testing.assert_array_equal(bits_of(y), bits_of(y_ws), err_msg=f"call {call}")
        else:
            assert_rows_close(bf16_to_f64(y), bf16_to_f64(y_ws), rel=CONTRACT_REL)


def test_static_ws_rejects_shapes_beyond_the_built_in_scratch():
    from paper_2412_01034_b200 import _lib, api
    lib = _lib.load()
    M, N, K, G = 64, 8192, 4096, 128
    assert lib.qil_linear_w4a16_static_ws_need(M, N, K, G) > 4 * 1024 * 1024
    a = C.c_void_p(0x10000)  # aligned dummy addresses: the call must fail before touching them
    rc = lib.qil_linear_w4a16_static_ws(a, a, a, a, a, M, N, K, G, api.LAYOUT_TILE16, None)
    assert rc == 5 and b"workspace" in lib.qil_status_string(rc)
    assert lib.qil_linear_w4a16_static_ws(None, a, a, a, a, 1, 16, 128, 128, 0, None) == 1
    assert lib.qil_linear_w4a16_static_ws(a, a, a, a, a, 1, 128, 128, 128, api.LAYOUT_STREAM128, None) == 4
