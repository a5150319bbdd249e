// Weight-only 4-bit linear, general shapes (any K % 8 == 0, any group size that
// divides K, canonical layout).  One warp per output feature; the dequantisation
// (q - z) * s of the paper's weight-only deployment (Sec. 5.4) is fused into the
// dot product; accumulation is fp32, lanes are combined with warp shuffles.
// This is the path for shapes the tensor-core kernels do not take; it makes no
// attempt to amortise weight reads over rows of x beyond four at a time.
#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kRowsPerPass = 4;

__global__ void __launch_bounds__(256) w4a16_general_kernel(const uint16_t* __restrict__ x,
                                                            const uint32_t* __restrict__ qw,
                                                            const __half* __restrict__ scales,
                                                            const __half* __restrict__ zeros,
                                                            __nv_bfloat16* __restrict__ y, int M, int N, int K,
                                                            int G) {
    const int lane = threadIdx.x & 31;
    const int words = K >> 3;
    const int ng = K / G;
    const int warps = gridDim.x * (blockDim.x >> 5);
    for (int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); n < N; n += warps) {
        const uint32_t* wrow = qw + (size_t)n * words;
        for (int m0 = 0; m0 < M; m0 += kRowsPerPass) {
            float acc[kRowsPerPass] = {0.f, 0.f, 0.f, 0.f};
            for (int i = lane; i < words; i += 32) {
                const uint32_t word = wrow[i];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int k = i * 8 + j;
                    const int g = k / G;
                    const float s = __half2float(scales[(size_t)n * ng + g]);
                    const float z = __half2float(zeros[(size_t)n * ng + g]);
                    const float wv = ((float)((word >> (4 * j)) & 0xFu) - z) * s;
#pragma unroll
                    for (int r = 0; r < kRowsPerPass; ++r)
                        if (m0 + r < M) acc[r] = fmaf(bf16_bits_to_f32(x[(size_t)(m0 + r) * K + k]), wv, acc[r]);
                }
            }
#pragma unroll
            for (int r = 0; r < kRowsPerPass; ++r) {
                const float v = warp_sum(acc[r]);
                if (lane == 0 && m0 + r < M) y[(size_t)(m0 + r) * N + n] = __float2bfloat16_rn(v);
            }
        }
    }
}

}  // namespace

qil_status launch_w4a16_general(const void* x, const uint32_t* qw, const void* scales, const void* zeros,
                                void* y, int M, int N, int K, int G, cudaStream_t st) {
    int blocks = (N + 7) / 8;
    const int cap = num_sms() * 8;
    if (blocks > cap) blocks = cap;
    w4a16_general_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), qw,
                                                 reinterpret_cast<const __half*>(scales),
                                                 reinterpret_cast<const __half*>(zeros),
                                                 reinterpret_cast<__nv_bfloat16*>(y), M, N, K, G);
    return launch_status();
}

}  // namespace qil
