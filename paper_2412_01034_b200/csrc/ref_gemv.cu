// Measurement helpers, not part of the quantised path: the dense bf16 GEMV the
// paper's 16-bit baseline corresponds to (Table "OpenVLA performance", BFloat16
// row), and a read-only streaming probe.
#include "qil_common.cuh"

namespace qil {

namespace {

// One warp per output row; 128-bit loads of W (8 bf16), x through the read-only path.
__global__ void __launch_bounds__(256) ref_gemv_bf16_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w,
                                                            __nv_bfloat16* __restrict__ y, int N, int K) {
    const int lane = threadIdx.x & 31;
    const int chunks = K >> 3;
    const int warps = gridDim.x * (blockDim.x >> 5);
    for (int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); n < N; n += warps) {
        const uint4* row = w + (size_t)n * chunks;
        float acc = 0.f;
#pragma unroll 4
        for (int i = lane; i < chunks; i += 32) {
            const uint4 a = ld_stream_u4(row + i);
            const uint4 b = __ldg(x + i);
            const uint32_t au[4] = {a.x, a.y, a.z, a.w}, bu[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc = fmaf(__uint_as_float(au[j] << 16), __uint_as_float(bu[j] << 16), acc);
                acc = fmaf(__uint_as_float(au[j] & 0xFFFF0000u), __uint_as_float(bu[j] & 0xFFFF0000u), acc);
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) y[n] = __float2bfloat16_rn(acc);
    }
}

__global__ void __launch_bounds__(256) probe_read_kernel(const uint4* __restrict__ buf, size_t n16,
                                                         unsigned int* sink) {
    unsigned int acc = 0;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n16; i += 4 * stride) {
        const uint4 a = ld_stream_u4(buf + i), b = ld_stream_u4(buf + i + stride);
        const uint4 c = ld_stream_u4(buf + i + 2 * stride), d = ld_stream_u4(buf + i + 3 * stride);
        acc += a.x + a.y + a.z + a.w + b.x + b.y + b.z + b.w + c.x + c.y + c.z + c.w + d.x + d.y + d.z + d.w;
    }
    for (; i < n16; i += stride) {
        const uint4 a = ld_stream_u4(buf + i);
        acc += a.x + a.y + a.z + a.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) atomicAdd(sink, acc);
}

}  // namespace

qil_status launch_ref_gemv_bf16(const void* x, const void* w, void* y, int N, int K, cudaStream_t st) {
    int blocks = (N + 7) / 8;
    const int cap = num_sms() * 8;
    if (blocks > cap) blocks = cap;
    ref_gemv_bf16_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const uint4*>(x), reinterpret_cast<const uint4*>(w),
                                                 reinterpret_cast<__nv_bfloat16*>(y), N, K);
    return launch_status();
}

qil_status launch_probe_hbm_read(const void* buf, size_t bytes, unsigned int* sink, cudaStream_t st) {
    probe_read_kernel<<<num_sms() * 8, 256, 0, st>>>(reinterpret_cast<const uint4*>(buf), bytes / 16, sink);
    return launch_status();
}

}  // namespace qil
