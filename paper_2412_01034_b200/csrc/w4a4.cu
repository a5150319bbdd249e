// W4A4 integer GEMM (the compute-bound driving-policy deployment of the paper,
// Sec. 5.1 / Sec. 5.4): acc = qx . qw^T in int32, y = bf16(float(acc) * sx[m] * sw[n]).
//
// Unpacking trick shared by every path in this file: for a packed word w,
//   (w << 4) & 0xF0F0F0F0  holds nibbles 0,2,4,6 and  w & 0xF0F0F0F0  holds nibbles
//   1,3,5,7, each as a signed byte equal to 16 x the int4 value (the nibble is the
//   byte's high half, so its sign bit is the byte's sign bit).
// Both operands are scaled by 16, the int32 accumulator is exactly 256 x the true
// sum (|acc| <= 64 K, so 256 |acc| < 2^31 for K <= 131072) and is shifted back.
// The order of k inside a word differs from memory order, identically for both
// operands, which leaves the sum unchanged.
#include "qil_common.cuh"

namespace qil {

namespace {

__device__ __forceinline__ void mma_s8_16832(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t even_nibbles_x16(uint32_t w) { return (w << 4) & 0xF0F0F0F0u; }
__device__ __forceinline__ uint32_t odd_nibbles_x16(uint32_t w) { return w & 0xF0F0F0F0u; }

constexpr int kNT = 8;  // 8-column tiles per warp: warp tile 16 x 64

// Register-only kernel: each warp computes a 16 x 64 tile, operands come straight
// from global memory (they are L2 resident at the sizes this path serves).
__global__ void __launch_bounds__(128) w4a4_mma_sync_kernel(const uint32_t* __restrict__ qx,
                                                            const float* __restrict__ sx,
                                                            const uint32_t* __restrict__ qw,
                                                            const float* __restrict__ sw,
                                                            __nv_bfloat16* __restrict__ y,
                                                            int32_t* __restrict__ acc_out, int M, int N, int K) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int m0 = (blockIdx.x * 4 + warp) * 16;
    const int n0 = blockIdx.y * (8 * kNT);
    if (m0 >= M) return;
    const int chunks = K >> 5;  // 128-bit chunks (32 codes) per row
    const uint4* xa = reinterpret_cast<const uint4*>(qx) + (size_t)(m0 + g) * chunks;
    const uint4* xb = reinterpret_cast<const uint4*>(qx) + (size_t)(m0 + g + 8) * chunks;
    const bool a_ok = (m0 + g) < M, b_ok = (m0 + g + 8) < M;

    int acc[kNT][4];
#pragma unroll
    for (int nt = 0; nt < kNT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[nt][c] = 0;

    for (int ks = 0; ks * 4 < chunks; ++ks) {
        const int ch = ks * 4 + t;
        const bool in = ch < chunks;
        uint4 va = make_uint4(0, 0, 0, 0), vb = make_uint4(0, 0, 0, 0);
        if (in && a_ok) va = xa[ch];
        if (in && b_ok) vb = xb[ch];
        const uint32_t wa[4] = {va.x, va.y, va.z, va.w};
        const uint32_t wb[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
        for (int nt = 0; nt < kNT; ++nt) {
            const int n = n0 + nt * 8 + g;
            uint4 vw = make_uint4(0, 0, 0, 0);
            if (in && n < N) vw = (reinterpret_cast<const uint4*>(qw) + (size_t)n * chunks)[ch];
            const uint32_t ww[4] = {vw.x, vw.y, vw.z, vw.w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                mma_s8_16832(acc[nt], even_nibbles_x16(wa[j]), even_nibbles_x16(wb[j]), odd_nibbles_x16(wa[j]),
                             odd_nibbles_x16(wb[j]), even_nibbles_x16(ww[j]), odd_nibbles_x16(ww[j]));
        }
    }

#pragma unroll
    for (int nt = 0; nt < kNT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int m = m0 + g + ((c & 2) ? 8 : 0);
            const int n = n0 + nt * 8 + 2 * t + (c & 1);
            if (m < M && n < N) {
                const int a = acc[nt][c] >> 8;  // exact: the accumulator is a multiple of 256
                if (acc_out) acc_out[(size_t)m * N + n] = a;
                y[(size_t)m * N + n] = __float2bfloat16_rn((float)a * (sx[m] * sw[n]));
            }
        }
}

}  // namespace

size_t w4a4_workspace(int M, int N, int K) {
    (void)M; (void)N; (void)K;
    return 0;
}

qil_status launch_w4a4(const uint32_t* qx, const float* sx, const uint32_t* qw, const float* sw, void* y,
                       int32_t* acc_out, int M, int N, int K, void* ws, size_t ws_bytes, cudaStream_t st) {
    (void)ws; (void)ws_bytes;
    const dim3 grid((M + 63) / 64, (N + 8 * kNT - 1) / (8 * kNT));
    w4a4_mma_sync_kernel<<<grid, 128, 0, st>>>(qx, sx, qw, sw, reinterpret_cast<__nv_bfloat16*>(y), acc_out, M, N, K);
    return launch_status();
}

}  // namespace qil
