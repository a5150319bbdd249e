// Low-rank side path of a quantised linear: y += scale * (x . A^T) . B^T with rank r <= 32 (the paper fine-tunes
// OpenVLA with QLoRA adapters of rank 32 over the frozen quantised base, App. A.1.2; kept unmerged, the
// adapter is this extra term beside the 4-bit linear).
//   x [M][K] bf16    A [r][K] bf16    B [N][r] bf16    y [M][N] bf16, updated in place
// Two small kernels, fp32 accumulation:
//   1. t[ks][M][r] = x . A^T over slice ks of K, into the workspace (fp32).  A block owns 8 token rows and one slice of
//      K, a warp 4 of the r columns, lanes split the slice: A is read once per 8 tokens, and at decode length (one
//      block of rows) the slices spread A over the SMs.
//   2. y[m][n] = bf16(float(y[m][n]) + scale * sum_j (sum_ks t[ks][m][j]) B[n][j]), the slices added in order.  A thread
//      owns two neighbouring outputs and reads its two rows of B with 16-byte loads; the 8 token rows of t a block
//      works on sit in shared memory.  This pass is the read-modify-write of y.
#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kRows = 8, kMaxRank = 32, kMaxSlices = 32;

__global__ void __launch_bounds__(256) lora_down_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ a,
                                                        float* __restrict__ t, int M, int K, int r, int slice) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * kRows;
    const int k_begin = blockIdx.y * slice, k_end = min(K, k_begin + slice);   // (slice is even)
    t += (size_t)blockIdx.y * M * kMaxRank;
    float acc[kRows][4];
#pragma unroll
    for (int i = 0; i < kRows; ++i)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[i][c] = 0.f;
    // columns j = warp + 8 c of t; K in pairs of bf16
    for (int k = k_begin + 2 * lane; k < k_end; k += 64) {
        float2 av[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int j = warp + 8 * c;
            av[c] = j < r ? __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(a + (size_t)j * K + k)) : make_float2(0.f, 0.f);
        }
#pragma unroll
        for (int i = 0; i < kRows; ++i) {
            if (m0 + i >= M) break;
            const float2 xv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(x + (size_t)(m0 + i) * K + k));
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[i][c] = fmaf(xv.y, av[c].y, fmaf(xv.x, av[c].x, acc[i][c]));
        }
    }
#pragma unroll
    for (int i = 0; i < kRows; ++i)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float v = warp_sum(acc[i][c]);
            const int j = warp + 8 * c;
            if (lane == 0 && m0 + i < M && j < r) t[(size_t)(m0 + i) * kMaxRank + j] = v;
        }
}

__global__ void __launch_bounds__(256) lora_up_add_kernel(const float* __restrict__ t, const __nv_bfloat16* __restrict__ b,
                                                          __nv_bfloat16* __restrict__ y, int M, int N, int r, float scale,
                                                          int slices, int vec) {
    __shared__ float st[kRows][kMaxRank];
    const int m0 = blockIdx.y * kRows;
    for (int i = threadIdx.x; i < kRows * kMaxRank; i += blockDim.x) {
        const int mi = i / kMaxRank, j = i % kMaxRank;
        float v = 0.f;
        if (m0 + mi < M && j < r)
            for (int ks = 0; ks < slices; ++ks) v += t[((size_t)ks * M + m0 + mi) * kMaxRank + j];
        st[mi][j] = v;
    }
    __syncthreads();
    const int n = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
    if (n >= N) return;
    const bool two = n + 1 < N;
    float acc[kRows][2];
#pragma unroll
    for (int i = 0; i < kRows; ++i) acc[i][0] = acc[i][1] = 0.f;
    if (vec) {
        // rows of B are multiples of 16 bytes and B is 16-byte aligned: 8 columns of both rows per pair of loads
        for (int j0 = 0; j0 < r; j0 += 8) {
            const uint4 q0 = __ldg(reinterpret_cast<const uint4*>(b + (size_t)n * r + j0));
            const uint4 q1 = two ? __ldg(reinterpret_cast<const uint4*>(b + (size_t)(n + 1) * r + j0)) : make_uint4(0, 0, 0, 0);
            const uint32_t w0[4] = {q0.x, q0.y, q0.z, q0.w}, w1[4] = {q1.x, q1.y, q1.z, q1.w};
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float b0 = __uint_as_float((c & 1) ? (w0[c >> 1] & 0xFFFF0000u) : (w0[c >> 1] << 16));
                const float b1 = __uint_as_float((c & 1) ? (w1[c >> 1] & 0xFFFF0000u) : (w1[c >> 1] << 16));
#pragma unroll
                for (int i = 0; i < kRows; ++i) {
                    acc[i][0] = fmaf(st[i][j0 + c], b0, acc[i][0]);
                    acc[i][1] = fmaf(st[i][j0 + c], b1, acc[i][1]);
                }
            }
        }
    } else {
        for (int j = 0; j < r; ++j) {
            const float b0 = __bfloat162float(b[(size_t)n * r + j]);
            const float b1 = two ? __bfloat162float(b[(size_t)(n + 1) * r + j]) : 0.f;
#pragma unroll
            for (int i = 0; i < kRows; ++i) {
                acc[i][0] = fmaf(st[i][j], b0, acc[i][0]);
                acc[i][1] = fmaf(st[i][j], b1, acc[i][1]);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kRows; ++i) {
        if (m0 + i >= M) break;
        __nv_bfloat16* out = y + (size_t)(m0 + i) * N + n;
        out[0] = __float2bfloat16_rn(fmaf(scale, acc[i][0], __bfloat162float(out[0])));
        if (two) out[1] = __float2bfloat16_rn(fmaf(scale, acc[i][1], __bfloat162float(out[1])));
    }
}

}  // namespace

// slices of K: enough blocks to occupy the GPU at small M, at least 256 columns each
static int lora_slices(int M, int K) {
    const int mb = (M + kRows - 1) / kRows;
    int s = (2 * num_sms() + mb - 1) / mb;
    if (s > kMaxSlices) s = kMaxSlices;
    if (s > K / 256) s = K / 256;
    return s < 1 ? 1 : s;
}

size_t lora_side_workspace(int M) { return (size_t)kMaxSlices * M * kMaxRank * sizeof(float); }

bool lora_side_supported(int M, int N, int K, int r) { return M >= 1 && N >= 1 && K >= 2 && K % 2 == 0 && r >= 1 && r <= kMaxRank; }

qil_status launch_lora_side_add(const void* x, const void* a, const void* b, void* y, int M, int N, int K, int r, float scale,
                                void* ws, cudaStream_t st) {
    float* t = reinterpret_cast<float*>(ws);
    const unsigned mb = (unsigned)((M + kRows - 1) / kRows);
    const int slices = lora_slices(M, K);
    const int slice = ((K + slices - 1) / slices + 1) & ~1;
    lora_down_kernel<<<dim3(mb, (unsigned)slices), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(x),
                                                                 reinterpret_cast<const __nv_bfloat16*>(a), t, M, K, r, slice);
    const int threads = N >= 8192 ? 256 : 64;   // (a thread owns two outputs: small N still gets many blocks)
    const dim3 grid((unsigned)((N + 2 * threads - 1) / (2 * threads)), mb);
    lora_up_add_kernel<<<grid, threads, 0, st>>>(t, reinterpret_cast<const __nv_bfloat16*>(b), reinterpret_cast<__nv_bfloat16*>(y), M, N, r, scale, slices,
                                                 ((r & 7) == 0 && reinterpret_cast<uintptr_t>(b) % 16 == 0) ? 1 : 0);
    return launch_status();
}

}  // namespace qil
