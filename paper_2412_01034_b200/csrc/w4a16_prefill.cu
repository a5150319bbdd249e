// Weight-only 4-bit linear at prefill length (the prompt / vision-token stage of the paper's OpenVLA deployment,
// App. A.4.2; M tokens, typically 280): a tensor-bound GEMM on tcgen05.mma kind::f16 (bf16 operands, fp32
// accumulators in tensor memory over the whole K).
//
// A CTA computes a 128 (tokens) x 128 (output features) tile.  Per step of 64 input features
//   * four weight-loader warps read 64 packed codes of one weight row per thread, turn them into bf16 with a
//     mask/or (0x4300 | q = 128 + q, exact), subtract 128 + z (exact in bf16: integers below 256) and multiply by
//     the group's scale (one rounding per weight; the scale itself is rounded from fp16 to bf16 once per group),
//   * four activation-loader warps read the activations (bf16) of one token row per thread,
// each thread keeping the global loads of three steps in flight (the step time is otherwise one L2 / DRAM
// latency), and store both as K-major operands without swizzle (8 rows x 16 bytes per core matrix).  Inside every 8-element
// piece the order is {0,4,1,5,2,6,3,7} for both operands - the order in which a packed word gives up its nibble
// pairs - which leaves the dot product unchanged.  One thread issues four tcgen05.mma (128 x 128 x 16) per step;
// tcgen05.commit recycles the shared-memory stage.  The activation-loader warps then read the accumulators, round to bf16
// and store 16-byte pieces.  Canonical packed layout only.
#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kTile = 128, kStepK = 64, kStages = 4;
constexpr int kOpStage = kTile * kStepK * 2;  // bytes of one weight operand tile (bf16)
// The activation tile is loaded by eight lanes per token row (one 128-byte line per row and step) and stored with
// the K-adjacent core matrices 16 bytes further apart than they are long, so that those eight lanes hit different banks.
constexpr int kLboA = kTile * 16 + 16;
constexpr int kOpStageA = 8 * kLboA;
constexpr int kThreads = 288;  // 4 activation loader warps, 4 weight loader warps, 1 MMA warp
constexpr int kPre = 3;        // steps whose global loads are in flight per loader thread
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {  // bounded: false when the limit ran out
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        if (t - t0 > kWaitLimitNs) return false;
    }
}
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of this architecture
    return d;
}
// D[128 x 128] (+)= A[128 x 16 bf16, shared memory] * B[128 x 16 bf16, shared memory]^T, fp32 accumulate
__device__ __forceinline__ void mma_bf16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
    // instruction descriptor: D = f32 (1 at bit 4), A = bf16 (1 at bit 7), B = bf16 (1 at bit 10), both K-major,
    // N >> 3 at bit 17, M >> 4 at bit 24
    constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)kTile >> 3) << 17) | (((uint32_t)kTile >> 4) << 24);
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// One packed word (8 codes) -> 8 dequantised bf16 in the order {0,4,1,5,2,6,3,7}.
// off = bf16x2 {128 + z, 128 + z}, sc = bf16x2 {s, s}
__device__ __forceinline__ uint4 dequant8(uint32_t w, __nv_bfloat162 off, __nv_bfloat162 sc) {
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t v = ((w >> (4 * j)) & 0x000F000Fu) | 0x43004300u;  // {128 + q_j, 128 + q_(j+4)}, exact
        const __nv_bfloat162 d = __hmul2(__hsub2(*reinterpret_cast<const __nv_bfloat162*>(&v), off), sc);
        o[j] = *reinterpret_cast<const uint32_t*>(&d);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}
// 8 bf16 in memory order -> the order {0,4,1,5,2,6,3,7}
__device__ __forceinline__ uint4 permute8(const uint4& x) {
    return make_uint4(__byte_perm(x.x, x.z, 0x5410), __byte_perm(x.x, x.z, 0x7632), __byte_perm(x.y, x.w, 0x5410),
                      __byte_perm(x.y, x.w, 0x7632));
}

__global__ void __launch_bounds__(kThreads, 1) w4a16_prefill_kernel(const __nv_bfloat16* __restrict__ x,
                                                                   const uint32_t* __restrict__ qw,
                                                                   const __half* __restrict__ scales,
                                                                   const __half* __restrict__ zeros,
                                                                   __nv_bfloat16* __restrict__ y, int M, int N, int K, int G,
                                                                   int* __restrict__ status) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sa = smem;                                   // [kStages][kOpStageA] activations
    unsigned char* sb = smem + (size_t)kStages * kOpStageA;     // [kStages][kOpStage] weights
    uint64_t* bars = reinterpret_cast<uint64_t*>(sb + (size_t)kStages * kOpStage);
    const uint32_t full0 = smem_u32(bars), free0 = smem_u32(bars + kStages), done0 = smem_u32(bars + 2 * kStages);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * kTile, m0 = blockIdx.y * kTile;
    const int steps = K / kStepK, ng = K / G;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8 * s, 8);
            mbar_init(free0 + 8 * s, 1);
        }
        mbar_init(done0, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTile));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (warp < 4) {
        // ---------------- activation loaders: lane = 16-byte piece tid % 8 of token rows tid / 8 + 16 j ----------------
        const int r = tid;
        const bool a_row = m0 + r < M;  // (for the epilogue: thread r reads out token row m0 + r)
        const int pc = tid & 7, pr = tid >> 3;
        const __nv_bfloat16* xa = x + (size_t)m0 * K + 8 * pc;
        uint4 pa[kPre][8];
        auto fetch = [&](uint4 (&dst)[8], int step) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int row = pr + 16 * j;
                dst[j] = (m0 + row < M) ? __ldg(reinterpret_cast<const uint4*>(xa + (size_t)row * K + step * kStepK))
                                        : make_uint4(0, 0, 0, 0);
            }
        };
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
#pragma unroll
            for (int j = 0; j < 8; ++j) pa[u][j] = make_uint4(0, 0, 0, 0);
            if (u < steps) fetch(pa[u], u);
        }
        for (int step0 = 0; ok && step0 < steps; step0 += kPre) {
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                const int step = step0 + u;
                if (step >= steps) break;
                const int s = step % kStages, use = step / kStages;
                ok = mbar_wait(free0 + 8 * s, (use & 1) ^ 1);  // the MMAs that read this stage last are complete
                if (!ok) break;
                unsigned char* a_st = sa + (size_t)s * kOpStageA + (size_t)pc * kLboA + (size_t)pr * 16;
#pragma unroll
                for (int j = 0; j < 8; ++j) *reinterpret_cast<uint4*>(a_st + (size_t)j * (16 * 16)) = permute8(pa[u][j]);
                if (step + kPre < steps) fetch(pa[u], step + kPre);  // kPre steps stay in flight
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMAs read through the async proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(full0 + 8 * s);
            }
        }
        // ---------------- epilogue: thread r = token row m0 + r ----------------
        if (ok) ok = mbar_wait(done0, 0);
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;
            const bool vec = (N % 8) == 0;
            __nv_bfloat16* yr = y + (size_t)(m0 + r) * N;
#pragma unroll 1
            for (int c0 = 0; c0 < kTile; c0 += 16) {
                uint32_t d[16];
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                    : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]), "=r"(d[8]),
                      "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15])
                    : "r"(tmem + lane_base + (uint32_t)c0));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int j = 0; j < 16; ++j) asm volatile("" : "+r"(d[j]));
                if (!a_row) continue;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int nb = n0 + c0 + 8 * h;
                    if (nb >= N) continue;
                    if (vec) {
                        uint32_t pk[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(d[8 * h + 2 * j]), __uint_as_float(d[8 * h + 2 * j + 1]));
                            pk[j] = *reinterpret_cast<const uint32_t*>(&v);
                        }
                        *reinterpret_cast<uint4*>(yr + nb) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (nb + j < N) yr[nb + j] = __float2bfloat16_rn(__uint_as_float(d[8 * h + j]));
                    }
                }
            }
        }
    } else if (warp < 8) {
        // ---------------- weight loaders: thread r owns weight row n0 + r ----------------
        const int r = tid - 128;
        const bool b_row = n0 + r < N;
        const uint32_t* wb = qw + (size_t)(n0 + (b_row ? r : 0)) * (K >> 3);
        const __half* sr = scales + (size_t)(n0 + (b_row ? r : 0)) * ng;
        const __half* zr = zeros + (size_t)(n0 + (b_row ? r : 0)) * ng;
        uint4 pb[kPre][2];
        __half ps[kPre], pz[kPre];
        auto fetch = [&](uint4 (&dst)[2], __half& s_, __half& z_, int step) {
            const int k0 = step * kStepK;
#pragma unroll
            for (int q = 0; q < 2; ++q)
                dst[q] = b_row ? __ldg(reinterpret_cast<const uint4*>(wb + (k0 >> 3) + 4 * q)) : make_uint4(0, 0, 0, 0);
            s_ = b_row ? sr[k0 / G] : __float2half(0.f);
            z_ = b_row ? zr[k0 / G] : __float2half(0.f);
        };
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
            pb[u][0] = pb[u][1] = make_uint4(0, 0, 0, 0);
            ps[u] = pz[u] = __float2half(0.f);
            if (u < steps) fetch(pb[u], ps[u], pz[u], u);
        }
        for (int step0 = 0; ok && step0 < steps; step0 += kPre) {
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                const int step = step0 + u;
                if (step >= steps) break;
                const int s = step % kStages, use = step / kStages;
                ok = mbar_wait(free0 + 8 * s, (use & 1) ^ 1);
                if (!ok) break;
                unsigned char* b_st = sb + (size_t)s * kOpStage + (size_t)r * 16;
                const float zf = b_row ? __half2float(pz[u]) + 128.f : 128.f;
                const float sf = b_row ? __half2float(ps[u]) : 0.f;
                const __nv_bfloat162 off = __float2bfloat162_rn(zf), sc = __float2bfloat162_rn(sf);
                const uint32_t w[8] = {pb[u][0].x, pb[u][0].y, pb[u][0].z, pb[u][0].w, pb[u][1].x, pb[u][1].y, pb[u][1].z, pb[u][1].w};
#pragma unroll
                for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(b_st + (size_t)c * (kTile * 16)) = dequant8(w[c], off, sc);
                if (step + kPre < steps) fetch(pb[u], ps[u], pz[u], step + kPre);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(full0 + 8 * s);
            }
        }
    } else if (lane == 0) {
        // ---------------- MMA issuer ----------------
        constexpr uint32_t kLbo = kTile * 16;  // K-adjacent core matrices of the weight operand
        for (int step = 0; step < steps; ++step) {
            const int s = step % kStages, use = step / kStages;
            ok = mbar_wait(full0 + 8 * s, use & 1);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = smem_u32(sa + (size_t)s * kOpStageA), b_addr = smem_u32(sb + (size_t)s * kOpStage);
#pragma unroll
            for (int i = 0; i < 4; ++i)  // K = 16 each: 16-byte pieces 2i, 2i + 1
                mma_bf16_ss(tmem, smem_desc(a_addr + 2 * i * kLboA, kLboA, 128), smem_desc(b_addr + 2 * i * kLbo, kLbo, 128),
                            (step > 0 || i > 0) ? 1u : 0u);
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(free0 + 8 * s) : "memory");
        }
        // all MMAs of this thread are complete when this arrival happens (also needed before tensor memory is released)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(done0) : "memory");
        unsigned long long t0, t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        while (!mbar_try_wait(done0, 0)) {
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
            if (t - t0 > kWaitLimitNs) { ok = false; break; }
        }
    }
    if (!ok && status) atomicOr(status, (int)QIL_ERR_TIMEOUT);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 8) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTile));
}

constexpr size_t kSmemBytes = (size_t)kStages * (kOpStage + kOpStageA) + (2 * kStages + 1) * 8 + 16;

}  // namespace

bool w4a16_prefill_supported(int M, int N, int K, int G, qil_layout layout) {
    return layout == QIL_LAYOUT_CANONICAL && M > 16 && N >= 1 && K % kStepK == 0 && G % kStepK == 0 && K % G == 0;
}

// ws (optional): its first int receives QIL_ERR_TIMEOUT if a bounded device-side wait runs out.
qil_status launch_w4a16_prefill(const void* x, const uint32_t* qw, const void* scales, const void* zeros, void* y, int M,
                                int N, int K, int G, void* ws, cudaStream_t st) {
    if (cudaFuncSetAttribute(w4a16_prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    const dim3 grid((N + kTile - 1) / kTile, (M + kTile - 1) / kTile);
    w4a16_prefill_kernel<<<grid, kThreads, kSmemBytes, st>>>(reinterpret_cast<const __nv_bfloat16*>(x), qw,
                                                            reinterpret_cast<const __half*>(scales),
                                                            reinterpret_cast<const __half*>(zeros),
                                                            reinterpret_cast<__nv_bfloat16*>(y), M, N, K, G,
                                                            reinterpret_cast<int*>(ws));
    return launch_status();
}

}  // namespace qil
