// W4A4 and W8A8 integer GEMMs (the compute-bound driving-policy deployment of the paper,
// Sec. 5.1 / Sec. 5.4, Table "CILRS performance"): acc = qx . qw^T in int32,
// y = bf16(float(acc) * sx[m] * sw[n]), on the 5th-generation tensor cores (tcgen05.mma kind::i8,
// accumulators in tensor memory).  The text below describes the 4-bit operands; with 8-bit operands
// (one signed byte per element) a step is 64 input channels, the bytes are stored as they are and
// the accumulator is the sum itself.
//
// A CTA computes a 128 (tokens) x 64 (output channels) tile.  Per step of 128 input
// channels its four loader warps read the packed nibbles of both operands from global
// memory (the operands of this workload stay in L2), split them into signed bytes and store
// them to shared memory in the tensor core's K-major layout without swizzle (8 rows x 16
// bytes per core matrix; K-adjacent core matrices `rows x 16` bytes apart, 8-row groups 128
// bytes apart).  One thread issues four tcgen05.mma (128 x 64 x 32) per step; a
// tcgen05.commit hands the shared-memory stage back to the loaders.  After the last step the
// same four warps read the accumulators (tcgen05.ld), rescale and store bf16.
//
// Unpacking: for a packed word w, (w << 4) & 0xF0F0F0F0 holds nibbles 0,2,4,6 and
// w & 0xF0F0F0F0 holds nibbles 1,3,5,7, each as a signed byte equal to 16 x the int4 value
// (the nibble is the byte's high half, so its sign bit is the byte's sign bit).  Both
// operands are scaled by 16, the int32 accumulator is exactly 256 x the true sum
// (|acc| <= 64 K, so 256 |acc| < 2^31 for K <= 131072) and is shifted back.  The order of k
// inside a word differs from memory order, identically for both operands, which leaves the
// sum unchanged.
#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kTileM = 128, kTileN = 64;
constexpr int kStepBytes = 64;  // operand bytes per row and step: 128 four-bit or 64 eight-bit elements
constexpr int kStages = 3;
// Operand tiles in shared memory: one byte per element after the split, K-major core matrices (8 rows x 16 bytes).
// The K-adjacent core matrices lie 16 bytes further apart than they are long: the four lanes that hold the four
// 16-byte pieces of one packed row then store to different banks.
constexpr int kALbo = kTileM * 16 + 16, kBLbo = kTileN * 16 + 16;
constexpr int kAStage = 8 * kALbo;  // (sized for the 8 chunks of a 4-bit step; an 8-bit step uses 4)
constexpr int kBStage = 8 * kBLbo;
constexpr int kPre = 2;                   // steps whose global loads are in flight per loader thread
constexpr int kThreads = 160;             // 4 loader / epilogue warps + the MMA warp
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
// Bounded wait: false when the limit ran out (the caller then stops issuing work).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
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
// D[128 x 64] (+)= A[128 x 32 s8, shared memory] * B[64 x 32 s8, shared memory]^T, int32 accumulate
__device__ __forceinline__ void mma_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
    // instruction descriptor: D = s32 (2 at bit 4), A = s8 (1 at bit 7), B = s8 (1 at bit 10), both K-major,
    // N >> 3 at bit 17, M >> 4 at bit 24
    constexpr uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)kTileN >> 3) << 17) | (((uint32_t)kTileM >> 4) << 24);
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// rint(f / s) with the IEEE division of the specification, without paying for a division per element: the product
// with the reciprocal is within a few ulp of the quotient, so unless it lies that close to a rounding boundary
// (k + 0.5) it rounds to the same integer; the rare close calls (and anything not finite) take the true division.
// (The division primitive also leaves its fast path for a zero numerator, which is every other element after a ReLU:
// an epilogue of 64 divisions per thread then cost 10 us a launch.)
__device__ __forceinline__ float rint_div(float f, float s, float inv_s) {
    const float r = f * inv_s;
    const float dist = fabsf(fabsf(r - rintf(r)) - 0.5f);  // distance of r from the nearest k + 0.5
    if (dist > 1e-4f * fmaxf(fabsf(r), 1.0f) && fabsf(r) < 1e6f) return rintf(r);
    return rintf(__fdiv_rn(f, s));
}

// 32 packed codes (one uint4) -> 32 signed bytes (x16) = two 16-byte K chunks
__device__ __forceinline__ void split32(const uint4& w, uint4& c0, uint4& c1) {
    constexpr uint32_t m = 0xF0F0F0F0u;
    c0 = make_uint4((w.x << 4) & m, w.x & m, (w.y << 4) & m, w.y & m);
    c1 = make_uint4((w.z << 4) & m, w.z & m, (w.w << 4) & m, w.w & m);
}

// 3 x 3 convolution (stride 1, zero padding 1) read straight from the feature map, without a materialised im2col
// matrix: row m of the GEMM is pixel (b, h, w), column (3 kh + kw) C + c is channel c of pixel (h + kh - 1,
// w + kw - 1).  C = 0: a plain GEMM.  With a feature map every row has the tensor's static scale x_scale.
struct ConvGeom {
    int C, H, W;
    float x_scale;
};

template <int kBits>
__global__ void __launch_bounds__(kThreads, 1) w4a4_tc_kernel(const uint32_t* __restrict__ qx, const float* __restrict__ sx,
                                                             const uint32_t* __restrict__ qw, const float* __restrict__ sw,
                                                             __nv_bfloat16* __restrict__ y, int32_t* __restrict__ acc_out,
                                                             int M, int N, int K, int* __restrict__ status,
                                                             uint32_t* __restrict__ qy, float out_scale, int relu,
                                                             const ConvGeom cg) {
    // qy != null: instead of bf16 outputs the epilogue writes the next layer's int4 activations, quantised with the
    // static scale out_scale from the fp32 product (optionally after ReLU), packed 8 per word (needs N % 8 == 0)
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sa = smem;                                  // [kStages][kAStage]
    unsigned char* sb = smem + (size_t)kStages * kAStage;      // [kStages][kBStage]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sb + (size_t)kStages * kBStage);
    const uint32_t full0 = smem_u32(bars), free0 = smem_u32(bars + kStages), done0 = smem_u32(bars + 2 * kStages);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 1);
    float* sws = reinterpret_cast<float*>(tmem_slot + 2);  // [kTileN] weight scales of the tile
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kTileM, n0 = blockIdx.y * kTileN;
    constexpr int kStepK = kStepBytes * 8 / kBits;   // elements per step
    constexpr int kChunks = kStepK / 16;             // 16-byte K chunks of a step in shared memory
    const int steps = (K + kStepK - 1) / kStepK;
    const int row_words = K * kBits / 32;  // 32-bit words per operand row

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8 * s, 4);
            mbar_init(free0 + 8 * s, 1);
        }
        mbar_init(done0, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < kTileN) sws[tid] = (n0 + tid < N) ? sw[n0 + tid] : 0.f;
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTileN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (warp < 4) {
        // ---------------- loaders: lane = 16-byte piece tid % 4 (32 codes) of the step's 64 packed bytes of token rows
        // tid / 4 + 32 j (j < 4) and weight rows tid / 4 + 32 j (j < 2): four lanes read one row's bytes together ----------------
        const int r = tid;
        const bool a_row = m0 + r < M;  // (for the epilogue: thread r reads out accumulator row r)
        const int pq = tid & 3, pr = tid >> 2;
        const uint32_t* xa = qx + (size_t)m0 * row_words + 4 * pq;
        const uint32_t* wb = qw + (size_t)n0 * row_words + 4 * pq;
        uint4 pa[kPre][4], pb[kPre][2];
        // feature-map mode: the pixels of this thread's four rows
        int px_h[4], px_w[4];
        long long px_lin[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            px_h[j] = px_w[j] = 0;
            px_lin[j] = -1;
            if (cg.C > 0 && m0 + pr + 32 * j < M) {
                const int m = m0 + pr + 32 * j;
                px_w[j] = m % cg.W;
                px_h[j] = (m / cg.W) % cg.H;
                px_lin[j] = m;
            }
        }
        auto fetch = [&](uint4 (&da)[4], uint4 (&db)[2], int step) {  // packed words of one step (zeros beyond the matrix)
            const int w0 = step * (kStepBytes / 4);
            const bool in_k = w0 + 4 * pq < row_words;
            if (cg.C > 0) {
                // this thread's 16 bytes of the step lie inside one tap (C % 32 == 0)
                constexpr int kPerWord = 32 / kBits;
                const int k0 = (w0 + 4 * pq) * kPerWord, tap = k0 / cg.C, c0 = k0 - tap * cg.C;
                const int dh = tap / 3 - 1, dw = tap - (tap / 3) * 3 - 1;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int hh = px_h[j] + dh, ww = px_w[j] + dw;
                    const bool inside = in_k && px_lin[j] >= 0 && hh >= 0 && hh < cg.H && ww >= 0 && ww < cg.W;
                    da[j] = inside ? __ldg(reinterpret_cast<const uint4*>(qx + ((px_lin[j] + dh * cg.W + dw) * cg.C + c0) / kPerWord))
                                   : make_uint4(0, 0, 0, 0);
                }
            } else
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int row = pr + 32 * j;
                da[j] = (in_k && m0 + row < M) ? __ldg(reinterpret_cast<const uint4*>(xa + (size_t)row * row_words + w0))
                                               : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int row = pr + 32 * j;
                db[j] = (in_k && n0 + row < N) ? __ldg(reinterpret_cast<const uint4*>(wb + (size_t)row * row_words + w0))
                                               : make_uint4(0, 0, 0, 0);
            }
        };
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
#pragma unroll
            for (int j = 0; j < 4; ++j) pa[u][j] = make_uint4(0, 0, 0, 0);
            pb[u][0] = pb[u][1] = make_uint4(0, 0, 0, 0);
            if (u < steps) fetch(pa[u], pb[u], u);
        }
        for (int step0 = 0; ok && step0 < steps; step0 += kPre) {
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                const int step = step0 + u;
                if (step >= steps) break;
                const int s = step % kStages, use = step / kStages;
                ok = mbar_wait(free0 + 8 * s, (use & 1) ^ 1);  // the MMAs that read this stage last are complete
                if (!ok) break;
                // 4-bit: piece pq = K chunks 2 pq, 2 pq + 1 of the step; 8-bit: piece pq = chunk pq
                constexpr int kPer = kBits == 4 ? 2 : 1;
                unsigned char* a_st = sa + (size_t)s * kAStage + (size_t)(kPer * pq) * kALbo + (size_t)pr * 16;
                unsigned char* b_st = sb + (size_t)s * kBStage + (size_t)(kPer * pq) * kBLbo + (size_t)pr * 16;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if constexpr (kBits == 4) {
                        uint4 c0, c1;
                        split32(pa[u][j], c0, c1);
                        *reinterpret_cast<uint4*>(a_st + (size_t)j * (32 * 16)) = c0;
                        *reinterpret_cast<uint4*>(a_st + (size_t)j * (32 * 16) + kALbo) = c1;
                    } else {
                        *reinterpret_cast<uint4*>(a_st + (size_t)j * (32 * 16)) = pa[u][j];
                    }
                }
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    if constexpr (kBits == 4) {
                        uint4 c0, c1;
                        split32(pb[u][j], c0, c1);
                        *reinterpret_cast<uint4*>(b_st + (size_t)j * (32 * 16)) = c0;
                        *reinterpret_cast<uint4*>(b_st + (size_t)j * (32 * 16) + kBLbo) = c1;
                    } else {
                        *reinterpret_cast<uint4*>(b_st + (size_t)j * (32 * 16)) = pb[u][j];
                    }
                }
                if (step + kPre < steps) fetch(pa[u], pb[u], step + kPre);  // kPre steps stay in flight
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMAs read through the async proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(full0 + 8 * s);
            }
        }
        // ---------------- epilogue: thread r = accumulator row r ----------------
        if (ok) ok = mbar_wait(done0, 0);
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int m = m0 + r;
            const float sxm = a_row ? (cg.C > 0 ? cg.x_scale : sx[m]) : 0.f;
            const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;
            const bool vec = (N % 8) == 0;  // rows of y are then 16-byte aligned pieces of 8 outputs
            const float inv_out = __frcp_rn(out_scale);
#pragma unroll 1
            for (int c0 = 0; c0 < kTileN; c0 += 16) {
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
                for (int h = 0; h < 2; ++h) {  // 8 outputs = one 16-byte piece of the row
                    const int nb = n0 + c0 + 8 * h;
                    if (nb >= N) continue;
                    int a[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) a[j] = kBits == 4 ? ((int)d[8 * h + j] >> 8) : (int)d[8 * h + j];  // (4-bit: exact, the accumulator is a multiple of 256)
                    if (qy) {
                        uint32_t word = 0;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            float v = __fmul_rn((float)a[j], __fmul_rn(sxm, sws[c0 + 8 * h + j]));
                            if (relu) v = fmaxf(v, 0.f);
                            const int q = (int)fminf(fmaxf(rint_div(v, out_scale, inv_out), -8.f), 7.f);
                            word |= ((uint32_t)q & 0xFu) << (4 * j);
                        }
                        qy[(size_t)m * (N >> 3) + (nb >> 3)] = word;
                    } else if (vec) {
                        uint32_t pk[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const __nv_bfloat162 v = __floats2bfloat162_rn((float)a[2 * j] * (sxm * sws[c0 + 8 * h + 2 * j]),
                                                                           (float)a[2 * j + 1] * (sxm * sws[c0 + 8 * h + 2 * j + 1]));
                            pk[j] = *reinterpret_cast<const uint32_t*>(&v);
                        }
                        *reinterpret_cast<uint4*>(y + (size_t)m * N + nb) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        if (acc_out) {
                            *reinterpret_cast<int4*>(acc_out + (size_t)m * N + nb) = make_int4(a[0], a[1], a[2], a[3]);
                            *reinterpret_cast<int4*>(acc_out + (size_t)m * N + nb + 4) = make_int4(a[4], a[5], a[6], a[7]);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (nb + j < N) {
                                if (acc_out) acc_out[(size_t)m * N + nb + j] = a[j];
                                y[(size_t)m * N + nb + j] = __float2bfloat16_rn((float)a[j] * (sxm * sws[c0 + 8 * h + j]));
                            }
                    }
                }
            }
        }
    } else if (lane == 0) {
        // ---------------- MMA issuer ----------------
        for (int step = 0; step < steps; ++step) {
            const int s = step % kStages, use = step / kStages;
            ok = mbar_wait(full0 + 8 * s, use & 1);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = smem_u32(sa + (size_t)s * kAStage), b_addr = smem_u32(sb + (size_t)s * kBStage);
#pragma unroll
            for (int i = 0; i < kChunks / 2; ++i)  // K = 32 each: chunks 2i, 2i + 1
                mma_i8_ss(tmem, smem_desc(a_addr + 2 * i * kALbo, kALbo, 128), smem_desc(b_addr + 2 * i * kBLbo, kBLbo, 128),
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
    if (warp == 4) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTileN));
}

constexpr size_t kSmemBytes = (size_t)kStages * (kAStage + kBStage) + (2 * kStages + 1) * 8 + 8 + kTileN * 4 + 8;

}  // namespace

// The first int of the workspace receives QIL_ERR_TIMEOUT if a bounded device-side wait runs out.
size_t w4a4_workspace(int M, int N, int K) {
    (void)M; (void)N; (void)K;
    return 16;
}

// bits = 4: packed nibbles [M][K/8], [N][K/8]; bits = 8: signed bytes [M][K], [N][K]
qil_status launch_w4a4(const void* qx, const float* sx, const void* qw, const float* sw, void* y, int32_t* acc_out, int M,
                       int N, int K, int bits, void* ws, size_t ws_bytes, cudaStream_t st, uint32_t* qy, float out_scale,
                       int relu, int conv_C, int conv_H, int conv_W, float x_scale) {
    ConvGeom cg;
    cg.C = conv_C; cg.H = conv_H; cg.W = conv_W; cg.x_scale = x_scale;
    if (ws == nullptr || ws_bytes < 16) return QIL_ERR_WORKSPACE;
    const dim3 grid((M + kTileM - 1) / kTileM, (N + kTileN - 1) / kTileN);
    cudaError_t e;
    if (bits == 8) {
        e = cudaFuncSetAttribute(w4a4_tc_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e == cudaSuccess)
            w4a4_tc_kernel<8><<<grid, kThreads, kSmemBytes, st>>>(reinterpret_cast<const uint32_t*>(qx), sx, reinterpret_cast<const uint32_t*>(qw), sw,
                                                                 reinterpret_cast<__nv_bfloat16*>(y), acc_out, M, N, K, reinterpret_cast<int*>(ws), nullptr, 1.f, 0, cg);
    } else {
        e = cudaFuncSetAttribute(w4a4_tc_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e == cudaSuccess)
            w4a4_tc_kernel<4><<<grid, kThreads, kSmemBytes, st>>>(reinterpret_cast<const uint32_t*>(qx), sx, reinterpret_cast<const uint32_t*>(qw), sw,
                                                                 reinterpret_cast<__nv_bfloat16*>(y), acc_out, M, N, K, reinterpret_cast<int*>(ws), qy, out_scale, relu, cg);
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    return launch_status();
}

}  // namespace qil
