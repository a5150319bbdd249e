// Weight-only linears at prefill length (the prompt / vision-token stage of the paper's OpenVLA deployment,
// App. A.4.2; M tokens, typically 280; 4-bit weights, and the 8-bit weights of the INT8 deployment point of
// Sec. 5.4): a GEMM on tcgen05.mma kind::f16 (bf16 operands, fp32 accumulators in tensor memory).
//
// A CTA computes 256 output features x up to 144 tokens over a range of K.  The weights are the M side of the
// MMAs (two accumulators of 128 features), the tokens the N side, so that every weight of the tile is dequantised
// once for all its tokens.  Per step of 64 input features
//   * one thread copies the 144 x 64 activation tile with one bulk tensor copy (128-byte swizzle; rows beyond M
//     arrive as zeros),
//   * another copies the packed 256 x 64 weight tile with one bulk tensor copy into a ring that runs eight steps
//     ahead (the weights are the only operand that comes from HBM; loading them thread by thread, 16 or 32 bytes
//     of a different row each, measured several times slower),
//   * eight dequantising warps (thread = weight row) turn 64 codes of their row into bf16 - 128 + q by a byte
//     permute, a multiply and a mask (exact), minus 128 + z (exact: integers below 256), times the group's scale
//     rounded to bf16 (one rounding per weight) - and store them as the K-major operand in the 128-byte swizzle.
//     The scales and zero points of two groups come with one 32-bit load each, four steps ahead: a 2-byte gather
//     over 256 rows per step was the slowest thing in the loop,
//   * one thread issues eight tcgen05.mma (128 x 144 x 16); tcgen05.commit recycles the stages (three).
// The dequantising warps then read the accumulators (lane = feature) and write bf16 outputs, or, when K is split
// over several CTAs to fill the GPU, fp32 partial tiles to the workspace; the last CTA of a tile to arrive (an
// atomic counter, nobody waits) adds the partial tiles in split order, so the result does not depend on timing.
// A stage of a ring is released only after the data read from it has been used (releasing it once the loads were
// issued let the next copy overwrite words still in flight: seen as one warp's rows going wrong now and then).
// Canonical layout only.  Every wait is bounded and polls; when one runs out QIL_ERR_TIMEOUT is recorded.
#include <cuda.h>

#include <mutex>

#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kTileF = 256, kHalfF = 128, kStepK = 64, kStages = 3, kBStages = 3, kMaxTN = 144;
constexpr int kWRingBytes = 65536;                // ring of packed weight tiles (256 rows x 64 codes each)
constexpr int kAHalf = kHalfF * kStepK * 2;       // one half of the weight operand tile (bf16): 8 KiB
constexpr int kAStage = 2 * kAHalf;
constexpr int kBStage = kMaxTN * kStepK * 2;      // activation tile: 9 KiB (a multiple of 1024)
constexpr int kThreads = 352;                     // activation copy warp, MMA warp, 8 dequantising / read-out warps, weight copy warp
constexpr int kDqWarps = 8;
constexpr int kMetaPre = 8;                       // steps by which a dequantising thread's scale / zero loads run ahead
constexpr int kTmemCols = 512;
constexpr int kCounterBytes = 16384;              // tile counters at the start of the scratch (same place as the skinny kernel's)
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct PrefillParams {
    const void* qw;
    const __half* scales;
    const __half* zeros;
    __nv_bfloat16* y;
    int M, N, K, G;
    int g_shift;   // log2(G / 64) when that is a power of two, else -1
    int pair_meta; // groups of 128 columns, an even number of them per row, K % 256 == 0: scales are loaded two groups at a time
    int TN;        // tokens per tile (multiple of 16, <= 144)
    int split;     // CTAs along K per tile
    int* status;
    int* counters;
    float* partials;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
// Bounded wait: false when the limit ran out.  The wait polls (test_wait) instead of letting the hardware suspend the
// thread (try_wait): a suspended thread wakes up about a microsecond after the phase completes, and in a pipeline
// whose rings are full every hand-over is such a wake-up - measured: one step per microsecond whatever the work.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_test_wait(bar, parity)) return true;
    unsigned long long t0 = 0, t;
#pragma unroll 1
    for (uint32_t i = 0;; ++i) {
        if (mbar_test_wait(bar, parity)) return true;
        if ((i & 63u) == 0u) {
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
            if (i == 0u) t0 = t;
            else if (t - t0 > kWaitLimitNs) return false;
        }
    }
}
// 2-D bulk tensor copy global -> shared (no multicast), completion on an mbarrier
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
                 : "memory");
}
// shared-memory operand descriptor, K-major, rows of 128 bytes in the 128-byte swizzle (tiles aligned to 1024 bytes)
__device__ __forceinline__ uint64_t desc_swizzle128(uint32_t addr) {
    uint64_t d = (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)1 << 16;                        // (unused with a swizzle)
    d |= (uint64_t)(1024u >> 4) << 32;             // 8 rows of 128 bytes
    d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                        // 128-byte swizzle
    return d;
}
// D[128 x N] (+)= A[128 x 16 bf16] * B[N x 16 bf16]^T, fp32 accumulate, operands in shared memory
__device__ __forceinline__ void mma_bf16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// bf16x2 {(a - off) * sc, (b - off) * sc} of two exact bf16x2 inputs
__device__ __forceinline__ uint32_t scale2(uint32_t v, __nv_bfloat162 off, __nv_bfloat162 sc) {
    const __nv_bfloat162 d = __hmul2(__hsub2(*reinterpret_cast<const __nv_bfloat162*>(&v), off), sc);
    return *reinterpret_cast<const uint32_t*>(&d);
}
// One packed word (8 four-bit codes) -> 8 dequantised bf16 in memory order.  off = {128 + z}, sc = {s}.
// Byte j of the word holds codes 2j (low nibble) and 2j + 1: a byte permute isolates it, a multiply by 0x1001 copies
// it 12 bits up (the two copies do not overlap), and one logic operation keeps nibble 2j in the low half-word and
// nibble 2j + 1 in the high one under the bf16 pattern 0x4300 (= 128 + q, exact).  Two operations on the integer
// pipe per pair of weights; the multiply runs on the floating-point pipe.
__device__ __forceinline__ uint4 dequant8_w4(uint32_t w, __nv_bfloat162 off, __nv_bfloat162 sc) {
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t b = __byte_perm(w, 0u, 0x4440u | (uint32_t)j);  // byte j, zero-extended
        const uint32_t v = ((b * 0x1001u) & 0x000F000Fu) | 0x43004300u;
        o[j] = scale2(v, off, sc);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}
// Four 8-bit codes -> 4 dequantised bf16.  offf = 2^23 + z (fp32), sc = {s}.
__device__ __forceinline__ uint2 dequant4_w8(uint32_t w, float offf, __nv_bfloat162 sc) {
    uint32_t o[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        // 2^23 + code as fp32 bits (a byte permute puts the code under 0x4B0000), minus 2^23 + z: the exact integer
        // code - z, which bf16 holds exactly (|.| <= 255)
        const float a = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7440u | (uint32_t)(2 * j))) - offf;
        const float b = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7440u | (uint32_t)(2 * j + 1))) - offf;
        const __nv_bfloat162 d = __hmul2(__floats2bfloat162_rn(a, b), sc);
        o[j] = *reinterpret_cast<const uint32_t*>(&d);
    }
    return make_uint2(o[0], o[1]);
}

template <int kBits>
__global__ void __launch_bounds__(kThreads, 1) w4a16_prefill_kernel(const __grid_constant__ CUtensorMap tmap_x,
                                                                   const __grid_constant__ CUtensorMap tmap_w,
                                                                   const PrefillParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // (the swizzled activation tiles need 1024-byte alignment)
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* sb = smem;                                  // [kStages][kBStage] activations
    unsigned char* sa = smem + (size_t)kBStages * kBStage;     // [kStages][kAStage] weights
    constexpr int kWStage = kTileF * kStepK * kBits / 8;       // packed weight tile: 8 KiB (4-bit), 16 KiB (8-bit)
    constexpr int kWStages = kWRingBytes / kWStage;
    unsigned char* sw = sa + (size_t)kStages * kAStage;        // [kWStages][256 rows][kStepK * kBits / 8 bytes]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sw + kWRingBytes);
    const uint32_t full_a0 = smem_u32(bars), free0 = smem_u32(bars + kStages), done0 = smem_u32(bars + 2 * kStages);
    const uint32_t full_b0 = smem_u32(bars + 2 * kStages + 1), free_b0 = smem_u32(bars + 2 * kStages + 1 + kBStages);
    uint64_t* wbars = bars + 2 * kStages + 1 + 2 * kBStages;
    const uint32_t full_w0 = smem_u32(wbars), free_w0 = smem_u32(wbars + kWStages);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(wbars + 2 * kWStages);
    int* is_last = reinterpret_cast<int*>(tmem_slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * kTileF, m0 = blockIdx.y * p.TN;
    const int steps_all = p.K / kStepK;
    const int z = blockIdx.z;
    // (with pair_meta the splits begin at multiples of 4 steps = two groups of 128 columns)
    const int s_unit = p.pair_meta ? 4 : 1;
    const int s_begin = (int)((long long)(steps_all / s_unit) * z / p.split) * s_unit,
              s_end = (int)((long long)(steps_all / s_unit) * (z + 1) / p.split) * s_unit;
    const int steps = s_end - s_begin;
    const int ng = p.K / p.G;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_a0 + 8 * s, kDqWarps);   // the dequantising warps
            mbar_init(free0 + 8 * s, 1);     // the commit of the MMAs that read the stage
        }
        for (int s = 0; s < kBStages; ++s) {
            mbar_init(full_b0 + 8 * s, 1);   // the copy (transaction bytes)
            mbar_init(free_b0 + 8 * s, 1);   // the commit of the MMAs that read the stage
        }
        mbar_init(done0, 1);
        for (int s = 0; s < kWStages; ++s) {
            mbar_init(full_w0 + 8 * s, 1);   // the copy (transaction bytes)
            mbar_init(free_w0 + 8 * s, kDqWarps);   // the dequantising warps have read the tile
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (warp == 0) {
        // ---------------- activation copies ----------------
        if (lane == 0) {
            int issued = 0;
            for (int i = 0; i < steps; ++i, ++issued) {
                const int s = i % kBStages, use = i / kBStages;
                ok = mbar_wait(free_b0 + 8 * s, (use & 1) ^ 1);  // the MMAs that read this stage last are complete
                if (!ok) break;
                mbar_expect_tx(full_b0 + 8 * s, (uint32_t)p.TN * kStepK * 2);
                tma_load_2d(smem_u32(sb + (size_t)s * kBStage), &tmap_x, (s_begin + i) * kStepK, m0, full_b0 + 8 * s);
            }
            // no copy may still be in flight when the CTA retires (this wait also holds after a time-out elsewhere)
            for (int back = 0; back < kBStages && back < issued; ++back) {
                const int i = issued - 1 - back;
                (void)mbar_wait(full_b0 + 8 * (i % kBStages), (i / kBStages) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)p.TN >> 3) << 17) | (((uint32_t)kHalfF >> 4) << 24);
            for (int i = 0; i < steps; ++i) {
                const int s = i % kStages, use = i / kStages, bs = i % kBStages, buse = i / kBStages;
                ok = mbar_wait(full_a0 + 8 * s, use & 1) && mbar_wait(full_b0 + 8 * bs, buse & 1);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(sa + (size_t)s * kAStage), b_addr = smem_u32(sb + (size_t)bs * kBStage);
#pragma unroll
                for (int k = 0; k < kStepK / 16; ++k) {  // K = 16 each: 32 bytes of a swizzled row of either operand
                    const uint64_t bd = desc_swizzle128(b_addr + 32 * k);
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        mma_bf16_ss(tmem + 256 * h, desc_swizzle128(a_addr + h * kAHalf + 32 * k), bd, idesc, (i > 0 || k > 0) ? 1u : 0u);
                }
                tc_commit(free0 + 8 * s);
                tc_commit(free_b0 + 8 * bs);
            }
            // all MMAs of this thread are complete when this arrival happens (also needed before tensor memory is released)
            tc_commit(done0);
            if (!mbar_wait(done0, 0)) ok = false;
        }
    } else if (warp == 2 + kDqWarps) {
        // ---------------- packed weight copies (rows beyond N arrive as zeros) ----------------
        if (lane == 0) {
            int issued = 0;
            for (int i = 0; i < steps; ++i, ++issued) {
                const int s = i % kWStages, use = i / kWStages;
                ok = mbar_wait(free_w0 + 8 * s, (use & 1) ^ 1);
                if (!ok) break;
                mbar_expect_tx(full_w0 + 8 * s, (uint32_t)kWStage);
                tma_load_2d(smem_u32(sw + (size_t)s * kWStage), &tmap_w, (s_begin + i) * (kStepK * kBits / 8), n0, full_w0 + 8 * s);
            }
            for (int back = 0; back < kWStages && back < issued; ++back) {
                const int i = issued - 1 - back;
                (void)mbar_wait(full_w0 + 8 * (i % kWStages), (i / kWStages) & 1);
            }
        }
    } else {
        // ---------------- dequantising warps: a thread owns half a step (32 codes) of weight row n0 + r ----------------
        const int r = tid - 64;
        const int h = r >> 7, rr = r & 127;
        const bool w_row = n0 + r < p.N;
        const size_t nrow = (size_t)(n0 + (w_row ? r : 0));
        const __half* sr = p.scales + nrow * ng;
        const __half* zr = p.zeros + nrow * ng;
        // scale and zero point of the step's group, loaded kMetaPre steps ahead
        uint32_t meta[kMetaPre];
        auto fetch_meta = [&](int step) -> uint32_t {
            const int g = p.g_shift >= 0 ? (step >> p.g_shift) : step * kStepK / p.G;  // steps per group: a power of two, usually
            return w_row ? ((uint32_t)__half_as_ushort(__ldg(sr + g)) | ((uint32_t)__half_as_ushort(__ldg(zr + g)) << 16)) : 0u;
        };
#pragma unroll
        for (int u = 0; u < kMetaPre; ++u) meta[u] = (u < steps && !p.pair_meta) ? fetch_meta(s_begin + u) : 0u;
        // shared-memory addresses as 32-bit numbers, ring positions kept incrementally (this loop is issue bound)
        constexpr int kRowW = kStepK * kBits / 8;                    // bytes of a row in the packed tile
        const uint32_t w_row0 = smem_u32(sw) + (uint32_t)r * kRowW;
        // weight operand: rows of 128 bytes (one step), 128-byte swizzle: 16-byte piece c of row rr sits at piece c ^ (rr % 8)
        const uint32_t a_row0 = smem_u32(sa) + (uint32_t)h * kAHalf + (uint32_t)rr * 128;
        const uint32_t a_xor = (uint32_t)(rr & 7), c_first = 0u;
        uint32_t s = 0, sph = 1;     // stage of the operand ring and the parity of "stage free" to wait for
        uint32_t ws_ = 0, wph = 0;   // stage of the packed ring and the parity of "tile landed"
        auto one_step = [&](uint32_t m) -> bool {
            if (!mbar_wait(full_w0 + 8 * ws_, wph)) return false;     // the packed tile has landed
            uint32_t pk[kBits == 4 ? 8 : 16];
#pragma unroll
            for (int q = 0; q < (kBits == 4 ? 2 : 4); ++q)
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(pk[4 * q]), "=r"(pk[4 * q + 1]), "=r"(pk[4 * q + 2]), "=r"(pk[4 * q + 3])
                             : "r"(w_row0 + ws_ * kWStage + 16 * q));
            if (!mbar_wait(free0 + 8 * s, sph)) return false;         // the MMAs that read this stage last are complete
            const uint32_t a_st = a_row0 + s * kAStage;
            const float sf = __half2float(__ushort_as_half((unsigned short)(m & 0xFFFFu)));
            const float zf = __half2float(__ushort_as_half((unsigned short)(m >> 16)));
            const __nv_bfloat162 sc = __float2bfloat162_rn(sf);
            if constexpr (kBits == 4) {
                const __nv_bfloat162 off = __float2bfloat162_rn(zf + 128.f);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 v = dequant8_w4(pk[c], off, sc);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a_st + (((c_first + c) ^ a_xor) << 4)), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
                }
            } else {
                const float offf = 8388608.f + zf;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint2 lo = dequant4_w8(pk[2 * c], offf, sc), hi = dequant4_w8(pk[2 * c + 1], offf, sc);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a_st + (((c_first + c) ^ a_xor) << 4)), "r"(lo.x), "r"(lo.y), "r"(hi.x), "r"(hi.y) : "memory");
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMAs read through the async proxy
            __syncwarp();
            if (lane == 0) {
                // (the packed tile is released only now: its words were still being consumed above)
                mbar_arrive(free_w0 + 8 * ws_);
                mbar_arrive(full_a0 + 8 * s);
            }
            if (++s == kStages) { s = 0; sph ^= 1u; }
            if (++ws_ == kWStages) { ws_ = 0; wph ^= 1u; }
            return true;
        };
        int i = 0;
        if (p.pair_meta) {
            // One 32-bit load fetches the scales of two groups (4 steps), another their zero points, one block of
            // steps ahead: a load per step and thread would be a 2-byte gather over 256 rows, and those gathers, not
            // the arithmetic, then set the pace of the whole pipeline.
            const uint32_t* s2 = reinterpret_cast<const uint32_t*>(sr);
            const uint32_t* z2 = reinterpret_cast<const uint32_t*>(zr);
            uint32_t ns = w_row ? __ldg(s2 + (s_begin >> 2)) : 0u, nz = w_row ? __ldg(z2 + (s_begin >> 2)) : 0u;
            for (; ok && i < steps; i += 4) {
                const uint32_t cs = ns, cz = nz;
                if (i + 4 < steps) {
                    ns = w_row ? __ldg(s2 + ((s_begin + i + 4) >> 2)) : 0u;
                    nz = w_row ? __ldg(z2 + ((s_begin + i + 4) >> 2)) : 0u;
                }
                const uint32_t m_lo = (cs & 0xFFFFu) | (cz << 16), m_hi = (cs >> 16) | (cz & 0xFFFF0000u);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (ok) ok = one_step(u < 2 ? m_lo : m_hi);
            }
            i = steps;
        }
        for (; ok && i + kMetaPre <= steps; i += kMetaPre) {
#pragma unroll
            for (int u = 0; u < kMetaPre; ++u) {
                if (ok) ok = one_step(meta[u]);
                if (i + u + kMetaPre < steps) meta[u] = fetch_meta(s_begin + i + u + kMetaPre);
            }
        }
#pragma unroll
        for (int u = 0; u < kMetaPre; ++u)   // the last, partial block of steps
            if (ok && i + u < steps) ok = one_step(meta[u]);
        // ---------------- read-out: lane = feature 32 q + lane of half h ----------------
        if (ok) ok = mbar_wait(done0, 0);
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int q = warp & 3;                       // the quarter of the tensor-memory lanes this warp may read
            const int f = 128 * h + 32 * q + lane;        // (h from the thread's row: of every 8 warps the first 4 read half 0)
            const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16) + 256u * (uint32_t)h;
            const int n = n0 + f;
            const int tile_id = blockIdx.x * gridDim.y + blockIdx.y;
            float* part = p.split > 1 ? p.partials + ((size_t)(tile_id * p.split + z) * p.TN) * kTileF + f : nullptr;
            const int c_begin = 0, c_end = p.TN;
#pragma unroll 1
            for (int c0 = c_begin; c0 < c_end; c0 += 16) {
                uint32_t d[16];
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                    : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]), "=r"(d[8]),
                      "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15])
                    : "r"(taddr + (uint32_t)c0));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int j = 0; j < 16; ++j) asm volatile("" : "+r"(d[j]));
                if (part) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) __stcg(part + (size_t)(c0 + j) * kTileF, __uint_as_float(d[j]));
                } else if (n < p.N) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (m0 + c0 + j < p.M) p.y[(size_t)(m0 + c0 + j) * p.N + n] = __float2bfloat16_rn(__uint_as_float(d[j]));
                }
            }
        }
    }
    if (!ok && p.status) atomicOr(p.status, (int)QIL_ERR_TIMEOUT);
    if (p.split > 1) {
        // the last CTA of the tile to arrive adds the partial tiles in split order
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int tile_id = blockIdx.x * gridDim.y + blockIdx.y;
            const int prev = atomicAdd(&p.counters[tile_id], 1);
            *is_last = (prev == p.split - 1);
            if (*is_last) p.counters[tile_id] = 0;  // ready for the next call
        }
        __syncthreads();
        if (*is_last && tid >= 64 && tid < 64 + kTileF) {
            __threadfence();
            const int f = tid - 64, n = n0 + f;
            const int tile_id = blockIdx.x * gridDim.y + blockIdx.y;
            const float* base = p.partials + ((size_t)tile_id * p.split * p.TN) * kTileF + f;
            if (n < p.N) {
                for (int t0 = 0; t0 < p.TN && m0 + t0 < p.M; t0 += 8) {  // 8 tokens x split loads in flight
                    float acc[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
                    for (int sl = 0; sl < p.split; ++sl) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[j] += __ldcg(base + ((size_t)sl * p.TN + t0 + j) * kTileF);
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (m0 + t0 + j < p.M) p.y[(size_t)(m0 + t0 + j) * p.N + n] = __float2bfloat16_rn(acc[j]);
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols));
}

constexpr size_t kSmemBytes = (size_t)kStages * kAStage + (size_t)kBStages * kBStage + kWRingBytes +
                              (2 * kStages + 1 + 2 * kBStages + 2 * 12) * 8 + 16 + 1024;
static_assert(kSmemBytes <= 232448, "shared memory per CTA");

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
    static std::mutex mu;
    static EncodeFn fn = nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<EncodeFn>(ptr);
    }
    return fn;
}

struct PrefillPlan {
    int chunks, TN, ftiles, split;
};

PrefillPlan plan_prefill(int M, int N, int K) {
    PrefillPlan pl;
    pl.chunks = (M + kMaxTN - 1) / kMaxTN;
    const int per = (M + pl.chunks - 1) / pl.chunks;
    pl.TN = (per + 15) / 16 * 16;
    pl.ftiles = (N + kTileF - 1) / kTileF;
    // K is split where that fills the GPU.  Cost in steps: waves x (steps per CTA + the fixed cost of a CTA, about 12
    // steps: launch, first loads, read-out) + the reduction of the partial tiles (about 10 steps), as measured.
    const int tiles = pl.ftiles * pl.chunks, steps = K / kStepK, sms = num_sms();
    int best = 1;
    long best_cost = -1;
    for (int s = 1; s <= 8; ++s) {
        if (s > 1 && steps / s < 4) break;
        const long waves = ((long)tiles * s + sms - 1) / sms;
        const long cost = waves * ((steps + s - 1) / s + 12) + (s > 1 ? 10 : 0);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    pl.split = best;
    return pl;
}

}  // namespace

bool w4a16_prefill_supported(int M, int N, int K, int G, qil_layout layout) {
    return layout == QIL_LAYOUT_CANONICAL && M > 8 && N >= 1 && K % kStepK == 0 && G % kStepK == 0 && K % G == 0 &&
           (long long)((N + kTileF - 1) / kTileF) * ((M + kMaxTN - 1) / kMaxTN) <= kCounterBytes / 4 && (M + kMaxTN - 1) / kMaxTN <= 65535;
}

// Scratch the split along K needs (0 when K is not split): tile counters, then fp32 partial tiles.
size_t w4a16_prefill_workspace(int M, int N, int K) {
    const PrefillPlan pl = plan_prefill(M, N, K);
    if (pl.split == 1) return 0;
    return (size_t)kCounterBytes + (size_t)pl.ftiles * pl.chunks * pl.split * pl.TN * kTileF * sizeof(float);
}

// status (optional): receives QIL_ERR_TIMEOUT if a bounded device-side wait runs out.  scratch: as sized above; when it
// is missing or too small K is not split.
qil_status launch_w4a16_prefill(const void* x, const void* qw, const void* scales, const void* zeros, void* y, int M, int N,
                                int K, int G, int bits, int* status, void* scratch, size_t scratch_bytes, cudaStream_t st) {
    PrefillPlan pl = plan_prefill(M, N, K);
    if (pl.split > 1 && (scratch == nullptr || scratch_bytes < w4a16_prefill_workspace(M, N, K))) pl.split = 1;
    const EncodeFn enc = encode_fn();
    if (!enc) return QIL_ERR_CUDA;
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kStepK, (cuuint32_t)pl.TN};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return QIL_ERR_CUDA;
    // the packed weights as a byte matrix [N][K * bits / 8]: box = 64 codes x 256 rows, no swizzle
    CUtensorMap tmap_w;
    const cuuint64_t wdims[2] = {(cuuint64_t)K * bits / 8, (cuuint64_t)N};
    const cuuint64_t wstrides[1] = {(cuuint64_t)K * bits / 8};
    const cuuint32_t wbox[2] = {(cuuint32_t)(kStepK * bits / 8), (cuuint32_t)kTileF};
    if (enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(qw), wdims, wstrides, wbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return QIL_ERR_CUDA;
    PrefillParams p;
    p.qw = qw;
    p.scales = reinterpret_cast<const __half*>(scales);
    p.zeros = reinterpret_cast<const __half*>(zeros);
    p.y = reinterpret_cast<__nv_bfloat16*>(y);
    p.M = M; p.N = N; p.K = K; p.G = G;
    p.pair_meta = (G == 128 && (K / G) % 2 == 0 && K % 256 == 0) ? 1 : 0;
    const int spg = G / kStepK;  // steps per group
    p.g_shift = -1;
    if ((spg & (spg - 1)) == 0)
        for (int sh = 0; sh < 31; ++sh)
            if ((1 << sh) == spg) p.g_shift = sh;
    p.TN = pl.TN;
    p.split = pl.split;
    p.status = status;
    p.counters = reinterpret_cast<int*>(scratch);
    p.partials = scratch ? reinterpret_cast<float*>(static_cast<char*>(scratch) + kCounterBytes) : nullptr;
    const dim3 grid(pl.ftiles, pl.chunks, pl.split);
    cudaError_t e;
    if (bits == 8) {
        e = cudaFuncSetAttribute(w4a16_prefill_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e == cudaSuccess) w4a16_prefill_kernel<8><<<grid, kThreads, kSmemBytes, st>>>(tmap, tmap_w, p);
    } else {
        e = cudaFuncSetAttribute(w4a16_prefill_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e == cudaSuccess) w4a16_prefill_kernel<4><<<grid, kThreads, kSmemBytes, st>>>(tmap, tmap_w, p);
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    return launch_status();
}

}  // namespace qil
