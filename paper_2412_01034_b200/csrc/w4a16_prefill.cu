// Weight-only linears at prefill length (the prompt / vision-token stage of the paper's OpenVLA deployment,
// App. A.4.2; M tokens, typically 280; 4-bit weights, and the 8-bit weights of the INT8 deployment point of
// Sec. 5.4): a GEMM on tcgen05.mma kind::f16 (bf16 operands, fp32 accumulators in tensor memory).
//
// A tile is 128 output features x up to 288 tokens.  The weights are the M side of the MMAs and live in TENSOR
// MEMORY: the dequantising warps write the bf16 operand there with tcgen05.st (lane = feature, two bf16 per 32-bit
// column), so that a dequantised weight never touches shared memory, needs no swizzle and no proxy fence, and the
// MMAs read only the token tile from shared memory.  (With both operands in shared memory, 256 features x 144
// tokens per CTA, the step time sat at what the shared-memory traffic of operand stores plus MMA reads allows,
// whatever else was changed.)  Every weight of the tile is dequantised once for all its tokens.
//
// The launch is persistent: the (tile, step) pairs of the whole GEMM, a step being 64 input features, are numbered
// tile by tile and dealt out to the CTAs in equal contiguous ranges, so that every SM has the same work whatever the
// number of tiles (86 tiles of a 11008-wide projection on 148 SMs left 40 % of the GPU idle).  A tile that several
// CTAs share is completed by the CTA that holds its first steps - the end of that CTA's range, so the last thing it
// does: the others meet the tile at the beginning of their ranges, write their fp32 accumulators to their slot of the
// workspace and count themselves in; the completing CTA adds the parts to its own accumulators in the order of the
// CTAs (the result does not depend on timing) and writes the outputs.  Its wait for the count is bounded like every
// other wait, and the launch is cooperative so that the CTAs it waits for are resident.
// Where the ranges are short against a tile (four or more CTAs per tile) every CTA writes its parts instead and a
// second, fully parallel kernel adds them: the completing CTA's serial additions cost more there.
//
// Per step
//   * one thread copies the token tile with one or two bulk tensor copies (up to 144 tokens x 64 features each,
//     128-byte swizzle; tokens beyond M arrive as zeros),
//   * another copies the packed 128 x 64 weight tile with one bulk tensor copy into a ring that runs eight steps
//     ahead (loading the weights thread by thread, 16 or 32 bytes of a different row each, measured several
//     times slower),
//   * eight dequantising warps (thread = weight row and half of the step) turn 32 codes into bf16 - 128 + q by a
//     byte permute, a multiply and a mask (exact), minus 128 + z (exact: integers below 256), times the group's
//     scale rounded to bf16 (one rounding per weight) - and store them to the operand ring in tensor memory (four
//     stages of 32 columns).  The scales and zero points of two groups come with one 32-bit load each, a block of
//     steps ahead: a 2-byte gather per step over all rows was the slowest thing in the loop,
//   * one thread issues four or eight tcgen05.mma (128 x up to 144 x 16, A from tensor memory); tcgen05.commit
//     recycles the stages.
// The dequantising warps then read the accumulators (lane = feature) and write bf16 outputs or the fp32 part.
// A stage of a ring is released only after the data read from it has been used.
// Canonical layout only.  Every wait is bounded and polls; when one runs out QIL_ERR_TIMEOUT is recorded.
#include <cuda.h>

#include <mutex>

#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kTileF = 128, kStepK = 64, kStages = 4, kMaxNN = 144, kMaxTT = 2 * kMaxNN;
constexpr int kAccCols = kMaxTT;                  // accumulator columns (fp32, column = token)
constexpr int kAStageCols = kStepK / 2;           // a step of the weight operand: 64 bf16 per lane = 32 columns
constexpr int kBHalf = kMaxNN * kStepK * 2;       // up to 144 tokens x 64 bf16: 18 KiB (a multiple of 1024)
constexpr int kBStage = 2 * kBHalf;
constexpr int kWStages = 8;                       // ring of packed weight tiles (128 rows x 64 codes each)
constexpr int kThreads = 352;                     // token copy warp, MMA warp, 8 dequantising / read-out warps, weight copy warp
constexpr int kDqWarps = 8;
constexpr int kMetaPre = 8;                       // steps by which a dequantising thread's scale / zero loads run ahead
constexpr int kTmemCols = 512;
static_assert(kAccCols + kStages * kAStageCols <= kTmemCols, "tensor memory");
constexpr int kCounterBytes = 16384;              // tile counters at the start of the scratch (same place as the skinny kernel's)
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct PrefillParams {
    const void* qw;
    const __half* scales;
    const __half* zeros;
    __nv_bfloat16* y;
    int M, N, K, G;
    int g_shift;     // log2(G / 64) when that is a power of two, else -1
    int pair_meta;   // groups of 128 columns, an even number of them per row, K % 256 == 0: scales are loaded two groups at a time
    int NN, nh;      // tokens per MMA (multiple of 16, <= 144) and MMAs side by side (1 or 2): nh * NN tokens per tile
    int mt;          // token tiles
    int nchain;      // accumulators per output that take the K slices in turn (nh == 1 only): 2 or 4, else 1
    int unit_steps;  // the ranges of the CTAs begin at multiples of this many steps
    long long units; // unit_steps-sized pieces of the whole GEMM: tiles * (K / 64) / unit_steps
    int swiglu;      // rows 2i, 2i + 1 of the weights are gate i and up i: the output is silu(gate) * up, [M][N / 2]
    int* status;
    int fix;         // 1: shared tiles are completed inside this kernel; 0: every part is written out and a second kernel adds them
    int* counters;   // fix: per tile, parts written so far (zero between launches)
    float* partials; // [2 * CTAs][nh * NN][128]: slot 2c holds the part CTA c begins its range with, slot 2c + 1 the part it ends with
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

// D[128 x N] (+)= A[128 x 16 bf16] * B[N x 16 bf16]^T with A in tensor memory (lane = row, 8 columns of two bf16) and
// B in shared memory.  The descriptor of B comes as its two 32-bit halves: the issuing thread keeps the high half and
// the low half of every stage ready and adds small constants, because its own instruction stream - descriptors put
// together from 64-bit shifts for every MMA, divisions for the ring positions - was what set the pace of the whole
// pipeline before (a step took the same time with or without the MMAs' work, at any MMA width).
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 bd;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 bd, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 16 consecutive 32-bit columns of this thread's lane of tensor memory
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&d)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]), "=r"(d[8]),
          "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) asm volatile("" : "+r"(d[j]));
}

// silu(g) * u in fp32 (the gated MLP of the Llama-2 backbone; fused epilogue).  sigmoid(g) = (1 + tanh(g / 2)) / 2 with
// the hardware tanh (one special-function instruction instead of an exponential and a reciprocal; its error, about
// 2^-11 relative, is below the bf16 rounding of the result): the special-function unit set the pace of this epilogue.
__device__ __forceinline__ float swiglu(float g, float u) {
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * g));
    return fmaf(0.5f * g, t, 0.5f * g) * u;
}

// The CTA's next run of steps inside one tile: steps [s0, s1) of tile `tile`.  g walks the CTA's range of numbered steps.
struct Segment {
    int tile, s0, s1;
};
__device__ __forceinline__ bool next_segment(long long& g, long long g_end, int S, Segment& sg) {
    if (g >= g_end) return false;
    sg.tile = (int)(g / S);
    sg.s0 = (int)(g - (long long)sg.tile * S);
    const long long n = min((long long)(S - sg.s0), g_end - g);
    sg.s1 = sg.s0 + (int)n;
    g += n;
    return true;
}
// ranges of the CTAs in units: CTA c holds [units * c / C, units * (c + 1) / C)
__device__ __forceinline__ long long range_begin(long long units, int C, int c) { return units * c / C; }
__device__ __forceinline__ int cta_of_unit(long long units, int C, long long u) { return (int)(((u + 1) * C - 1) / units); }

template <int kBits>
__global__ void __launch_bounds__(kThreads, 1) w4a16_prefill_kernel(const __grid_constant__ CUtensorMap tmap_x,
                                                                   const __grid_constant__ CUtensorMap tmap_w,
                                                                   const PrefillParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // (the swizzled token tiles need 1024-byte alignment)
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char* sb = smem;                                  // [kStages][kBStage] tokens
    constexpr int kWStage = kTileF * kStepK * kBits / 8;       // packed weight tile: 4 KiB (4-bit), 8 KiB (8-bit)
    unsigned char* sw = sb + (size_t)kStages * kBStage;       // [kWStages][128 rows][kStepK * kBits / 8 bytes]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sw + (size_t)kWStages * kWStage);
    // stage s of the weight operand (tensor memory) and of the token tiles (shared memory) travel together: one
    // "free" barrier, one tcgen05.commit per step
    const uint32_t full_a0 = smem_u32(bars), full_b0 = smem_u32(bars + kStages), free0 = smem_u32(bars + 2 * kStages);
    uint64_t* wbars = bars + 3 * kStages;
    const uint32_t full_w0 = smem_u32(wbars), free_w0 = smem_u32(wbars + kWStages);
    uint64_t* obars = wbars + 2 * kWStages;
    const uint32_t done0 = smem_u32(obars), acc_free0 = smem_u32(obars + 1), part0 = smem_u32(obars + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(obars + 3);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = p.K / kStepK;                   // steps per tile
    const int C = (int)gridDim.x, cta = (int)blockIdx.x;
    const long long g_begin = range_begin(p.units, C, cta) * p.unit_steps, g_end = range_begin(p.units, C, cta + 1) * p.unit_steps;
    const int TT = p.NN * p.nh;
    const int ng = p.K / p.G;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_a0 + 8 * s, kDqWarps);   // the dequantising warps: weights stored, token tile seen to have landed
            mbar_init(full_b0 + 8 * s, 1);          // the token copies (transaction bytes)
            mbar_init(free0 + 8 * s, 1);            // the commit of the MMAs that read the stage
        }
        for (int s = 0; s < kWStages; ++s) {
            mbar_init(full_w0 + 8 * s, 1);          // the copy (transaction bytes)
            mbar_init(free_w0 + 8 * s, kDqWarps);   // the dequantising warps have read the tile
        }
        mbar_init(done0, 1);             // the commit after the last MMA of a segment
        mbar_init(acc_free0, kDqWarps);  // the accumulators of a segment have been read
        mbar_init(part0, kDqWarps);      // the CTA's part of a shared tile has been written
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
        // ---------------- token copies ----------------
        if (lane == 0) {
            int it = 0;
            Segment sg;
            for (long long g = g_begin; ok && next_segment(g, g_end, S, sg);) {
                const int m0 = (sg.tile % p.mt) * TT;
                for (int i = sg.s0; i < sg.s1; ++i, ++it) {
                    const int s = it % kStages, use = it / kStages;
                    ok = mbar_wait(free0 + 8 * s, (use & 1) ^ 1);    // the MMAs that read this stage last are complete
                    if (!ok) break;
                    mbar_expect_tx(full_b0 + 8 * s, (uint32_t)TT * kStepK * 2);
                    for (int hb = 0; hb < p.nh; ++hb)
                        tma_load_2d(smem_u32(sb + (size_t)s * kBStage) + (uint32_t)hb * p.NN * (kStepK * 2), &tmap_x, i * kStepK,
                                    m0 + hb * p.NN, full_b0 + 8 * s);
                }
            }
            // no copy may still be in flight when the CTA retires (this wait also holds after a time-out elsewhere)
            for (int back = 0; back < kStages && back < it; ++back) {
                const int i = it - 1 - back;
                (void)mbar_wait(full_b0 + 8 * (i % kStages), (i / kStages) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)p.NN >> 3) << 17) | (((uint32_t)kTileF >> 4) << 24);
            // descriptor of a token tile (K-major, 128-byte swizzle, 8 rows = 1024 bytes apart, version 1): its high half is
            // a constant, its low half the address in 16-byte units
            const uint32_t d_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t b_lo0 = ((smem_u32(sb) >> 4) & 0x3FFFu) | (1u << 16);
            const uint32_t half_lo = ((uint32_t)p.NN * (kStepK * 2)) >> 4;   // the second MMA's tokens
            const bool two = p.nh == 2;
            // MMAs into one accumulator follow one another at the latency of the tensor pipe, not at its throughput (about
            // 200 cycles each here, whatever their width).  Two token halves are two independent chains; a tile of up to
            // 144 tokens leaves room for more accumulators, which take the K slices in turn and are added at the read-out.
            const uint32_t cmask = (uint32_t)p.nchain - 1u, cstride = p.nchain == 4 ? 64u : (uint32_t)kMaxNN;   // (columns 0, 64, 128, 192 or 0, 144)
            uint32_t s = 0, aph = 0;
            int seg = 0;
            Segment sg;
            for (long long g = g_begin; ok && next_segment(g, g_end, S, sg); ++seg) {
                if (seg > 0) {
                    ok = mbar_wait(acc_free0, (seg - 1) & 1);   // the accumulators of the segment before have been read
                    if (!ok) break;
                }
                uint32_t acc = 0u;                               // the first MMAs of a segment overwrite the accumulators
#pragma unroll 1
                for (int i = sg.s0; i < sg.s1; ++i) {
                    // (the dequantising warps arrive once the step's token tile has landed as well: one wait here)
                    ok = mbar_wait(full_a0 + 8 * s, aph);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_tmem = tmem + (uint32_t)kAccCols + s * kAStageCols;
                    const uint32_t b_lo = b_lo0 + s * (kBStage >> 4);
#pragma unroll
                    for (int k = 0; k < kStepK / 16; ++k) {  // K = 16 each: 8 columns of A, 32 bytes of a swizzled row of B
                        if (two) {
                            mma_bf16_ts(tmem, a_tmem + 8 * k, b_lo + 2 * k, d_hi, idesc, k == 0 ? acc : 1u);
                            mma_bf16_ts(tmem + (uint32_t)p.NN, a_tmem + 8 * k, b_lo + half_lo + 2 * k, d_hi, idesc, k == 0 ? acc : 1u);
                        } else {
                            mma_bf16_ts(tmem + ((uint32_t)k & cmask) * cstride, a_tmem + 8 * k, b_lo + 2 * k, d_hi, idesc,
                                        (uint32_t)k <= cmask ? acc : 1u);
                        }
                    }
                    acc = 1u;
                    tc_commit(free0 + 8 * s);
                    if (++s == kStages) { s = 0; aph ^= 1u; }
                }
                if (!ok) break;
                tc_commit(done0);   // every MMA of the segment is complete when this arrival happens
            }
            // all MMAs are complete before tensor memory is released
            if (ok && seg > 0 && !mbar_wait(done0, (seg - 1) & 1)) ok = false;
        }
    } else if (warp == 2 + kDqWarps) {
        // ---------------- packed weight copies (rows beyond N arrive as zeros) ----------------
        if (lane == 0) {
            int it = 0;
            Segment sg;
            for (long long g = g_begin; ok && next_segment(g, g_end, S, sg);) {
                const int n0 = (sg.tile / p.mt) * kTileF;
                for (int i = sg.s0; i < sg.s1; ++i, ++it) {
                    const int s = it % kWStages, use = it / kWStages;
                    ok = mbar_wait(free_w0 + 8 * s, (use & 1) ^ 1);
                    if (!ok) break;
                    mbar_expect_tx(full_w0 + 8 * s, (uint32_t)kWStage);
                    tma_load_2d(smem_u32(sw + (size_t)s * kWStage), &tmap_w, i * (kStepK * kBits / 8), n0, full_w0 + 8 * s);
                }
            }
            for (int back = 0; back < kWStages && back < it; ++back) {
                const int i = it - 1 - back;
                (void)mbar_wait(full_w0 + 8 * (i % kWStages), (i / kWStages) & 1);
            }
        }
    } else {
        // ---------------- dequantising warps: a thread owns half a step (32 codes) of weight row rr of the tile ----------------
        // (a warp reaches the 32 lanes of tensor memory its number modulo 4 selects; two warps share a quarter and
        //  split the step's columns)
        const int q = warp & 3, hh = (warp - 2) >> 2;
        const int rr = 32 * q + lane;
        constexpr int kRowW = kStepK * kBits / 8;                     // bytes of a row in the packed tile
        const uint32_t w_row0 = smem_u32(sw) + (uint32_t)rr * kRowW + (uint32_t)hh * (kRowW / 2);
        const uint32_t a_lane = tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(kAccCols + hh * (kAStageCols / 2));
        uint32_t s = 0, sph = 1;     // stage of the operand ring and the parity of "stage free" to wait for
        uint32_t ws_ = 0, wph = 0;   // stage of the packed ring and the parity of "tile landed"
        auto one_step = [&](uint32_t m) -> bool {
            if (!mbar_wait(full_w0 + 8 * ws_, wph)) return false;     // the packed tile has landed
            uint32_t pk[kBits == 4 ? 4 : 8];
#pragma unroll
            for (int c = 0; c < (kBits == 4 ? 1 : 2); ++c)
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(pk[4 * c]), "=r"(pk[4 * c + 1]), "=r"(pk[4 * c + 2]), "=r"(pk[4 * c + 3])
                             : "r"(w_row0 + ws_ * kWStage + 16 * c));
            const float sf = __half2float(__ushort_as_half((unsigned short)(m & 0xFFFFu)));
            const float zf = __half2float(__ushort_as_half((unsigned short)(m >> 16)));
            const __nv_bfloat162 sc = __float2bfloat162_rn(sf);
            uint32_t v[16];
            if constexpr (kBits == 4) {
                const __nv_bfloat162 off = __float2bfloat162_rn(zf + 128.f);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 d = dequant8_w4(pk[c], off, sc);
                    v[4 * c] = d.x; v[4 * c + 1] = d.y; v[4 * c + 2] = d.z; v[4 * c + 3] = d.w;
                }
            } else {
                const float offf = 8388608.f + zf;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint2 d = dequant4_w8(pk[c], offf, sc);
                    v[2 * c] = d.x; v[2 * c + 1] = d.y;
                }
            }
            if (!mbar_wait(free0 + 8 * s, sph)) return false;         // the MMAs that read this stage last are complete
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            tmem_st16(a_lane + s * kAStageCols, v);
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            // the step's token tile has landed (parity of its ring = the complement of the one just waited for): the MMA
            // thread, which acquires this warp's arrival below, then needs no wait of its own for it
            if (!mbar_wait(full_b0 + 8 * s, sph ^ 1u)) return false;
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
        int seg = 0;
        Segment sg;
        for (long long g = g_begin, g_seg = g_begin; ok && next_segment(g, g_end, S, sg); ++seg, g_seg = g) {
            const int n0 = (sg.tile / p.mt) * kTileF, m0 = (sg.tile % p.mt) * TT;
            const bool w_row = n0 + rr < p.N;
            const size_t nrow = (size_t)(n0 + (w_row ? rr : 0));
            const __half* sr = p.scales + nrow * ng;
            const __half* zr = p.zeros + nrow * ng;
            const int s_begin = sg.s0, steps = sg.s1 - sg.s0;
            int i = 0;
            if (p.pair_meta) {
                // One 32-bit load fetches the scales of two groups (4 steps), another their zero points, one block of
                // steps ahead: a load per step and thread would be a 2-byte gather over all rows, and those gathers,
                // not the arithmetic, then set the pace of the whole pipeline.  (Segments begin at multiples of 4 steps.)
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
            } else {
                // scale and zero point of the step's group, loaded kMetaPre steps ahead
                auto fetch_meta = [&](int step) -> uint32_t {
                    const int gi = p.g_shift >= 0 ? (step >> p.g_shift) : step * kStepK / p.G;
                    return w_row ? ((uint32_t)__half_as_ushort(__ldg(sr + gi)) | ((uint32_t)__half_as_ushort(__ldg(zr + gi)) << 16)) : 0u;
                };
                uint32_t meta[kMetaPre];
#pragma unroll
                for (int u = 0; u < kMetaPre; ++u) meta[u] = u < steps ? fetch_meta(s_begin + u) : 0u;
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
            }
            // ---------------- read-out: lane = feature; the two warps of a quarter take alternate blocks of 16 tokens ----------------
            if (ok) ok = mbar_wait(done0, seg & 1);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const bool whole = sg.s0 == 0 && sg.s1 == S;               // the CTA holds every step of the tile
            const int n = n0 + rr;
            // A tile that several CTAs share: the CTA with the tile's first steps - for that CTA the last thing it does -
            // adds the others' parts to its own accumulators, in the order of the CTAs, and writes the outputs.  The others
            // meet the tile at the beginning of their ranges, write their part to their slot of the workspace and count
            // themselves in; by the time the first CTA gets there they are long done (its wait is bounded all the same).
            int c_first = cta, c_last = cta;
            if (!whole) {
                const long long su = S / p.unit_steps;                  // units per tile
                c_first = cta_of_unit(p.units, C, (long long)sg.tile * su);
                c_last = cta_of_unit(p.units, C, (long long)sg.tile * su + su - 1);
            }
            const bool fixer = p.fix && !whole && c_first == cta;
            if (fixer) {
                const int need = c_last - c_first;
                const int* cnt = p.counters + sg.tile;
                unsigned long long t0 = 0, t;
                for (uint32_t spin = 0;; ++spin) {
                    int have;
                    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(have) : "l"(cnt) : "memory");
                    if (have >= need) break;
                    if ((spin & 63u) == 0u) {
                        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
                        if (spin == 0u) t0 = t;
                        else if (t - t0 > kWaitLimitNs) { ok = false; break; }
                    }
                }
                if (!ok) break;
            }
            float* part = (!whole && !fixer) ? p.partials + ((size_t)(2 * cta + (g_seg == g_begin ? 0 : 1)) * TT) * kTileF + rr : nullptr;
            const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16);
#pragma unroll 1
            for (int c0 = 16 * hh; c0 < TT; c0 += 32) {
                uint32_t d[16];
                tmem_ld16(taddr + (uint32_t)c0, d);
                for (int ch = 1; ch < p.nchain; ++ch) {   // the other accumulators of these outputs
                    uint32_t e[16];
                    tmem_ld16(taddr + (uint32_t)(ch * (p.nchain == 4 ? 64 : kMaxNN) + c0), e);
#pragma unroll
                    for (int j = 0; j < 16; ++j) d[j] = __float_as_uint(__uint_as_float(d[j]) + __uint_as_float(e[j]));
                }
                if (part) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) __stcg(part + (size_t)(c0 + j) * kTileF, __uint_as_float(d[j]));
                } else {
                    const bool live = n < p.N && m0 + c0 < p.M;
                    if (live)
                    for (int cc = c_first + 1; cc <= c_last; ++cc) {
                        const float* other = p.partials + ((size_t)(2 * cc) * TT + c0) * kTileF + rr;  // (their first part)
                        float v[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = __ldcg(other + (size_t)j * kTileF);
#pragma unroll
                        for (int j = 0; j < 16; ++j) d[j] = __float_as_uint(__uint_as_float(d[j]) + v[j]);
                    }
                    if (p.swiglu) {
                        // lane = feature: the even lane holds gate i, its neighbour up i (N is even, so both are live or
                        // neither).  The pair shares the work: of tokens j, j + 1 the even lane takes j (its own gate, the
                        // neighbour's up), the odd lane j + 1 (the neighbour's gate, its own up): one exchange per two tokens,
                        // no lane computes a value that is thrown away.
                        const bool odd = (lane & 1) != 0;
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            const uint32_t mine = odd ? d[j + 1] : d[j];
                            const uint32_t theirs = __shfl_xor_sync(0xFFFFFFFFu, odd ? d[j] : d[j + 1], 1);
                            const float o = odd ? swiglu(__uint_as_float(theirs), __uint_as_float(mine))
                                                : swiglu(__uint_as_float(mine), __uint_as_float(theirs));
                            const int tk = m0 + c0 + j + (odd ? 1 : 0);
                            if (live && tk < p.M) p.y[(size_t)tk * (p.N >> 1) + (n >> 1)] = __float2bfloat16_rn(o);
                        }
                    } else if ((p.N & 1) == 0) {
                        // the same exchange: the even lane writes features n, n + 1 of token j as one 32-bit store, the odd
                        // lane those of token j + 1 (half the store instructions; the read-out is bound by them)
                        const bool odd = (lane & 1) != 0;
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            const uint32_t mine = odd ? d[j + 1] : d[j];
                            const uint32_t theirs = __shfl_xor_sync(0xFFFFFFFFu, odd ? d[j] : d[j + 1], 1);
                            const __nv_bfloat162 o = odd ? __floats2bfloat162_rn(__uint_as_float(theirs), __uint_as_float(mine))
                                                         : __floats2bfloat162_rn(__uint_as_float(mine), __uint_as_float(theirs));
                            const int tk = m0 + c0 + j + (odd ? 1 : 0);
                            if (live && tk < p.M) *reinterpret_cast<__nv_bfloat162*>(p.y + (size_t)tk * p.N + (n & ~1)) = o;
                        }
                    } else if (live) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (m0 + c0 + j < p.M) p.y[(size_t)(m0 + c0 + j) * p.N + n] = __float2bfloat16_rn(__uint_as_float(d[j]));
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_free0);
            if (part && p.fix) {
                // (a CTA writes at most one part per launch here: the barrier is used once)
                __threadfence();
                __syncwarp();
                if (lane == 0) mbar_arrive(part0);
                if (warp == 2) {
                    ok = mbar_wait(part0, 0);
                    if (!ok) break;
                    if (lane == 0) {
                        __threadfence();
                        atomicAdd(p.counters + sg.tile, 1);
                    }
                }
            }
        }
    }
    if (!ok && p.status) atomicOr(p.status, (int)QIL_ERR_TIMEOUT);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols));
    if (tid == 0 && g_end > g_begin && p.fix) {
        // the counter of the shared tile this CTA completed (its last one) goes back to zero for the next launch
        const int last_tile = (int)((g_end - 1) / S);
        const long long su = S / p.unit_steps;
        if (cta_of_unit(p.units, C, (long long)last_tile * su) == cta && cta_of_unit(p.units, C, (long long)last_tile * su + su - 1) != cta)
            p.counters[last_tile] = 0;
    }
}

// Adds the parts of every tile that several CTAs share, in the order of the CTAs, and writes the bf16 outputs.
// grid (tiles, blocks of 8 tokens); a warp = one token, a thread = 4 features.
__global__ void __launch_bounds__(256) w4a16_prefill_reduce_kernel(const PrefillParams p, int C) {
    const int tile = blockIdx.x, S = p.K / kStepK;
    const long long su = S / p.unit_steps;                  // units per tile
    const int c_first = cta_of_unit(p.units, C, (long long)tile * su), c_last = cta_of_unit(p.units, C, (long long)tile * su + su - 1);
    if (c_first == c_last) return;                          // one CTA held the whole tile and wrote the outputs itself
    const int TT = p.NN * p.nh;
    const int n0 = (tile / p.mt) * kTileF, m0 = (tile % p.mt) * TT;
    const int t = blockIdx.y * 8 + (threadIdx.x >> 5), f = 4 * (threadIdx.x & 31);
    if (t >= TT || m0 + t >= p.M || n0 + f >= p.N) return;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int cc = c_first; cc <= c_last; ++cc) {
        // the part a CTA begins its range with is in slot 2 * cta, the part it ends with in slot 2 * cta + 1
        const int slot = 2 * cc + (range_begin(p.units, C, cc) * p.unit_steps >= (long long)tile * S ? 0 : 1);
        const float4 v = __ldcg(reinterpret_cast<const float4*>(p.partials + ((size_t)slot * TT + t) * kTileF + f));
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    if (p.swiglu) {   // features f, f + 1 and f + 2, f + 3 are two (gate, up) pairs
        __nv_bfloat16* out = p.y + (size_t)(m0 + t) * (p.N >> 1) + ((n0 + f) >> 1);
        out[0] = __float2bfloat16_rn(swiglu(acc.x, acc.y));
        if (n0 + f + 2 < p.N) out[1] = __float2bfloat16_rn(swiglu(acc.z, acc.w));
        return;
    }
    __nv_bfloat16* out = p.y + (size_t)(m0 + t) * p.N + n0 + f;
    if ((p.N & 3) == 0) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 o;
        o.x = *reinterpret_cast<const uint32_t*>(&lo);
        o.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(out) = o;
    } else {
        const float a4[4] = {acc.x, acc.y, acc.z, acc.w};
        for (int j = 0; j < 4 && n0 + f + j < p.N; ++j) out[j] = __float2bfloat16_rn(a4[j]);
    }
}

constexpr size_t kSmemBytes = (size_t)kStages * kBStage + (size_t)kWStages * (kTileF * kStepK) +
                              (3 * kStages + 2 * kWStages + 3) * 8 + 16 + 1024;
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
    int mt, NN, nh, nchain, ftiles, ctas, unit_steps;
    long long units;
};

// with_parts: the workspace can hold the parts of tiles that several CTAs share; without it every CTA gets whole tiles.
PrefillPlan plan_prefill(int M, int N, int K, int G, bool with_parts) {
    PrefillPlan pl;
    pl.mt = (M + kMaxTT - 1) / kMaxTT;
    const int per = (M + pl.mt - 1) / pl.mt;
    pl.nh = per > kMaxNN ? 2 : 1;
    pl.NN = ((per + pl.nh - 1) / pl.nh + 15) / 16 * 16;
    pl.nchain = pl.nh == 2 ? 1 : (pl.NN <= 64 ? 4 : 2);
    pl.ftiles = (N + kTileF - 1) / kTileF;
    const int S = K / kStepK, sms = num_sms();
    const long long tiles = (long long)pl.ftiles * pl.mt;
    const bool pair = G == 128 && (K / G) % 2 == 0 && K % 256 == 0;
    pl.unit_steps = with_parts ? (pair ? 4 : 1) : S;
    pl.units = tiles * (S / pl.unit_steps);
    // a CTA is worth launching for about eight steps; never more CTAs than SMs or units
    long long c = with_parts ? tiles * S / 8 : tiles;
    if (c > sms) c = sms;
    if (c > pl.units) c = pl.units;
    if (c < 1) c = 1;
    pl.ctas = (int)c;
    return pl;
}

__global__ void swiglu_rows_kernel(const __nv_bfloat16* __restrict__ t, __nv_bfloat16* __restrict__ y, int M, int N) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x, half = N >> 1;
    if (i >= (long long)M * half) return;
    const long long m = i / half, c = i - m * half;
    const __nv_bfloat162 gu = *reinterpret_cast<const __nv_bfloat162*>(t + m * N + 2 * c);
    y[i] = __float2bfloat16_rn(swiglu(__bfloat162float(gu.x), __bfloat162float(gu.y)));
}

}  // namespace

qil_status launch_swiglu_rows(const void* t, void* y, int M, int N, cudaStream_t st) {
    const long long total = (long long)M * (N >> 1);
    swiglu_rows_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(t),
                                                                        reinterpret_cast<__nv_bfloat16*>(y), M, N);
    return launch_status();
}

bool w4a16_prefill_supported(int M, int N, int K, int G, qil_layout layout) {
    return layout == QIL_LAYOUT_CANONICAL && M > 8 && N >= 1 && K % kStepK == 0 && G % kStepK == 0 && K % G == 0 &&
           (long long)((N + kTileF - 1) / kTileF) * ((M + kMaxTT - 1) / kMaxTT) <= kCounterBytes / 4;
}

// Scratch for the parts of tiles that several CTAs share: tile counters, then two fp32 tiles per CTA.
size_t w4a16_prefill_workspace(int M, int N, int K, int G) {
    const PrefillPlan pl = plan_prefill(M, N, K, G, true);
    return (size_t)kCounterBytes + (size_t)2 * pl.ctas * pl.nh * pl.NN * kTileF * sizeof(float);
}

// status (optional): receives QIL_ERR_TIMEOUT if a bounded device-side wait runs out.  scratch: as sized above; when it
// is missing or too small every CTA computes whole tiles.
qil_status launch_w4a16_prefill(const void* x, const void* qw, const void* scales, const void* zeros, void* y, int M, int N,
                                int K, int G, int bits, int* status, void* scratch, size_t scratch_bytes, cudaStream_t st, int swiglu) {
    const bool with_parts = scratch != nullptr && scratch_bytes >= w4a16_prefill_workspace(M, N, K, G);
    const PrefillPlan pl = plan_prefill(M, N, K, G, with_parts);
    const EncodeFn enc = encode_fn();
    if (!enc) return QIL_ERR_CUDA;
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kStepK, (cuuint32_t)pl.NN};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return QIL_ERR_CUDA;
    // the packed weights as a byte matrix [N][K * bits / 8]: box = 64 codes x 128 rows, no swizzle
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
    p.NN = pl.NN; p.nh = pl.nh; p.mt = pl.mt; p.nchain = pl.nchain;
    p.unit_steps = pl.unit_steps;
    p.units = pl.units;
    p.status = status;
    p.swiglu = swiglu;
    p.counters = with_parts ? reinterpret_cast<int*>(scratch) : nullptr;
    // A tile shared by up to three CTAs is completed inside the kernel by the CTA that holds its first steps; when the
    // ranges are short against a tile (more CTAs per tile) that CTA's serial additions cost more than a second, fully
    // parallel kernel (measured on the 4096 x 4096 and 4096 x 11008 projections at 280 tokens).
    const long long per_cta = pl.units / pl.ctas, per_tile = (long long)(K / kStepK) / pl.unit_steps;
    p.fix = (with_parts && 2 * per_cta >= per_tile) ? 1 : 0;
    p.partials = with_parts ? reinterpret_cast<float*>(static_cast<char*>(scratch) + kCounterBytes) : nullptr;
    // The CTAs of a shared tile wait for one another's parts: the launch is cooperative, so that all of them are resident
    // (one CTA per SM by its shared memory, never more CTAs than SMs).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)pl.ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.fix ? 1 : 0;
    cudaError_t e;
    if (bits == 8) {
        e = cudaFuncSetAttribute(w4a16_prefill_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, w4a16_prefill_kernel<8>, tmap, tmap_w, p);
    } else {
        e = cudaFuncSetAttribute(w4a16_prefill_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, w4a16_prefill_kernel<4>, tmap, tmap_w, p);
    }
    if (e == cudaErrorCooperativeLaunchTooLarge) {
        (void)cudaGetLastError();
        return QIL_ERR_UNSUPPORTED;
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    if (with_parts && !p.fix && pl.ctas > 1) {
        const dim3 rgrid((unsigned)(pl.ftiles * pl.mt), (unsigned)((pl.nh * pl.NN + 7) / 8));
        w4a16_prefill_reduce_kernel<<<rgrid, 256, 0, st>>>(p, pl.ctas);
    }
    return launch_status();
}

}  // namespace qil
