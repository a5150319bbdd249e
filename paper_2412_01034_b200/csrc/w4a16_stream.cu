// Weight-only 4-bit decode linears as ONE persistent kernel over a list of linears
// (the memory-bound decode stage of the paper's OpenVLA deployment, Sec. 5.4 /
// App. A.4.2: q, k, v, o, gate, up, down of every decoder layer, M <= 4 rows).
//
// Data layout (QIL_LAYOUT_STREAM): the weight matrix is a sequence of self-contained
// 1088-byte units, unit u = (row tile rt = u / (K/128), column block kb = u % (K/128)):
// 1024 bytes of packed codes of 16 output features x 128 input features (16 rows of 64
// bytes) followed by 16 x {fp16 scale, fp16 zero} of those rows for that block.  Byte b
// of 32-bit word m of a row holds column 8m + b in its low and column 8m + 4 + b in its
// high nibble, so that one AND per word yields four unsigned bytes (the low nibbles as
// they are, the high nibbles times 16).  A linear is one contiguous byte stream, and any
// slice of units is too.
//
// Arithmetic: integer.  The activations of a linear are converted once to 16-bit block
// fixed point: per row and 128-column block a power-of-two scale 2^e with
// |x| / 2^e <= 32639, v = rint(x / 2^e) = 256 hi + lo stored as two int8 planes.  The
// codes multiply both planes on the tensor cores (mma.sync m16n8k32 u8 x s8 -> s32,
// exact); the 8 columns of the instruction are {row 0 hi, row 0 lo, row 1 hi, ...}.
// Scale and zero point are folded once per unit:
//     y += s 2^e ((256 D_hi + D_lo) - z X),   X = sum of the block's integers v.
// The only rounding beyond the fp32 accumulation over blocks is that of v (relative
// 2^-15 of the block maximum), far below the bf16 rounding of the output.
//
// Execution: one CTA per SM, alive for the whole list.  For every linear each CTA
// owns a contiguous slice of its units (balanced to +-1 unit).  A producer thread
// streams the slice through a shared-memory ring with bulk asynchronous copies
// (cp.async.bulk + mbarrier transaction counts), running ahead across linears as far
// as the ring allows, so HBM stays busy while the consumers finish a linear.
// Twenty-four compute warps (six per scheduler, to cover the latency of the dependent
// instruction chains) each take one unit per ring stage.
// They never wait for another CTA: per pass they leave per-warp partial tiles in a
// double-buffered shared array and go on.  A combiner group of two warps adds the
// partial tiles and writes finished outputs; two fixer warps do all cross-CTA work
// from small queues; three stager warps fetch and convert the activations of the next
// entry (two buffers) and wait for dependencies - all hidden behind the compute warps.
// Row tiles cut by a slice boundary are completed through small slots in the
// workspace: every CTA publishes its contribution to the tile it shares with the next
// CTA and completes the tile it shares with previous CTAs, adding the contributions in
// CTA order - so results do not depend on timing.  A slot is a set of {fp32 value, tag}
// pairs written with one 8-byte store each; the tag is the index of the entry the value
// belongs to (0 = free), because the CTA that completes a tile differs from entry to
// entry; slots form a ring over entries so that neighbouring CTAs need not run in
// lockstep.  An entry flagged
// QIL_DEP_PREVIOUS first waits until every row tile of all earlier entries is
// written (a monotonic counter in the workspace).
//
// Every wait (mbarrier, slot flag, dependency counter) is bounded; when a bound is
// hit the kernel records QIL_ERR_TIMEOUT in the workspace status word, stops waiting
// and runs to completion without touching memory outside its buffers.
#include <mutex>

#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kComputeWarps = 24;
constexpr int kComputeThreads = kComputeWarps * 32;
constexpr int kEpiThreads = 64;      // combiner group: 2 warps
constexpr int kStagerThreads = 96;   // activation stager: 3 warps
constexpr int kFixDepth = 4;         // records queued between the combiner group and each of the two fixer warps
constexpr int kFixThreads = 64;      // two fixer warps: one publishes contributions, one completes shared tiles
constexpr int kThreads = kComputeThreads + kEpiThreads + kFixThreads + kStagerThreads + 32;  // + producer warp
static_assert(kThreads <= 1024, "block size");
constexpr int kUnitBytes = 1088;
constexpr int kStageUnits = kComputeWarps;
constexpr int kStageBytes = kStageUnits * kUnitBytes;
constexpr int kMaxRows = 4;     // activation rows: two int8 planes each fill the 8 columns of the instruction
constexpr int kElemsMax = 64;   // fp32 values of one row tile: 16 rows x 4 activation rows (16 when M == 1)
constexpr int kMaxEntries = 256;
constexpr int kSlotDepth = 4;   // ring of slots per (CTA, first / last tile of its slice), indexed by entry % depth
constexpr int kSlotBytes = kElemsMax * 8;  // {fp32 value, tag} pairs, one 8-byte store each
constexpr int kWsHeader = 256;
constexpr int kRowPad = 16;
constexpr int kFlagDep = 1;      // StreamEntry::flags: wait for all earlier entries
constexpr int kFlagAligned = 2;  // StreamEntry::flags: slices are whole row tiles (set by the host)
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // every wait gives up after two seconds

struct StreamEntry {  // 48 bytes
    const uint16_t* x;
    const unsigned char* w;
    __nv_bfloat16* y;
    int N, K, M, flags;
    uint32_t tiles_before;  // row tiles of all earlier entries of this launch
    uint32_t pad;
};

struct StreamParams {
    StreamEntry e[kMaxEntries];
    int count;
    int stages;
    int x_rows;       // max M over the entries
    int x_row_bytes;  // one int8 plane of a row: max K + pad
    int kb_max;       // max K / 128
    int elems;        // fp32 values kept per (row tile, warp): 16 if every M == 1, else 64
    int max_tiles;    // row tiles per pass: 8 (elems 16) or 2 (elems 64)
    int* status;
    unsigned int* tiles_done;
    unsigned char* slots;
};

// ---- PTX wrappers -------------------------------------------------------------------------
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
// same, but the thread may stay suspended in hardware for up to `ns` nanoseconds while the phase is incomplete
// (a waiting role then does not compete with the compute warps for issue slots)
__device__ __forceinline__ uint32_t mbar_try_wait_suspend(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok;
}
__device__ __forceinline__ void bulk_g2s_plain(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const unsigned int* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(unsigned int* p, uint32_t v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }
__device__ __forceinline__ void stager_sync() { asm volatile("bar.sync 2, %0;" ::"n"(kStagerThreads) : "memory"); }

// D[16 x 8] += A[16 x 32 unsigned bytes] * B[32 x 8 signed bytes], int32 accumulate (exact)
__device__ __forceinline__ void mma_u8s8_16832(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---- bounded waits --------------------------------------------------------------------------
struct Guard {
    int* status;
    volatile int* poisoned;  // shared memory flag of this CTA
    __device__ __forceinline__ void fail() const {
        if (!*poisoned) {
            *poisoned = 1;
            atomicOr(status, (int)QIL_ERR_TIMEOUT);
        }
    }
    static __device__ __forceinline__ unsigned long long now_ns() {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        return t;
    }
    __device__ __forceinline__ void wait_mbar(uint32_t bar, uint32_t parity) const {
        if (mbar_try_wait(bar, parity)) return;
        if (*poisoned) return;
        const unsigned long long t0 = now_ns();
        for (uint32_t i = 1;; ++i) {
            if (mbar_try_wait_suspend(bar, parity, 200u)) return;
            if ((i & 15u) == 0 && (*poisoned || now_ns() - t0 > kWaitLimitNs)) break;
        }
        fail();
    }
    template <typename Pred>
    __device__ __forceinline__ void wait_flag(Pred done) const {
        if (*poisoned) return;
        if (done()) return;
        const unsigned long long t0 = now_ns();
        for (uint32_t i = 1;; ++i) {
            if (done()) return;
            __nanosleep(i < 64 ? 20 : 200);
            if ((i & 63u) == 0 && (*poisoned || now_ns() - t0 > kWaitLimitNs)) break;
        }
        fail();
    }
};

// slice of `units` owned by CTA c of C
__device__ __forceinline__ void slice_of(uint32_t units, uint32_t c, uint32_t C, uint32_t& u0, uint32_t& u1) {
    u0 = (uint32_t)(((uint64_t)c * units) / C);
    u1 = (uint32_t)(((uint64_t)(c + 1) * units) / C);
}
// CTA that owns unit u (the largest c whose slice starts at or before u)
__device__ __forceinline__ uint32_t owner_of(uint32_t u, uint32_t units, uint32_t C) {
    return (uint32_t)((((uint64_t)(u + 1)) * C - 1) / units);
}
// slot (0 or 1) in which CTA cc publishes its contribution to row tile rt; false if cc has no units
__device__ __forceinline__ bool contributor_slot(uint32_t cc, uint32_t rt, uint32_t units, uint32_t KB, uint32_t C,
                                                 uint32_t& which) {
    uint32_t cu0, cu1;
    slice_of(units, cc, C, cu0, cu1);
    which = (cu0 / KB == rt) ? 0u : 1u;
    return cu0 != cu1;
}

// Iterates over the work of one CTA: entries with a non-empty slice, cut into passes of at most
// `max_tiles` row tiles.  Producer, compute warps and the epilogue group all walk the same sequence.
struct Walk {
    const StreamParams& p;
    uint32_t C, c;
    int ei;                       // current entry (-1 before the first)
    uint32_t KB, units, u0, u1;   // of the current entry
    uint32_t t_first, t_last;
    __device__ Walk(const StreamParams& p_, uint32_t C_, uint32_t c_) : p(p_), C(C_), c(c_), ei(-1) {}
    // advance to the next entry in which this CTA owns units; false at the end of the list
    __device__ bool next_entry() {
        for (++ei; ei < p.count; ++ei) {
            KB = (uint32_t)p.e[ei].K >> 7;
            const uint32_t RT = (uint32_t)p.e[ei].N >> 4;
            units = RT * KB;
            if (p.e[ei].flags & kFlagAligned) {  // whole row tiles only: no tile is shared between CTAs
                u0 = (uint32_t)(((uint64_t)c * RT) / C) * KB;
                u1 = (uint32_t)(((uint64_t)(c + 1) * RT) / C) * KB;
            } else {
                slice_of(units, c, C, u0, u1);
            }
            if (u0 != u1) {
                t_first = u0 / KB;
                t_last = (u1 - 1) / KB;
                return true;
            }
        }
        return false;
    }
};

// Records the combiner group hands to the fixer warp (cross-CTA work, off the compute path).
enum : int { kRecContrib = 2, kRecFinish = 3, kRecEnd = 4 };
struct FixRec {
    int type;
    int ei;        // entry index
    uint32_t arg;  // kRecContrib: slot (0/1); kRecFinish: row tile
    uint32_t pad;
    float data[kElemsMax];
};

__global__ void __launch_bounds__(kThreads, 1) w4a16_stream_kernel(const __grid_constant__ StreamParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x;
    const uint32_t C = gridDim.x, c = blockIdx.x;
    const int elems = p.elems, max_tiles = p.max_tiles;
    const int part_floats = max_tiles * kComputeWarps * elems;  // one tile_part buffer

    // ---- carve shared memory ----
    unsigned char* ring = smem;
    float* tile_part = reinterpret_cast<float*>(ring + (size_t)p.stages * kStageBytes);  // [2][max_tiles][compute warps][elems]
    float* stash_first = tile_part + 2 * part_floats;                                    // [kElemsMax]
    float* stash_last = stash_first + kElemsMax;                                         // [kElemsMax]
    FixRec* fixq = reinterpret_cast<FixRec*>(stash_last + kElemsMax);                    // [2 queues][kFixDepth]
    unsigned char* xs = reinterpret_cast<unsigned char*>(fixq + 2 * kFixDepth);  // [2][2 x_rows planes][x_row_bytes]
    unsigned char* xraw = xs + (size_t)4 * p.x_rows * p.x_row_bytes;         // [x_rows][256 kb_max] bf16 as copied
    int* xsum = reinterpret_cast<int*>(xraw + (size_t)p.x_rows * p.kb_max * 256);  // [2][kMaxRows][kb_max]
    float* xscale = reinterpret_cast<float*>(xsum + 2 * kMaxRows * p.kb_max);      // [2][kMaxRows][kb_max]
    unsigned int* pmax = reinterpret_cast<unsigned int*>(xscale + 2 * kMaxRows * p.kb_max);  // [16 kb_max] piece maxima
    int* psum = reinterpret_cast<int*>(pmax + 16 * p.kb_max);                                // [16 kb_max] piece sums
    uint64_t* bars = reinterpret_cast<uint64_t*>(psum + 16 * p.kb_max);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + p.stages);
    uint64_t* b2 = bars + 2 * p.stages;
    const uint32_t xfull0 = smem_u32(b2);          // [2] activations of an entry are staged
    const uint32_t xempty0 = smem_u32(b2 + 2);     // [2] the compute warps are done with them
    const uint32_t accfull0 = smem_u32(b2 + 4);    // [2] all compute warps left their partial tiles
    const uint32_t accempty0 = smem_u32(b2 + 6);   // [2] the combiner is done with the buffer
    const uint32_t fqfull0 = smem_u32(b2 + 8);     // [2][kFixDepth] a record is ready for its fixer warp
    const uint32_t fqempty0 = smem_u32(b2 + 8 + 2 * kFixDepth);  // [2][kFixDepth] the fixer warp has consumed it
    const uint32_t xraw0 = smem_u32(b2 + 8 + 4 * kFixDepth);  // [2] the bulk copies of the rows of x have landed
    volatile int* poisoned = reinterpret_cast<volatile int*>(b2 + 10 + 4 * kFixDepth);

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kComputeWarps);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(xfull0 + 8 * b, 1);
            mbar_init(xempty0 + 8 * b, kComputeWarps);
            mbar_init(accfull0 + 8 * b, kComputeWarps);
            mbar_init(accempty0 + 8 * b, 1);
            mbar_init(xraw0 + 8 * b, 1);
        }
        for (int q = 0; q < 2 * kFixDepth; ++q) {
            mbar_init(fqfull0 + 8 * q, 1);
            mbar_init(fqempty0 + 8 * q, 1);
        }
        *poisoned = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < 2 * part_floats; i += kThreads) tile_part[i] = 0.f;
    for (int i = tid; i < 2 * kMaxRows * p.kb_max; i += kThreads) {
        xsum[i] = 0;
        xscale[i] = 0.f;
    }
    __syncthreads();
    const Guard guard{p.status, poisoned};

    if (tid < kComputeThreads) {
        // =============================== compute warps ===============================
        // Lane (g = lane / 4, t = lane % 4) owns weight rows g and g + 8 of the unit and activation row t:
        // accumulator columns 2t and 2t + 1 are the high- and low-byte planes of activation row t.
        const int lane = tid & 31, warp = tid >> 5;
        const int g = lane >> 2, t = lane & 3;
        const bool compact = elems == 16;  // M == 1: only the lanes with t == 0 hold real outputs
        uint32_t item = 0, xe = 0;
        uint32_t rs = 0, rph = 0;  // ring stage and its phase
        Walk wk(p, C, c);
        while (wk.next_entry()) {
            const int M = p.e[wk.ei].M;
            const uint32_t KB = wk.KB;
            const uint32_t xb = xe & 1;
            guard.wait_mbar(xfull0 + 8 * xb, (xe >> 1) & 1);
            ++xe;
            // B fragments: plane row g (= 2 * activation row + {high, low}), 32 consecutive columns per lane
            const unsigned char* xlane =
                xs + ((size_t)xb * 2 * p.x_rows + g) * p.x_row_bytes + (size_t)t * 32;
            const bool has_b = g < 2 * M;
            const int* xsum_lane = xsum + ((size_t)xb * kMaxRows + t) * p.kb_max;
            const float* xscale_lane = xscale + ((size_t)xb * kMaxRows + t) * p.kb_max;
            for (uint32_t tp = wk.t_first; tp <= wk.t_last; tp += max_tiles, ++item) {
                const uint32_t pu0 = max(wk.u0, tp * KB), pu1 = min(wk.u1, (tp + max_tiles) * KB);
                const uint32_t ab = item & 1;
                guard.wait_mbar(accempty0 + 8 * ab, ((item >> 1) & 1) ^ 1);
                float* part = tile_part + (size_t)ab * part_floats + (size_t)warp * elems + (compact ? g * 2 : lane * 2);
                const bool writer = !compact || t == 0;
                float fin0 = 0.f, fin1 = 0.f;  // rows g and g + 8, activation row t
                int cur_tile = -1;
                // this warp's unit of the first chunk, as (tile within the pass, column block); later chunks advance by one stage
                uint32_t u = pu0 + warp;
                uint32_t tl = u / KB - tp, kb = u % KB;
                for (uint32_t cu = pu0; cu < pu1; cu += kStageUnits) {
                    guard.wait_mbar(full0 + 8 * rs, rph);
                    if (cu + warp < pu1) {
                        if ((int)tl != cur_tile) {
                            if (cur_tile >= 0 && writer)
                                *reinterpret_cast<float2*>(part + (size_t)cur_tile * kComputeWarps * elems) =
                                    make_float2(fin0, fin1);
                            fin0 = fin1 = 0.f;
                            cur_tile = (int)tl;
                        }
                        const unsigned char* ub = ring + (size_t)rs * kStageBytes + (size_t)warp * kUnitBytes;
                        const uint4 wa = *reinterpret_cast<const uint4*>(ub + lane * 16);        // row g, columns 32t..
                        const uint4 wb = *reinterpret_cast<const uint4*>(ub + 512 + lane * 16);  // row g + 8
                        const __half2 ma = *reinterpret_cast<const __half2*>(ub + 1024 + 4 * g);
                        const __half2 mb = *reinterpret_cast<const __half2*>(ub + 1024 + 4 * (g + 8));
                        uint4 b0 = make_uint4(0, 0, 0, 0), b1 = make_uint4(0, 0, 0, 0);
                        if (has_b) {
                            const uint4* xp = reinterpret_cast<const uint4*>(xlane + (size_t)kb * 128);
                            b0 = xp[0];  // columns 32t + {0-3, 4-7, 8-11, 12-15}
                            b1 = xp[1];  // columns 32t + 16 + ...
                        }
                        // word j of the lane: low nibbles = columns 8j..8j+3, high nibbles = columns 8j+4..8j+7.
                        // Low nibbles accumulate as they are, high nibbles times 16 in an accumulator of their own.
                        constexpr uint32_t kLo = 0x0F0F0F0Fu, kHi = 0xF0F0F0F0u;
                        int lo[4] = {0, 0, 0, 0}, hi[4] = {0, 0, 0, 0};
                        mma_u8s8_16832(lo, wa.x & kLo, wb.x & kLo, wa.y & kLo, wb.y & kLo, b0.x, b0.z);
                        mma_u8s8_16832(hi, wa.x & kHi, wb.x & kHi, wa.y & kHi, wb.y & kHi, b0.y, b0.w);
                        mma_u8s8_16832(lo, wa.z & kLo, wb.z & kLo, wa.w & kLo, wb.w & kLo, b1.x, b1.z);
                        mma_u8s8_16832(hi, wa.z & kHi, wb.z & kHi, wa.w & kHi, wb.w & kHi, b1.y, b1.w);
                        // 256 D_hi + D_lo of rows g and g + 8 (the high-nibble sums are exact multiples of 16)
                        const int va = (lo[0] * 256 + lo[1]) + ((hi[0] * 256 + hi[1]) >> 4);
                        const int vb = (lo[2] * 256 + lo[3]) + ((hi[2] * 256 + hi[3]) >> 4);
                        const float xsf = (float)xsum_lane[kb];
                        const float sc = xscale_lane[kb];
                        fin0 = fmaf(__low2float(ma) * sc, fmaf(-__high2float(ma), xsf, (float)va), fin0);
                        fin1 = fmaf(__low2float(mb) * sc, fmaf(-__high2float(mb), xsf, (float)vb), fin1);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty0 + 8 * rs);
                    if (++rs == (uint32_t)p.stages) { rs = 0; rph ^= 1; }
                    kb += kStageUnits;
                    while (kb >= KB) { kb -= KB; ++tl; }
                }
                if (cur_tile >= 0 && writer)
                    *reinterpret_cast<float2*>(part + (size_t)cur_tile * kComputeWarps * elems) = make_float2(fin0, fin1);
                __syncwarp();
                if (lane == 0) mbar_arrive(accfull0 + 8 * ab);
            }
            if (lane == 0) mbar_arrive(xempty0 + 8 * xb);  // (ordered after this warp's reads by the __syncwarp above)
        }
    } else if (tid < kComputeThreads + kEpiThreads) {
        // =============================== combiner group (2 warps) ===============================
        const int et = tid - kComputeThreads;  // 0..kEpiThreads-1
        uint32_t item = 0, fq[2] = {0, 0};
        // element index -> (row within the tile, activation row)
        auto decode = [&](int e, int& row, int& tok) {
            if (elems == 16) {  // e = 2 g + h
                row = (e >> 1) + ((e & 1) ? 8 : 0);
                tok = 0;
            } else {            // e = 2 lane + h, lane = 4 g + t
                row = (e >> 3) + ((e & 1) ? 8 : 0);
                tok = (e >> 1) & 3;
            }
        };
        // hand one record to fixer warp `which_q` (0: contributions, 1: completions)
        auto push = [&](int which_q, int type, int ei, uint32_t arg, const float* data) {
            const uint32_t q = which_q * kFixDepth + fq[which_q] % kFixDepth, round = fq[which_q] / kFixDepth;
            if (et == 0) guard.wait_mbar(fqempty0 + 8 * q, (round & 1) ^ 1);
            epi_sync();
            FixRec& r = fixq[q];
            if (et == 0) { r.type = type; r.ei = ei; r.arg = arg; }
            if (data != nullptr && et < elems) r.data[et] = data[et];
            epi_sync();
            if (et == 0) mbar_arrive(fqfull0 + 8 * q);
            ++fq[which_q];
        };

        Walk wk(p, C, c);
        while (wk.next_entry()) {
            const StreamEntry& E = p.e[wk.ei];
            const int M = E.M, N = E.N;
            const uint32_t KB = wk.KB, u0 = wk.u0, u1 = wk.u1;
            bool have_first = false, have_last = false;
            uint32_t last_rt = 0, n_full = 0;
            for (uint32_t tp = wk.t_first; tp <= wk.t_last; tp += max_tiles, ++item) {
                const uint32_t ntiles = min((uint32_t)max_tiles, wk.t_last - tp + 1);
                const uint32_t ab = item & 1;
                float* part = tile_part + (size_t)ab * part_floats;
                guard.wait_mbar(accfull0 + 8 * ab, (item >> 1) & 1);
                for (uint32_t tl = 0; tl < ntiles; ++tl) {
                    const uint32_t rt = tp + tl;
                    const bool cb = u0 <= rt * KB, ce = (rt + 1) * KB <= u1;
                    if (cb && ce) ++n_full;
                    else if (ce) have_first = true;
                    else { have_last = true; last_rt = rt; }
                }
                // combine the compute warps in a fixed order, clear the buffer, route every tile
                for (int idx = et; idx < (int)ntiles * elems; idx += kEpiThreads) {
                    const uint32_t tl = idx / elems;
                    const int e = idx % elems;
                    float* src = part + ((size_t)tl * kComputeWarps) * elems + e;
                    float sum = 0.f;
#pragma unroll
                    for (int w = 0; w < kComputeWarps; ++w) {
                        sum += src[w * elems];
                        src[w * elems] = 0.f;
                    }
                    const uint32_t rt = tp + tl;
                    const bool cb = u0 <= rt * KB, ce = (rt + 1) * KB <= u1;
                    if (cb && ce) {
                        int row, tok;
                        decode(e, row, tok);
                        if (tok < M) E.y[(size_t)tok * N + rt * 16 + row] = __float2bfloat16_rn(sum);
                    } else if (ce) {
                        stash_first[e] = sum;  // cut at its beginning: completed by this CTA's fixer
                    } else {
                        stash_last[e] = sum;   // continues in the next CTA: published by the fixer
                    }
                }
                epi_sync();
                if (et == 0) mbar_arrive(accempty0 + 8 * ab);
            }
            if (et == 0 && n_full && p.tiles_done) {  // outputs of whole tiles are out (ordered by the barrier above)
                __threadfence();
                red_release_add(p.tiles_done, n_full);
            }
            // cross-CTA work of this entry, in the order that cannot chain CTAs: publish first, complete second
            if (have_last) push(0, kRecContrib, wk.ei, (last_rt == wk.t_first) ? 0u : 1u, stash_last);
            if (have_first) push(1, kRecFinish, wk.ei, wk.t_first, stash_first);
        }
        push(0, kRecEnd, 0, 0, nullptr);
        push(1, kRecEnd, 0, 0, nullptr);
    } else if (tid < kComputeThreads + kEpiThreads + kFixThreads) {
        // =============================== fixer warps ===============================
        // Warp 0 publishes this CTA's contributions to row tiles that continue in the next CTA, warp 1 completes
        // the tile at the start of the slice from the contributions of earlier CTAs.  A contribution is a set of
        // {value, tag} pairs (one 8-byte store per element, tag = entry index + 1) in slot entry % kSlotDepth of
        // the publishing CTA; the completing CTA polls the pairs, adds them in CTA order and clears them, which
        // frees the slot.  Neither warp is ever waited for by the compute warps.
        const int lane = tid & 31;
        const int fw = (tid - (kComputeThreads + kEpiThreads)) >> 5;  // 0: contributions, 1: completions
        unsigned long long* slots = reinterpret_cast<unsigned long long*>(p.slots);
        for (uint32_t fq = 0;; ++fq) {
            const uint32_t q = fw * kFixDepth + fq % kFixDepth, round = fq / kFixDepth;
            guard.wait_mbar(fqfull0 + 8 * q, round & 1);
            const FixRec& r = fixq[q];
            const int type = r.type;
            if (*poisoned || type == kRecEnd) break;
            const uint32_t tag = (uint32_t)r.ei + 1u, ring_i = (uint32_t)r.ei % kSlotDepth;
            if (type == kRecContrib) {
                unsigned long long* slot = slots + (((size_t)c * 2 + r.arg) * kSlotDepth + ring_i) * kElemsMax;
                for (int e = lane; e < elems; e += 32) {
                    // the slot last served entry ei - kSlotDepth: whoever completed that tile has cleared it
                    guard.wait_flag([&] { return __ldcg(slot + e) == 0ull; });
                    __stcg(slot + e, ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(r.data[e]));
                }
            } else {  // kRecFinish
                const StreamEntry& E = p.e[r.ei];
                const uint32_t KB = (uint32_t)E.K >> 7, units = ((uint32_t)E.N >> 4) * KB;
                const uint32_t rt = r.arg;
                const uint32_t c_lo = owner_of(rt * KB, units, C);
                for (int e = lane; e < elems; e += 32) {
                    float sum = 0.f;
                    for (uint32_t cc = c_lo; cc < c; ++cc) {
                        uint32_t which;
                        if (!contributor_slot(cc, rt, units, KB, C, which)) continue;
                        unsigned long long* src = slots + (((size_t)cc * 2 + which) * kSlotDepth + ring_i) * kElemsMax + e;
                        unsigned long long v = 0ull;
                        guard.wait_flag([&] { v = __ldcg(src); return (uint32_t)(v >> 32) == tag; });
                        if ((uint32_t)(v >> 32) == tag) {
                            sum += __uint_as_float((uint32_t)v);
                            __stcg(src, 0ull);  // consumed: the slot may be reused
                        }
                    }
                    sum += r.data[e];
                    int row, tok;
                    if (elems == 16) {
                        row = (e >> 1) + ((e & 1) ? 8 : 0);
                        tok = 0;
                    } else {
                        row = (e >> 3) + ((e & 1) ? 8 : 0);
                        tok = (e >> 1) & 3;
                    }
                    if (tok < E.M) E.y[(size_t)tok * E.N + rt * 16 + row] = __float2bfloat16_rn(sum);
                }
                __syncwarp();
                if (lane == 0 && p.tiles_done) {
                    __threadfence();
                    red_release_add(p.tiles_done, 1u);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(fqempty0 + 8 * q);
        }
    } else if (tid < kComputeThreads + kEpiThreads + kFixThreads + kStagerThreads) {
        // =============================== activation stager (3 warps) ===============================
        // The rows of x arrive by bulk copy as they are.  8 columns (one 16-byte piece) per thread and step, no
        // shuffles and no atomics: (A) max |x| of every piece, (B) every piece reads the 16 maxima of its
        // 128-column block, converts with the block's scale, writes the two int8 planes and leaves the sum of its
        // integers, (C) one thread per block adds the 16 sums.
        const int st = tid - (kComputeThreads + kEpiThreads + kFixThreads);  // 0..95
        uint32_t xe = 0;
        Walk wk(p, C, c);
        while (wk.next_entry()) {
            const StreamEntry& E = p.e[wk.ei];
            const uint32_t KB = wk.KB;
            const uint32_t xb = xe & 1;
            unsigned char* xs_b = xs + (size_t)xb * 2 * p.x_rows * p.x_row_bytes;
            int* xsum_b = xsum + (size_t)xb * kMaxRows * p.kb_max;
            float* xscale_b = xscale + (size_t)xb * kMaxRows * p.kb_max;
            if (st == 0) {
                guard.wait_mbar(xempty0 + 8 * xb, ((xe >> 1) & 1) ^ 1);
                if (E.flags & kFlagDep) {  // the input is written by earlier entries: wait until all their tiles are out
                    const unsigned int need = E.tiles_before;
                    guard.wait_flag([&] { return ld_acquire(p.tiles_done) >= need; });
                    asm volatile("fence.proxy.async;" ::: "memory");  // the copies below read what that acquire ordered
                }
                mbar_expect_tx(xraw0, (uint32_t)E.M * (uint32_t)E.K * 2u);
                for (int r = 0; r < E.M; ++r)
                    bulk_g2s_plain(smem_u32(xraw + (size_t)r * p.kb_max * 256), E.x + (size_t)r * E.K, (uint32_t)E.K * 2u,
                                   xraw0);
            }
            guard.wait_mbar(xraw0, xe & 1);  // (the copies were issued after the compute warps released buffer xb)
            const int pieces = (int)KB * 16;  // 16-byte pieces per row, 16 per block
            for (int r = 0; r < E.M; ++r) {
                const unsigned char* xrow = xraw + (size_t)r * p.kb_max * 256;
                unsigned char* dst_hi = xs_b + (size_t)(2 * r) * p.x_row_bytes;
                unsigned char* dst_lo = dst_hi + p.x_row_bytes;
                // A: max |x| of every piece (bf16 magnitudes order like unsigned integers)
#pragma unroll 2
                for (int pc = st; pc < pieces; pc += kStagerThreads) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(xrow + (size_t)pc * 16);
                    const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
                    uint32_t amax = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) amax = max(amax, max((u[i] << 16) & 0x7FFFFFFFu, u[i] & 0x7FFF0000u));
                    pmax[pc] = amax;
                }
                stager_sync();
                // B: convert every piece with the scale of its block, leave the sum of its integers
#pragma unroll 2
                for (int pc = st; pc < pieces; pc += kStagerThreads) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(xrow + (size_t)pc * 16);
                    const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
                    const uint4* pm = reinterpret_cast<const uint4*>(pmax + (pc & ~15));
                    uint32_t amax = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint4 m4 = pm[i];
                        amax = max(amax, max(max(m4.x, m4.y), max(m4.z, m4.w)));
                    }
                    // 2^e = smallest power of two with max|x| / 2^e <= 32639: exponent field F -> e = F - 127 - 14, one
                    // more when the mantissa exceeds 32639/16384 (for bf16: all seven mantissa bits set)
                    int ef = (int)(amax >> 23);
                    if (ef < 1 || ef >= 255) ef = 127 + 14;  // zero / subnormal / non-finite block: scale 1
                    int e = ef - 127 - 14 + (((amax & 0x7FFFFFu) > 0x7EFE00u) ? 1 : 0);
                    if (e < -126) e = -126;
                    const float inv = __uint_as_float((uint32_t)(127 - e) << 23);  // 2^-e
                    // v = rint(x * 2^-e) through the 1.5 * 2^23 trick; v + 128 = 256 * hi + (lo + 128)
                    uint32_t vb[8];
                    int sum = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float f0 = fmaf(__uint_as_float(u[i] << 16), inv, 12582912.f);
                        const float f1 = fmaf(__uint_as_float(u[i] & 0xFFFF0000u), inv, 12582912.f);
                        const int q0 = (int)(__float_as_uint(f0) - 0x4B400000u), q1 = (int)(__float_as_uint(f1) - 0x4B400000u);
                        sum += q0 + q1;
                        vb[2 * i] = (uint32_t)(q0 + 128);
                        vb[2 * i + 1] = (uint32_t)(q1 + 128);
                    }
                    // byte 0 of each (v + 128) is lo + 128, byte 1 is hi
                    uint2 lo, hi;
                    lo.x = __byte_perm(__byte_perm(vb[0], vb[1], 0x0040), __byte_perm(vb[2], vb[3], 0x0040), 0x5410) ^ 0x80808080u;
                    lo.y = __byte_perm(__byte_perm(vb[4], vb[5], 0x0040), __byte_perm(vb[6], vb[7], 0x0040), 0x5410) ^ 0x80808080u;
                    hi.x = __byte_perm(__byte_perm(vb[0], vb[1], 0x0051), __byte_perm(vb[2], vb[3], 0x0051), 0x5410);
                    hi.y = __byte_perm(__byte_perm(vb[4], vb[5], 0x0051), __byte_perm(vb[6], vb[7], 0x0051), 0x5410);
                    *reinterpret_cast<uint2*>(dst_hi + (size_t)pc * 8) = hi;
                    *reinterpret_cast<uint2*>(dst_lo + (size_t)pc * 8) = lo;
                    psum[pc] = sum;
                    if ((pc & 15) == 0) xscale_b[r * p.kb_max + (pc >> 4)] = __uint_as_float((uint32_t)(127 + e) << 23);
                }
                stager_sync();
                // C: block sums
                for (int kb = st; kb < (int)KB; kb += kStagerThreads) {
                    const int4* ps = reinterpret_cast<const int4*>(psum + kb * 16);
                    int sum = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int4 v = ps[i];
                        sum += (v.x + v.y) + (v.z + v.w);
                    }
                    xsum_b[r * p.kb_max + kb] = sum;
                }
            }
            stager_sync();
            if (st == 0) mbar_arrive(xfull0 + 8 * xb);
            ++xe;
        }
    } else {
        // =============================== producer (one thread) ===============================
        if (tid == kThreads - 32) {
            uint32_t s = 0, ph = 0, issued = 0;
            Walk wk(p, C, c);
            while (wk.next_entry()) {
                const unsigned char* wbase = p.e[wk.ei].w;
                for (uint32_t tp = wk.t_first; tp <= wk.t_last; tp += max_tiles) {
                    const uint32_t pu0 = max(wk.u0, tp * wk.KB), pu1 = min(wk.u1, (tp + max_tiles) * wk.KB);
                    for (uint32_t cu = pu0; cu < pu1; cu += kStageUnits, ++issued) {
                        const uint32_t n = min((uint32_t)kStageUnits, pu1 - cu);
                        guard.wait_mbar(empty0 + 8 * s, ph ^ 1);
                        mbar_expect_tx(full0 + 8 * s, n * kUnitBytes);
                        bulk_g2s_plain(smem_u32(ring + (size_t)s * kStageBytes), wbase + (size_t)cu * kUnitBytes,
                                       n * kUnitBytes, full0 + 8 * s);
                        if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
                    }
                }
            }
            // every copy this thread issued must have landed before the CTA may retire: walk back over the
            // last `stages` chunks (s, ph now name the slot after the last one issued)
            for (uint32_t back = 0; back < (uint32_t)p.stages && back < issued; ++back) {
                if (s == 0) { s = p.stages; ph ^= 1; }
                --s;
                guard.wait_mbar(full0 + 8 * s, ph);
            }
        }
    }
    // nobody leaves before every copy has landed and everybody is done with shared memory
    __syncthreads();
}

// One thread per 32-bit word of the output: 256 code words + 16 {scale, zero} words per unit.
__global__ void __launch_bounds__(256) pack_stream_kernel(const uint8_t* __restrict__ codes,
                                                          const uint16_t* __restrict__ scales,
                                                          const uint16_t* __restrict__ zeros, int N, int K, int G,
                                                          uint32_t* __restrict__ out) {
    const int KB = K >> 7, ng = K / G, bpg = G >> 7;
    const long long total = (long long)(N >> 4) * KB * 272;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long unit = i / 272;
        const int w = (int)(i % 272);
        const int rt = (int)(unit / KB), kb = (int)(unit % KB);
        uint32_t word = 0;
        if (w < 256) {
            const int row = w >> 4, wi = w & 15;
            const uint2 cc = *reinterpret_cast<const uint2*>(codes + (size_t)(rt * 16 + row) * K + (size_t)kb * 128 + wi * 8);
            // byte b of the word: column b in the low nibble, column 4 + b in the high nibble
            word = (cc.x & 0x0F0F0F0Fu) | ((cc.y & 0x0F0F0F0Fu) << 4);
        } else {
            const size_t gi = (size_t)(rt * 16 + (w - 256)) * ng + kb / bpg;
            word = (uint32_t)scales[gi] | ((uint32_t)zeros[gi] << 16);
        }
        out[i] = word;
    }
}

inline int elems_for(int x_rows) { return x_rows == 1 ? 16 : 64; }
inline int max_tiles_for(int x_rows) { return x_rows == 1 ? 8 : 2; }

size_t smem_fixed_bytes(int x_rows, int x_row_bytes, int kb_max) {
    return (size_t)2 * max_tiles_for(x_rows) * kComputeWarps * elems_for(x_rows) * 4 + 2 * kElemsMax * 4 +
           (size_t)2 * kFixDepth * (16 + kElemsMax * 4) + (size_t)4 * x_rows * x_row_bytes + (size_t)x_rows * kb_max * 256 +
           (size_t)4 * kMaxRows * kb_max * 4 + (size_t)2 * 16 * kb_max * 4 + (10 + 4 * kFixDepth) * 8 + 64 /* flag + slack */;
}

constexpr size_t kSmemLimit = 232448;  // 227 KiB per CTA

int stages_for(int x_rows, int x_row_bytes, int kb_max) {
    const size_t fixed = smem_fixed_bytes(x_rows, x_row_bytes, kb_max);
    if (fixed >= kSmemLimit) return 0;
    long s = (long)((kSmemLimit - fixed) / (kStageBytes + 16));
    if (s > 12) s = 12;
    return (int)s;
}

}  // namespace

bool w4a16_stream_supported(int M, int N, int K, int G) {
    if (M < 1 || M > kMaxRows || N < 16 || N % 16 != 0 || K % 128 != 0 || G % 128 != 0) return false;
    return stages_for(M, K + kRowPad, K / 128) >= 3;
}

size_t w4a16_stream_weight_bytes(int N, int K) { return (size_t)(N / 16) * (K / 128) * kUnitBytes; }

size_t w4a16_stream_workspace() { return (size_t)kWsHeader + (size_t)num_sms() * 2 * kSlotDepth * kSlotBytes; }

qil_status launch_pack_stream_w4(const uint8_t* codes, const void* scales, const void* zeros, int N, int K, int G,
                                 void* out, cudaStream_t st) {
    const long long words = (long long)(N / 16) * (K / 128) * 272;
    long long blocks = (words + 255) / 256;
    const long long cap = (long long)num_sms() * 16;
    if (blocks > cap) blocks = cap;
    pack_stream_kernel<<<(int)blocks, 256, 0, st>>>(codes, reinterpret_cast<const uint16_t*>(scales),
                                                    reinterpret_cast<const uint16_t*>(zeros), N, K, G,
                                                    reinterpret_cast<uint32_t*>(out));
    return launch_status();
}

// Every entry must satisfy w4a16_stream_supported().  entries[i].flags bit 0 = QIL_DEP_PREVIOUS.
qil_status launch_w4a16_stream(const qil_linear_desc* entries, int count, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (ws == nullptr || ws_bytes < w4a16_stream_workspace()) return QIL_ERR_WORKSPACE;
    static StreamParams p;  // 12 KiB: kept off the caller's stack; guarded by the mutex below
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    const int C = num_sms();
    for (int base = 0; base < count; base += kMaxEntries) {
        const int n = count - base < kMaxEntries ? count - base : kMaxEntries;
        int x_rows = 1, kmax = 128;
        bool any_dep = false;
        uint32_t tiles = 0;
        for (int i = 0; i < n; ++i) {
            const qil_linear_desc& d = entries[base + i];
            StreamEntry& e = p.e[i];
            e.x = reinterpret_cast<const uint16_t*>(d.x);
            e.w = reinterpret_cast<const unsigned char*>(d.qweight);
            e.y = reinterpret_cast<__nv_bfloat16*>(d.y);
            e.N = d.N; e.K = d.K; e.M = d.M;
            // the first entry of a launch never waits: earlier launches are ordered by the stream
            e.flags = (i > 0) ? (d.flags & kFlagDep) : 0;
            // an entry right before a dependent one takes whole row tiles per CTA when there are enough of them:
            // a little imbalance is cheaper than completing shared tiles while everybody waits for the result
            if (i + 1 < n && (entries[base + i + 1].flags & kFlagDep) && d.N / 16 >= C) e.flags |= kFlagAligned;
            e.tiles_before = tiles;
            e.pad = 0;
            tiles += (uint32_t)(d.N / 16);
            any_dep |= (e.flags & kFlagDep) != 0;
            if (d.M > x_rows) x_rows = d.M;
            if (d.K > kmax) kmax = d.K;
        }
        p.count = n;
        p.x_rows = x_rows;
        p.x_row_bytes = kmax + kRowPad;
        p.kb_max = kmax / 128;
        p.stages = stages_for(p.x_rows, p.x_row_bytes, p.kb_max);
        if (p.stages < 3) return QIL_ERR_UNSUPPORTED;
        p.elems = elems_for(p.x_rows);
        p.max_tiles = max_tiles_for(p.x_rows);
        p.status = reinterpret_cast<int*>(ws);
        p.tiles_done = any_dep ? reinterpret_cast<unsigned int*>(ws) + 1 : nullptr;
        p.slots = reinterpret_cast<unsigned char*>(ws) + kWsHeader;
        if (any_dep && cudaMemsetAsync(reinterpret_cast<unsigned int*>(ws) + 1, 0, 4, st) != cudaSuccess) {
            (void)cudaGetLastError();
            return QIL_ERR_CUDA;
        }
        const size_t smem = smem_fixed_bytes(p.x_rows, p.x_row_bytes, p.kb_max) + (size_t)p.stages * (kStageBytes + 16);
        if (cudaFuncSetAttribute(w4a16_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess) {
            (void)cudaGetLastError();
            return QIL_ERR_CUDA;
        }
        w4a16_stream_kernel<<<C, kThreads, smem, st>>>(p);
        const qil_status s = launch_status();
        if (s != QIL_OK) return s;
    }
    return QIL_OK;
}

}  // namespace qil
