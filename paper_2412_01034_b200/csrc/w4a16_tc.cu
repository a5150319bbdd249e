// Weight-only 4-bit decode linears on the 5th-generation tensor cores (tcgen05), as one
// persistent kernel over a list of linears (the memory-bound decode stage of the paper's
// OpenVLA deployment, Sec. 5.4 / App. A.4.2; M <= 4 activation rows).
//
// The kernel is bound by HBM only if the SM spends very few instructions per weight.  A packed
// byte holds two codes, b = lo + 16 hi.  The tensor core multiplies the RAW bytes, read straight
// from the shared-memory ring, by the activations under the high nibbles (x_c), and the MASKED
// bytes (b & 0x0F: one logic instruction per 8 weights, written to tensor memory by the thread that
// owns the weight row) by 16 x_a - x_c, x_a being the activations under the low nibbles:
//     sum b x_c + sum lo (16 x_a - x_c) = 16 (sum lo x_a + sum hi x_c).
// Both are tcgen05.mma kind::i8 (128 rows x 8 columns x 32 bytes) with exact int32 accumulators in
// tensor memory.  The activations are converted once per linear to 16-bit block fixed point - per
// 128 columns a power-of-two scale 2^e and integers v - and enter as signed-byte planes (two for
// x_c, three for 16 x_a - x_c), K-major in shared memory.  Per 128-column block the epilogue
// thread of a weight row reads the accumulators back (tcgen05.ld) and folds scale and zero point:
//     y += s_w * 2^e * (((256 R1 + R0) + (65536 T2 + 256 T1 + T0)) / 16 - z * X),  X = sum of the block's v.
//
// Data layout (QIL_LAYOUT_STREAM128): unit u = (row tile of 128 rows, column block of 128)
// is 8704 bytes: 4 chunks (32 columns each) x 128 rows x 16 bytes of codes, byte b of
// word m of a chunk holding column 8m+b (low nibble) and 8m+4+b (high nibble); then
// 128 x {fp16 scale, fp16 zero}.  Rows beyond N are zero.  A linear is one contiguous
// stream of units.  The units of all entries of a phase (a run of entries that do not wait for each
// other) form one stream of which CTA c of C owns units [c q + min(c, r), ...), q = units / C,
// r = units % C (see launch_w4a16_tc).
//
// Roles in a CTA (one CTA per SM, alive for the whole list):
//   producer (1 thread)    streams the CTA's units through a shared-memory ring (cp.async.bulk +
//                          mbarrier), running ahead across linears as far as the ring allows, so
//                          HBM keeps streaming while the consumers wait for a dependency;
//   unpack warpgroups (2)  take turns on units: shared memory -> nibble split -> tensor memory;
//   MMA issuers (kGroup x 1 thread) units are handled in groups of kGroup (3), issuer w takes slot w of
//                          every group: four tcgen05.mma per unit, completion by tcgen05.commit;
//   epilogue warpgroup     thread =
//                          weight row: accumulators -> fp32 row sums (kept in registers over the units
//                          of a row tile); writes the bf16 outputs of row tiles the CTA owns entirely,
//                          or hands over the partial sums of a row tile it shares;
//   stager (4 warps)       waits for QIL_DEP_PREVIOUS, loads and converts the activation blocks the
//                          CTA's units need, into a ring of up to four buffers (up to three linears ahead);
//   fixer (4 warps)        all cross-CTA work, linear i's shared row tiles belonging to team i % 2: the
//                          team's publishing warp writes the partial sums of a row tile that ends in
//                          another CTA as {value, tag} pairs (one 8-byte store each, tag = entry index
//                          + 1) into a ring of slots in the workspace; its completing warp finishes the
//                          row tile whose end the CTA owns by adding the contributions in CTA order
//                          (bit-reproducible) and counts finished quarter tiles for the dependency
//                          counter.  Publishing never waits behind completing.
// No role uses a named barrier: every hand-over is an mbarrier or a flag in global memory, and
// every wait is bounded (2 s unless set otherwise).  When a wait runs out, QIL_ERR_TIMEOUT is recorded in the
// workspace status word (with the place in words 2..5 of the workspace), every role stops at its
// next wait without issuing further work, outstanding copies and tensor-core operations are
// waited for, tensor memory is released and the kernel returns.
#include <algorithm>
#include <atomic>
#include <mutex>

#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kUnitRows = 128;
constexpr int kUnitBytes = 8192 + 512;
// Role counts: the values below measured fastest on the Llama-2-7B list (a second read-out warpgroup, more units per
// read-out pass and polling instead of sleeping waits all measured slower).
constexpr int kNumWg = 2;                        // unpack warpgroups
constexpr int kUnpackThreads = 128 * kNumWg;
constexpr int kEpiBase = kUnpackThreads;         // the read-out warpgroup (its warps keep warp % 4 = lane quarter)
constexpr int kStagerBase = kEpiBase + 128;
constexpr int kFixBase = kStagerBase + 128;
constexpr int kFixTeams = 2;                     // fixer teams: entry i's shared tiles belong to team i % kFixTeams;
constexpr int kFixThreads = 64 * kFixTeams;      // a team is a publishing and a completing warp (a lane takes four rows)
constexpr int kGroup = 3;                        // units per group: one per MMA issuer, one epilogue pass
constexpr int kMmaBase = kFixBase + kFixThreads; // kGroup warps, one issuing thread each
constexpr int kProdBase = kMmaBase + 32 * kGroup;  // one warp, one thread issues
constexpr int kThreads = kProdBase + 32;
static_assert(kThreads <= 1024, "block size");
constexpr int kNG = 4;                           // groups in flight in tensor memory
constexpr int kNB = kGroup * kNG;                // = units in flight
constexpr int kTmemCols = 512;
// tensor-memory columns: per unit 16 of masked low nibbles (A), 8 accumulators of the raw-byte products and 8 (16 with
// four activation rows) of the masked ones, 1 of {scale, zero}
constexpr int kColD = 16 * kNB;
__host__ __device__ constexpr int d_unit_cols(int xr) { return 8 + (xr == 4 ? 16 : 8); }
__host__ __device__ constexpr int col_meta(int xr) { return kColD + d_unit_cols(xr) * kNB; }
static_assert(col_meta(4) + kNB <= kTmemCols, "tensor memory budget");
constexpr int kMaxXBufs = 4;                     // activation buffers at most
constexpr int kHandDepth = 2 * kFixTeams;        // hand-over buffers between the epilogue and the fixers: two per team
constexpr int kMaxEntries = 256;
constexpr int kMaxRows = 4;                      // activation rows
constexpr int kSlotDepth = 4;                    // ring of slots per (CTA, first / last tile), indexed by entry
static_assert(kSlotDepth % kFixTeams == 0, "a slot is always written by the same fixer warp, in entry order");
constexpr int kSlotElems = kMaxRows * kUnitRows; // {value, tag} pairs of 8 bytes
constexpr int kWsHeader = 256;
constexpr int kFlagDep = 1;
constexpr int kFlagNever = 2;
constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;

struct TcEntry {  // 56 bytes
    const uint16_t* x;
    const unsigned char* w;
    __nv_bfloat16* y;
    int N, K, M, flags;
    uint32_t tiles_before;  // row tiles of all earlier entries of this launch
    uint32_t q, rem;        // units of the entry's phase / CTAs, and the remainder
    uint32_t base;          // units of the phase before this entry
};

struct TcParams {
    TcEntry e[kMaxEntries];
    int count;
    int stages;
    int nb_max;      // 128-column blocks an activation buffer holds (>= the blocks a CTA touches in any entry)
    int xbufs;       // activation buffers (entries the stager may run ahead)
    int xbuf_bytes;  // one activation operand buffer
    unsigned long long wait_ns;  // limit of every device-side wait
    int* status;
    unsigned int* tiles_done;
    unsigned char* slots;
};

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// (a failed try_wait suspends the thread in hardware for a few microseconds or until the phase completes)
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
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t lds_acquire(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_release(uint32_t addr, uint32_t v) {
    asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const unsigned int* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(unsigned int* p, uint32_t v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t (&v)[16]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(addr),
                 "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
                 "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
                 : "memory");
}
__device__ __forceinline__ void tmem_st1(uint32_t addr, uint32_t v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t tmem_ld1(uint32_t addr) {
    uint32_t v;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
// kCols consecutive 32-bit columns of the thread's lane
template <int kCols>
__device__ __forceinline__ void tmem_ld(uint32_t addr, uint32_t (&v)[8]) {
    if constexpr (kCols == 2) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : "=r"(v[0]), "=r"(v[1]) : "r"(addr));
    } else if constexpr (kCols == 4) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3])
                     : "r"(addr));
    } else {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                     : "r"(addr));
    }
}
// the accumulator columns of the masked-byte products: 3 per activation row
template <int kXR>
__device__ __forceinline__ void tmem_ld_m(uint32_t addr, uint32_t (&v)[16]) {
    if constexpr (kXR == 1) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(addr));
    } else if constexpr (kXR == 2) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                     : "r"(addr));
    } else {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
              "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
            : "r"(addr));
    }
}
// shared-memory operand descriptor: K-major, no swizzle, 8-row x 16-byte core matrices `lbo` bytes apart along K
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo) {
    uint64_t d = (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(128u >> 4) << 32;  // stride between 8-row groups: unused with 8 columns
    d |= (uint64_t)1 << 46;            // descriptor version of this architecture
    return d;
}
// D[128 x kN] (+)= A[128 x 32 u8, tensor memory] * B[kN x 32 s8, shared memory]^T, int32 accumulate
template <int kN>
__device__ __forceinline__ void mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t accumulate) {
    // instruction descriptor: D = s32 (2 at bit 4), A = u8 (0 at bit 7), B = s8 (1 at bit 10), both K-major,
    // N >> 3 at bit 17, M >> 4 at bit 24
    constexpr uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | (((uint32_t)kN >> 3) << 17) | ((128u >> 4) << 24);
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// D[128 x 8] (+)= A[128 x 32 u8, shared memory] * B[8 x 32 s8, shared memory]^T, int32 accumulate
__device__ __forceinline__ void mma_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
    constexpr uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | ((8u >> 3) << 17) | ((128u >> 4) << 24);
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// ---- bounded waits ----------------------------------------------------------------------------
// A wait returns true when what it waited for has happened, false when the kernel is being abandoned: a wait ran out
// (here or in another role; the shared flag `poisoned` is then set and QIL_ERR_TIMEOUT recorded).  A role that gets
// false stops working and goes to the end of the kernel: it issues no further copies, tensor-core operations or
// barrier arrivals.
struct Guard {
    int* status;
    volatile int* poisoned;
    unsigned long long limit;  // nanoseconds
    static __device__ __forceinline__ unsigned long long now_ns() {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        return t;
    }
    // Diagnostics of the first wait that ran out, in words 2..5 of the workspace header: 1 + CTA, thread,
    // shared-memory address of the barrier (0 for a flag in global memory), parity waited for.
    static __device__ __forceinline__ void note_timeout(int* status, uint32_t bar, uint32_t parity) {
        if (atomicCAS(reinterpret_cast<unsigned int*>(status) + 2, 0u, 1u + blockIdx.x) == 0u) {
            status[3] = (int)threadIdx.x;
            status[4] = (int)bar;
            status[5] = (int)parity;
        }
    }
    __device__ __forceinline__ bool wait_mbar(uint32_t bar, uint32_t parity) const {
        if (mbar_try_wait(bar, parity)) return true;
        return wait_mbar_slow(status, poisoned, limit, bar, parity);
    }
    // (out of line, scalar arguments: the common case above stays one instruction and a branch)
    static __device__ __noinline__ bool wait_mbar_slow(int* status, volatile int* poisoned, unsigned long long limit,
                                                       uint32_t bar, uint32_t parity) {
        if (*poisoned) return false;
        const unsigned long long t0 = now_ns();
        for (;;) {
            if (mbar_try_wait(bar, parity)) return true;
            if (*poisoned) return false;
            if (now_ns() - t0 > limit) break;
        }
        *poisoned = 1;
        atomicOr(status, (int)QIL_ERR_TIMEOUT);
        note_timeout(status, bar, parity);
        return false;
    }
    // Waits until the counter at shared address `cnt` (one writer, never decreasing) has reached `need`.  The
    // counter is the truth; the mbarrier `bar`, which completes a phase each time all such counters have advanced,
    // only lets the thread sleep in between (its parity alone could not tell one completed phase from three).
    __device__ __forceinline__ bool wait_count(uint32_t cnt, uint32_t need, uint32_t bar) const {
        for (;;) {
            const uint32_t v = lds_acquire(cnt);
            if (v >= need) return true;
            if (!wait_mbar(bar, v & 1)) return false;
        }
    }
    template <typename Pred>
    __device__ __forceinline__ bool wait_flag(Pred done) const {
        unsigned long long t0 = 0;
#pragma unroll 1
        for (uint32_t i = 0;; ++i) {  // (one copy of the predicate's code: the kernel is sensitive to its size)
            if (done()) return true;
            if (i == 0) {
                if (*poisoned) return false;
                t0 = now_ns();
            }
            if (i > 8) __nanosleep(i < 64 ? 32 : 256);
            if ((i & 15u) == 15u) {
                if (*poisoned) return false;
                if (now_ns() - t0 > limit) break;
            }
        }
        *poisoned = 1;
        atomicOr(status, (int)QIL_ERR_TIMEOUT);
        note_timeout(status, 0u, 0u);
        return false;
    }
};

// ---- who owns which units ---------------------------------------------------------------------
__device__ __forceinline__ void slice_of(uint32_t q, uint32_t rem, uint32_t c, uint32_t& u0, uint32_t& u1) {
    u0 = c * q + min(c, rem);
    u1 = u0 + q + (c < rem ? 1u : 0u);
}
// The entries in which one CTA owns units.  The CTA's slice of every entry is worked out once, at the start of the
// kernel, into a table in shared memory ({first unit, first row tile, units | row tiles touched << 16, first
// column block | column blocks per row tile << 16}): six roles walk the list, and slicing costs divisions.
struct Walk {
    const uint4* plan;
    int count;
    int ei;
    uint32_t KB, u0, u1, t_first, t_last, kb0;
    __device__ Walk(const uint4* plan_, int count_) : plan(plan_), count(count_), ei(-1) {}
    __device__ __forceinline__ bool next_entry() {
        for (++ei; ei < count; ++ei) {
            const uint4 e = plan[ei];
            const uint32_t n = e.z & 0xFFFFu;
            if (n != 0u) {
                u0 = e.x;
                u1 = e.x + n;
                t_first = e.y;
                t_last = e.y + (e.z >> 16) - 1u;
                kb0 = e.w & 0xFFFFu;
                KB = e.w >> 16;
                return true;
            }
        }
        return false;
    }
};

// ring-style counter: index in [0, n) and the phase parity of its current use
struct Cyc {
    uint32_t idx, ph, n;
    __device__ Cyc(uint32_t n_) : idx(0), ph(0), n(n_) {}
    __device__ __forceinline__ void step() {
        if (++idx == n) { idx = 0; ph ^= 1; }
    }
};

// kXR = activation rows staged (1, 2 or 4; >= every M of the launch)
template <int kXR>
__global__ void __launch_bounds__(kThreads, 1) w4a16_tc_kernel(const __grid_constant__ TcParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    // Activation operands: per 16-byte K chunk the planes of all activation rows follow each other (2 per row for
    // x_c, 3 per row for 16 x_a - x_c); the rows of the tensor core's 8- or 16-row window beyond them belong to the
    // next chunks and only feed accumulator columns nobody reads.
    constexpr int kLboR = 32 * kXR, kLboM = 48 * kXR;
    constexpr int kRCols = 2 * kXR, kMCols = 3 * kXR;   // accumulator columns in use
    constexpr int kMskN = kXR == 4 ? 16 : 8;            // columns of the masked-byte MMA
    constexpr int kDUnit = d_unit_cols(kXR), kColMeta = col_meta(kXR);
    const int tid = threadIdx.x;
    const uint32_t c = blockIdx.x;

    // ---- carve shared memory ----
    unsigned char* ring = smem;                                                     // [stages][kUnitBytes]
    unsigned char* xs = ring + (size_t)p.stages * kUnitBytes;                       // [xbufs][xbuf_bytes]
    int2* xblk = reinterpret_cast<int2*>(xs + (size_t)p.xbufs * p.xbuf_bytes);      // [xbufs][kXR][nb_max] {sum v, bits of 2^e}
    float* hand = reinterpret_cast<float*>(xblk + p.xbufs * kXR * p.nb_max);        // [kHandDepth][2][kXR][128]
    uint64_t* bars = reinterpret_cast<uint64_t*>(hand + kHandDepth * 2 * kXR * kUnitRows);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + p.stages);
    uint64_t* b2 = bars + 2 * p.stages;
    // afull: per unit slot; dfull / dempty: per group of kGroup slots
    const uint32_t afull0 = smem_u32(b2), dfull0 = smem_u32(b2 + kNB), dempty0 = smem_u32(b2 + kNB + kNG);
    uint64_t* b3 = b2 + 3 * kNB;
    const uint32_t xfull0 = smem_u32(b3), xempty0 = smem_u32(b3 + kMaxXBufs);
    const uint32_t mdone0 = smem_u32(b3 + 12);  // (slots 8..11 are unused)
    const uint32_t hfull0 = smem_u32(b3 + 12 + kGroup), hempty0 = smem_u32(b3 + 12 + kGroup + kHandDepth);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(b3 + 12 + kGroup + 2 * kHandDepth);
    volatile int* poisoned = reinterpret_cast<volatile int*>(tmem_slot + 1);
    // rd[gs][q]: groups of slot group gs that epilogue warp q (tensor-memory lanes 32q..32q+31) has read out
    const uint32_t rd0 = smem_u32(tmem_slot + 2);
    uint4* plan = reinterpret_cast<uint4*>((reinterpret_cast<uintptr_t>(tmem_slot + 2 + 4 * kNG) + 15) & ~(uintptr_t)15);  // [count] this CTA's slice of every entry
    for (int i = tid; i < p.count; i += kThreads) {
        // the CTA's slice of the entry's phase, cut down to the entry (unit numbers inside the entry)
        uint32_t ph0, ph1;
        slice_of(p.e[i].q, p.e[i].rem, c, ph0, ph1);
        const uint32_t pKB = (uint32_t)p.e[i].K >> 7, base = p.e[i].base;
        const uint32_t units = (((uint32_t)p.e[i].N + kUnitRows - 1u) / kUnitRows) * pKB;
        const uint32_t lo = max(ph0, base), hi = min(ph1, base + units);
        const uint32_t pu0 = lo - base, pn = hi > lo ? hi - lo : 0u;
        uint4 e = make_uint4(pu0, 0u, 0u, pKB << 16);
        if (pn != 0u) {
            e.y = pu0 / pKB;
            const uint32_t pkb0 = pu0 - e.y * pKB;
            e.z = pn | (((pkb0 + pn - 1u) / pKB + 1u) << 16);
            e.w |= pkb0;
        }
        plan[i] = e;
    }

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 5);  // the four unpack warps and the commit of the MMAs that read the raw bytes
        }
        for (int i = 0; i < kNB; ++i) mbar_init(afull0 + 8 * i, 4);
        for (int i = 0; i < kNG; ++i) {
            mbar_init(dfull0 + 8 * i, kGroup);  // one arrival per issuer
            mbar_init(dempty0 + 8 * i, 4);      // the epilogue warps
        }
        for (int i = 0; i < kMaxXBufs; ++i) {
            mbar_init(xfull0 + 8 * i, 4);  // the stager warps
            mbar_init(xempty0 + 8 * i, 4);  // the warps of the warpgroup that read the linear out
        }
        for (int i = 0; i < kGroup; ++i) mbar_init(mdone0 + 8 * i, 1);
        for (int i = 0; i < kHandDepth; ++i) {
            mbar_init(hfull0 + 8 * i, 4);
            mbar_init(hempty0 + 8 * i, 2);  // the team's publishing and completing warp
        }
        *poisoned = 0;
        for (int i = 0; i < 4 * kNG; ++i) tmem_slot[2 + i] = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < p.xbufs * p.xbuf_bytes / 4; i += kThreads) reinterpret_cast<uint32_t*>(xs)[i] = 0u;
    if (tid < 32) {  // one warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const Guard guard{p.status, poisoned, p.wait_ns};

    if (tid < kUnpackThreads) {
        // ======================= unpack warpgroups: shared memory -> nibble split -> tensor memory =======================
        const uint32_t wg = tid >> 7, r = tid & 127, lane = tid & 31;
        const uint32_t lane_base = (r & ~31u) << 16;  // this warp's quarter of the tensor-memory lanes
        const uint32_t S = (uint32_t)p.stages;
        uint32_t stage0 = 0, ph0 = 0, turn0 = 0;  // ring stage / phase / turn of the entry's first unit
        uint32_t G = 0;                           // groups so far: unit j of an entry sits in group G + j / kGroup, slot j % kGroup
        bool alive = true;
        Walk wk(plan, p.count);
        while (alive && wk.next_entry()) {
            const uint32_t n = wk.u1 - wk.u0;
            uint32_t j = wg >= turn0 ? wg - turn0 : wg + kNumWg - turn0;  // this warpgroup's first unit of the entry
            uint32_t st_i = stage0 + j, st_ph = ph0;
            if (st_i >= S) { st_i -= S; st_ph ^= 1; }
            for (; j < n; j += kNumWg) {
                const uint32_t g = G + j / kGroup, a = (g % kNG) * kGroup + j % kGroup;
                // the groups that used these columns before have been read out (by the epilogue warp of the same
                // lanes); the unit has landed
                if (!guard.wait_count(rd0 + 4 * ((g % kNG) * 4 + (r >> 5)), g / kNG, dempty0 + 8 * (g % kNG)) ||
                    !guard.wait_mbar(full0 + 8 * st_i, st_ph)) {
                    alive = false;
                    break;
                }
                tc_fence_after();
                const unsigned char* ub = ring + (size_t)st_i * kUnitBytes;
                const uint32_t ta = tmem + lane_base + 16 * a;
                constexpr uint32_t kLo = 0x0F0F0F0Fu;
                uint4 w[4];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) w[ch] = *reinterpret_cast<const uint4*>(ub + ((size_t)ch * kUnitRows + r) * 16);
                const uint32_t meta = *reinterpret_cast<const uint32_t*>(ub + 8192 + 4 * r);
                uint32_t v[16];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    v[4 * ch] = w[ch].x & kLo; v[4 * ch + 1] = w[ch].y & kLo; v[4 * ch + 2] = w[ch].z & kLo; v[4 * ch + 3] = w[ch].w & kLo;
                }
                tmem_st16(ta, v);  // A of the two masked-byte MMAs: chunks 0, 1 and 2, 3 of the block
                tmem_st1(tmem + lane_base + kColMeta + a, meta);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(afull0 + 8 * a);
                    mbar_arrive(empty0 + 8 * st_i);
                }
                st_i += kNumWg;
                if (st_i >= S) { st_i -= S; st_ph ^= 1; }
            }
            G += (n + kGroup - 1) / kGroup;
            turn0 = (turn0 + n) % kNumWg;
            const uint32_t adv = stage0 + n;
            uint32_t wrapped = adv;  // (subtractions instead of a division: per-linear code is expensive here)
            while (wrapped >= S) {
                wrapped -= S;
                ph0 ^= 1;
            }
            stage0 = wrapped;
        }
    } else if (tid < kStagerBase) {
        // ======================= epilogue warpgroup (thread = weight row of the unit) =======================
        const uint32_t r = (uint32_t)(tid - kEpiBase) & 127, lane = tid & 31;
        const uint32_t lane_base = (r & ~31u) << 16;
        constexpr int kEB = 1;  // units read back per tcgen05.wait::ld
        uint32_t hc = 0, G = 0;          // hc: per fixer team, two bits counting the entries handed to it
        Cyc xc(p.xbufs);
        bool alive = true;
        Walk wk(plan, p.count);
        while (alive && wk.next_entry()) {
            const TcEntry& E = p.e[wk.ei];
            const int M = E.M, N = E.N;
            const uint32_t KB = wk.KB, u0 = wk.u0, u1 = wk.u1, n = u1 - u0;
            const uint32_t t_first = wk.t_first, t_last = wk.t_last;
            const bool shares = t_first * KB < u0 || (t_last + 1) * KB > u1;  // a row tile is shared with other CTAs
            const uint32_t xb = xc.idx, xph = xc.ph;
            xc.step();
            // the two hand-over buffers of the entry's fixer team alternate
            const uint32_t team = (uint32_t)wk.ei % kFixTeams, hcnt = (hc >> (2 * team)) & 3u;
            if (shares) hc = (hc & ~(3u << (2 * team))) | (((hcnt + 1u) & 3u) << (2 * team));
            const uint32_t hbuf = 2 * team + (hcnt & 1u);
            const uint32_t hph = (hcnt >> 1) & 1u;
            if (!guard.wait_mbar(xfull0 + 8 * xb, xph)) break;
            const int2* xblk_b = xblk + (size_t)xb * kXR * p.nb_max;
            float* hand_b = hand + (size_t)hbuf * 2 * kXR * kUnitRows;
            if (shares && !guard.wait_mbar(hempty0 + 8 * hbuf, hph ^ 1u)) break;
            uint32_t n_full = 0;
            float fin[kXR];
#pragma unroll
            for (int t = 0; t < kXR; ++t) fin[t] = 0.f;
            uint32_t rt = t_first, kb = wk.kb0;
            uint32_t bi = 0;  // block inside the activation buffer, which holds the blocks from the slice's first one on, cyclically
            // the CTA's part of row tile rt is complete
            auto close_tile = [&]() {
                {
                    const bool cb = u0 <= rt * KB, ce = (rt + 1) * KB <= u1;
                    if (cb && ce) {
                        ++n_full;
                        const uint32_t row = rt * kUnitRows + r;
                        if (row < (uint32_t)N) {
#pragma unroll
                            for (int t = 0; t < kXR; ++t)
                                if (t < M) E.y[(size_t)t * N + row] = __float2bfloat16_rn(fin[t]);
                        }
                    } else {  // first tile cut at its beginning (completed by the fixer) or last tile continued elsewhere
                        float* dst = hand_b + (size_t)(ce ? 0 : 1) * kXR * kUnitRows + r;
#pragma unroll
                        for (int t = 0; t < kXR; ++t) dst[t * kUnitRows] = fin[t];
                    }
                }
#pragma unroll
                for (int t = 0; t < kXR; ++t) fin[t] = 0.f;
                kb = 0;
                ++rt;
            };
            // one unit of this warpgroup: fold scale and zero point into the row sums
            // (cr: raw-byte accumulators {x_c high, low plane}; cm: masked-byte accumulators {top, middle, low plane})
            auto consume = [&](const uint32_t (&cr)[8], const uint32_t (&cm)[16], uint32_t meta) {
                const __half2 sz = *reinterpret_cast<const __half2*>(&meta);
                const float s = __low2float(sz);
                const int z = __half2int_rz(__high2half(sz));
#pragma unroll
                for (int t = 0; t < kXR; ++t)
                    if (t < M) {
                        const int v16 = ((int)cr[2 * t] * 256 + (int)cr[2 * t + 1]) +
                                        ((int)cm[3 * t] * 65536 + (int)cm[3 * t + 1] * 256 + (int)cm[3 * t + 2]);
                        const int2 xm = xblk_b[t * p.nb_max + bi];
                        const int v = (v16 >> 4) - z * xm.x;  // (v16 is an exact multiple of 16)
                        fin[t] = fmaf((float)v, s * __int_as_float(xm.y), fin[t]);
                    }
            };
            for (uint32_t j0 = 0; alive && j0 < n; j0 += kGroup, ++G) {
                const uint32_t gs = G % kNG, nreal = min((uint32_t)kGroup, n - j0);
                if (!guard.wait_mbar(dfull0 + 8 * gs, (G / kNG) & 1)) {  // all units of the group are accumulated
                    alive = false;
                    break;
                }
                tc_fence_after();
                for (uint32_t b0 = 0; alive && b0 < nreal; b0 += kEB) {
                    uint32_t dr[kEB][8], dm[kEB][16], meta[kEB];
#pragma unroll
                    for (int i = 0; i < kEB; ++i) {
#pragma unroll
                        for (int q = 0; q < kRCols; ++q) dr[i][q] = 0u;
#pragma unroll
                        for (int q = 0; q < kMCols; ++q) dm[i][q] = 0u;
                        meta[i] = 0u;
                        if (b0 + i < nreal) {
                            const uint32_t a = gs * kGroup + b0 + i;
                            const uint32_t td = tmem + lane_base + kColD + kDUnit * a;
                            tmem_ld<kRCols>(td, dr[i]);
                            tmem_ld_m<kXR>(td + 8, dm[i]);
                            meta[i] = tmem_ld1(tmem + lane_base + kColMeta + a);
                        }
                    }
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int i = 0; i < kEB; ++i) {  // no use of the loaded registers is scheduled before the wait
#pragma unroll
                        for (int q = 0; q < kRCols; ++q) asm volatile("" : "+r"(dr[i][q]));
#pragma unroll
                        for (int q = 0; q < kMCols; ++q) asm volatile("" : "+r"(dm[i][q]));
                        asm volatile("" : "+r"(meta[i]));
                    }
                    if (b0 + kEB >= nreal) {  // the group's columns may be reused
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            // (arrival first: whoever sees the counter and refills the columns can only lead to arrivals
                            // of the barrier's next phase; the counter may also be written by the other warpgroup's warp
                            // of these lanes, for a later use of the columns, which cannot start before this one ends)
                            mbar_arrive(dempty0 + 8 * gs);
                            sts_release(rd0 + 4 * (gs * 4 + (r >> 5)), G / kNG + 1);
                        }
                    }
#pragma unroll
                    for (int i = 0; i < kEB; ++i)
                        if (alive && b0 + i < nreal) {
                            consume(dr[i], dm[i], meta[i]);
                            if (++bi == KB) bi = 0;
                            if (++kb == KB || j0 + b0 + i + 1 == n) close_tile();
                        }
                }
            }
            if (!alive) break;
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(xempty0 + 8 * xb);
                if (shares) mbar_arrive(hfull0 + 8 * hbuf);
                // the dependency counter counts quarter tiles (32 rows), so that no warp has to wait for another
                // (the release covers the other lanes' stores as well: they are ordered before it by the __syncwarp above)
                if (n_full && p.tiles_done) {
                    red_release_add(p.tiles_done, n_full);
                }
            }
        }
    } else if (tid < kFixBase) {
        // ======================= activation stager (a half warp = one 128-column block per pass) =======================
        // bf16 row -> per 128 columns: e with max|x| / 2^e <= 32639, v = rint(x / 2^e) as signed-byte planes,
        // X = sum v.  Only the blocks the CTA's units touch are converted.  K order of both operands inside a block:
        // 16-byte chunk j (32 columns), byte 4m + b = the packed byte holding columns 32j + 8m + b (low nibble, x_a)
        // and 32j + 8m + 4 + b (high nibble, x_c).  The four warps work independently.
        const int st = tid - kStagerBase, lane = tid & 31, l16 = st & 15, hw = st >> 4;
        Cyc xc(p.xbufs);
        Walk wk(plan, p.count);
        while (wk.next_entry()) {
            const TcEntry& E = p.e[wk.ei];
            const uint32_t KB = wk.KB;
            const uint32_t xb = xc.idx;
            unsigned char* xs_b = xs + (size_t)xb * p.xbuf_bytes;                  // planes of x_c
            unsigned char* xm_b = xs_b + (size_t)p.nb_max * 4 * kLboR + 256;       // planes of 16 x_a - x_c
            int2* xblk_b = xblk + (size_t)xb * kXR * p.nb_max;
            bool ok = true;
            if (lane == 0) {  // the buffer is free; the rows of x are written (quarter tiles of all earlier entries)
                ok = guard.wait_mbar(xempty0 + 8 * xb, xc.ph ^ 1);
                if (ok && (E.flags & kFlagDep)) {
                    // (kFlagNever: a count that is never reached, so that this bounded wait runs out)
                    const unsigned int need = (E.flags & kFlagNever) ? 0xFFFFFFFFu : 4u * E.tiles_before;
                    ok = guard.wait_flag([&] { return ld_acquire(p.tiles_done) >= need; });
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            const uint32_t nblk = min(KB, wk.u1 - wk.u0), kb0 = wk.kb0;
            const uint32_t m = (uint32_t)l16 & 3;
            for (int t = 0; t < E.M; ++t) {
                const uint16_t* xrow = E.x + (size_t)t * E.K;
                // up to four passes of 8 blocks at a time: their loads are all in flight before the first conversion
                for (uint32_t ib0 = 0; ib0 < nblk; ib0 += 32) {
                    uint4 raws[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t i = ib0 + 8 * q + hw;
                        uint32_t kb = kb0 + i;
                        if (kb >= KB) kb -= KB;
                        raws[q] = make_uint4(0, 0, 0, 0);
                        if (i < nblk) raws[q] = __ldcg(reinterpret_cast<const uint4*>(xrow + (size_t)kb * 128 + l16 * 8));
                    }
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) {
                        if (ib0 + 8 * q >= nblk) break;  // (uniform over the warp: the shuffles below need every lane)
                        const uint32_t i = ib0 + 8 * q + hw;
                        const bool valid = i < nblk;
                        uint32_t kb = kb0 + i;
                        if (kb >= KB) kb -= KB;
                        const uint4 raw = q == 0 ? raws[0] : q == 1 ? raws[1] : q == 2 ? raws[2] : raws[3];
                        const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
                        uint32_t amax = 0;  // bf16 magnitudes order like unsigned integers
#pragma unroll
                        for (int j = 0; j < 4; ++j) amax = max(amax, max((u[j] << 16) & 0x7FFFFFFFu, u[j] & 0x7FFF0000u));
#pragma unroll
                        for (int o = 1; o < 16; o <<= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                        // 2^e = smallest power of two with max|x| / 2^e <= 32639: exponent field F -> e = F - 127 - 14, one
                        // more when the mantissa exceeds 32639/16384 (for bf16: all seven mantissa bits set)
                        int ef = (int)(amax >> 23);
                        if (ef < 1 || ef >= 255) ef = 127 + 14;  // zero / subnormal / non-finite block: scale 1
                        int e = ef - 127 - 14 + (((amax & 0x7FFFFFu) > 0x7EFE00u) ? 1 : 0);
                        if (e < -126) e = -126;
                        const float inv = __uint_as_float((uint32_t)(127 - e) << 23);  // 2^-e
                        // v = rint(x * 2^-e) through the 1.5 * 2^23 trick
                        int vq[8];
                        int sum = 0;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float f0 = fmaf(__uint_as_float(u[j] << 16), inv, 12582912.f);
                            const float f1 = fmaf(__uint_as_float(u[j] & 0xFFFF0000u), inv, 12582912.f);
                            vq[2 * j] = (int)(__float_as_uint(f0) - 0x4B400000u);
                            vq[2 * j + 1] = (int)(__float_as_uint(f1) - 0x4B400000u);
                            sum += vq[2 * j] + vq[2 * j + 1];
                        }
#pragma unroll
                        for (int o = 1; o < 16; o <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                        if (valid) {
                            // Columns 0-3 of the piece sit under low nibbles (x_a), columns 4-7 under high nibbles (x_c).
                            // A biased integer t + 0x808080 has the bytes b_i with t = sum (b_i - 128) 256^i: its bytes
                            // XOR 0x80 are the signed planes (two for x_c, three for 16 x_a - x_c, |.| < 2^20).
                            uint32_t uc[4], um[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                uc[j] = (uint32_t)(vq[4 + j] + 0x8080);
                                um[j] = (uint32_t)(16 * vq[j] - vq[4 + j] + 0x808080);
                            }
                            const uint32_t c0 = __byte_perm(__byte_perm(uc[0], uc[1], 0x0040), __byte_perm(uc[2], uc[3], 0x0040), 0x5410) ^ 0x80808080u;
                            const uint32_t c1 = __byte_perm(__byte_perm(uc[0], uc[1], 0x0051), __byte_perm(uc[2], uc[3], 0x0051), 0x5410) ^ 0x80808080u;
                            const uint32_t m0 = __byte_perm(__byte_perm(um[0], um[1], 0x0040), __byte_perm(um[2], um[3], 0x0040), 0x5410) ^ 0x80808080u;
                            const uint32_t m1 = __byte_perm(__byte_perm(um[0], um[1], 0x0051), __byte_perm(um[2], um[3], 0x0051), 0x5410) ^ 0x80808080u;
                            const uint32_t m2 = __byte_perm(__byte_perm(um[0], um[1], 0x0062), __byte_perm(um[2], um[3], 0x0062), 0x5410) ^ 0x80808080u;
                            // piece l16 = bytes 4m .. 4m+3 of 16-byte chunk l16 / 4 of the block
                            unsigned char* dr = xs_b + (size_t)(i * 4 + (l16 >> 2)) * kLboR + (size_t)(2 * t) * 16 + 4 * m;
                            *reinterpret_cast<uint32_t*>(dr) = c1;       // high plane of x_c
                            *reinterpret_cast<uint32_t*>(dr + 16) = c0;  // low plane
                            unsigned char* dm = xm_b + (size_t)(i * 4 + (l16 >> 2)) * kLboM + (size_t)(3 * t) * 16 + 4 * m;
                            *reinterpret_cast<uint32_t*>(dm) = m2;       // top plane of 16 x_a - x_c
                            *reinterpret_cast<uint32_t*>(dm + 16) = m1;
                            *reinterpret_cast<uint32_t*>(dm + 32) = m0;
                            if (l16 == 0) xblk_b[t * p.nb_max + i] = make_int2(sum, (int)((uint32_t)(127 + e) << 23));
                        }
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMAs read xs through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(xfull0 + 8 * xb);
            xc.step();
        }
    } else if (tid < kMmaBase) {
        // ======================= fixer warps (lane = four rows of the tile): all cross-CTA work =======================
        // Entry i's shared row tiles belong to team i % kFixTeams: its publishing warp hands the CTA's part of a tile
        // that ends in another CTA over to that CTA, its completing warp finishes the tile that ends here.  The two
        // are separate warps because completing waits for other CTAs and publishing must never wait behind it (CTA c
        // would otherwise publish only after CTA c - 1 had, and so on down the grid).
        const uint32_t fw = (uint32_t)(tid - kFixBase) >> 5, team = fw >> 1, lane = tid & 31;
        const bool completer = (fw & 1u) != 0u;
        constexpr uint32_t kRowsPer = kUnitRows / 32;
        unsigned long long* slots = reinterpret_cast<unsigned long long*>(p.slots);
        uint32_t cnt = 0;  // entries this team has taken over
        bool alive = true;
        Walk wk(plan, p.count);
        while (alive && wk.next_entry()) {
            if ((uint32_t)wk.ei % kFixTeams != team) continue;
            const TcEntry& E = p.e[wk.ei];
            const int M = E.M, N = E.N;
            const uint32_t KB = wk.KB, u0 = wk.u0, u1 = wk.u1;
            const uint32_t t_first = wk.t_first, t_last = wk.t_last;
            const bool have_last = (t_last + 1) * KB > u1;                          // contributes to a tile that ends elsewhere
            const bool have_first = t_first * KB < u0 && (t_first + 1) * KB <= u1;  // completes a tile begun elsewhere
            if (!have_last && !(t_first * KB < u0)) continue;
            const uint32_t tag = (uint32_t)wk.ei + 1u, ring_i = (uint32_t)wk.ei % kSlotDepth;
            const uint32_t hbuf = 2 * team + (cnt & 1u), hph = (cnt >> 1) & 1u;
            ++cnt;
            const float* hand_b = hand + (size_t)hbuf * 2 * kXR * kUnitRows;
            if (!completer) {
                unsigned long long* my_slot = nullptr;
                if (have_last) {
                    const uint32_t which = (t_last == t_first) ? 0u : 1u;
                    my_slot = slots + (((size_t)c * 2 + which) * kSlotDepth + ring_i) * kSlotElems;
                    // the slot must have been consumed (tags cleared) by whoever completed the tile it last served;
                    // checked now, while the units are still being computed
                    alive = guard.wait_flag([&] {
                        bool is_free = true;
                        for (uint32_t h = 0; h < kRowsPer; ++h)
                            for (int t = 0; t < kXR; ++t)
                                if (t < M) is_free &= (uint32_t)(__ldcg(my_slot + t * kUnitRows + lane + 32 * h) >> 32) == 0u;
                        return is_free;
                    });
                }
                alive = alive && guard.wait_mbar(hfull0 + 8 * hbuf, hph);
                alive = __all_sync(0xffffffffu, alive);
                if (!alive) break;
                if (have_last) {
                    for (uint32_t h = 0; h < kRowsPer; ++h) {
                        const uint32_t r = lane + 32 * h;
                        for (int t = 0; t < M; ++t)
                            __stcg(my_slot + t * kUnitRows + r,
                                   ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(hand_b[(kXR + t) * kUnitRows + r]));
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(hempty0 + 8 * hbuf);
                continue;
            }
            // ---- completing warp ----
            alive = guard.wait_mbar(hfull0 + 8 * hbuf, hph);
            alive = __all_sync(0xffffffffu, alive);
            if (!alive) break;
            if (have_first) {
                // the CTAs before this one that hold units of the tile (walked backwards: cheaper here than dividing);
                // slices are counted in units of the entry's phase, the tile begins at unit tile0 of the phase
                const uint32_t tile0 = E.base + t_first * KB;
                uint32_t c_lo = c;
                while (c_lo > 0) {
                    uint32_t a0, a1;
                    slice_of(E.q, E.rem, c_lo - 1, a0, a1);
                    if (a1 <= tile0) break;
                    --c_lo;
                }
                float sum[kRowsPer][kXR];
#pragma unroll
                for (uint32_t h = 0; h < kRowsPer; ++h)
#pragma unroll
                    for (int t = 0; t < kXR; ++t) sum[h][t] = 0.f;
                for (uint32_t cc = c_lo; cc < c; ++cc) {
                    uint32_t cu0, cu1;
                    slice_of(E.q, E.rem, cc, cu0, cu1);
                    if (cu0 == cu1) continue;
                    // the tile is that CTA's first tile of the entry, or its last
                    const uint32_t which = (max(cu0, E.base) >= tile0) ? 0u : 1u;
                    unsigned long long* src = slots + (((size_t)cc * 2 + which) * kSlotDepth + ring_i) * kSlotElems + lane;
                    unsigned long long got[kRowsPer][kXR];
                    auto arrived = [&] {
                        bool all = true;
#pragma unroll
                        for (uint32_t h = 0; h < kRowsPer; ++h) {
#pragma unroll
                            for (int t = 0; t < kXR; ++t)
                                if (t < M) {
                                    got[h][t] = __ldcg(src + t * kUnitRows + 32 * h);
                                    all &= (uint32_t)(got[h][t] >> 32) == tag;
                                }
                        }
                        return all;
                    };
                    alive = guard.wait_flag(arrived);
                    alive = __all_sync(0xffffffffu, alive);
                    if (!alive) break;
#pragma unroll
                    for (uint32_t h = 0; h < kRowsPer; ++h)  // (always summed in CTA order)
#pragma unroll
                        for (int t = 0; t < kXR; ++t)
                            if (t < M) {
                                sum[h][t] += __uint_as_float((uint32_t)got[h][t]);
                                __stcg(src + t * kUnitRows + 32 * h, 0ull);  // consumed: the slot may be reused
                            }
                }
                if (!alive) break;
#pragma unroll
                for (uint32_t h = 0; h < kRowsPer; ++h) {
                    const uint32_t r = lane + 32 * h, row = t_first * kUnitRows + r;
                    if (row < (uint32_t)N) {
#pragma unroll
                        for (int t = 0; t < kXR; ++t)
                            if (t < M) E.y[(size_t)t * N + row] = __float2bfloat16_rn(sum[h][t] + hand_b[t * kUnitRows + r]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(hempty0 + 8 * hbuf);
                if (have_first && p.tiles_done) {  // the tile is written: kRowsPer quarter tiles
                    red_release_add(p.tiles_done, kRowsPer);
                }
            }
        }
    } else if (tid < kProdBase) {
        // ======================= MMA issuers (one thread in each of kGroup warps) =======================
        // Issuing one tcgen05.mma costs a thread some 50 cycles, far more than the instruction occupies the tensor
        // core at 8 columns; issuer w therefore takes slot w of every group, so kGroup units are issued in parallel.
        if ((tid & 31) == 0) {
            const uint32_t w = (uint32_t)(tid - kMmaBase) >> 5;
            uint32_t G = 0;
            Cyc xc(p.xbufs);
            bool alive = true, issued = false;
            Walk wk(plan, p.count);
            const uint64_t desc_r = smem_desc(0, kLboR), desc_m = smem_desc(0, kLboM), desc_a = smem_desc(0, kUnitRows * 16);
            constexpr uint32_t lbor16 = (uint32_t)kLboR >> 4, lbom16 = (uint32_t)kLboM >> 4;
            const uint32_t S = (uint32_t)p.stages, ring16 = smem_u32(ring) >> 4;
            uint32_t stage0 = 0;  // ring stage of the entry's first unit
            while (alive && wk.next_entry()) {
                const uint32_t KB = wk.KB, n = wk.u1 - wk.u0;
                const uint32_t xb = xc.idx;
                if (!guard.wait_mbar(xfull0 + 8 * xb, xc.ph)) break;
                xc.step();
                const uint32_t xr16 = smem_u32(xs + (size_t)xb * p.xbuf_bytes) >> 4;
                const uint32_t xm16 = xr16 + (((uint32_t)p.nb_max * 4 * kLboR + 256) >> 4);
                uint32_t kb = w, kstep = (uint32_t)kGroup;  // block of the unit inside the activation buffer: unit j sits at j % KB
                while (kb >= KB) kb -= KB;
                while (kstep >= KB) kstep -= KB;
                uint32_t st_i = stage0 + w;
                if (st_i >= S) st_i -= S;
                for (uint32_t j = w; j < (n + kGroup - 1) / kGroup * kGroup; j += kGroup, ++G) {
                    const uint32_t gs = G % kNG, gph = (G / kNG) & 1;
                    if (j < n) {
                        const uint32_t a = gs * kGroup + w;
                        if (!guard.wait_mbar(afull0 + 8 * a, gph)) {  // (the unpack warps waited for the columns to be free)
                            alive = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t ta = tmem + 16 * a, td = tmem + kColD + kDUnit * a;
                        // raw bytes of the unit in the ring: 16-byte chunk j at j * 2048, rows 16 bytes apart
                        const uint64_t a0 = desc_a | (uint64_t)(ring16 + st_i * (kUnitBytes >> 4));
                        const uint64_t br = desc_r | (uint64_t)(xr16 + kb * 4 * lbor16);
                        const uint64_t bm = desc_m | (uint64_t)(xm16 + kb * 4 * lbom16);
                        mma_i8_ss(td, a0, br, 0u);                                        // raw bytes x x_c, chunks 0, 1
                        mma_i8_ss(td, a0 + 2 * (kUnitRows * 16 >> 4), br + 2 * lbor16, 1u);  // chunks 2, 3
                        mma_i8_ts<kMskN>(td + 8, ta, bm, 0u);                             // masked bytes x (16 x_a - x_c)
                        mma_i8_ts<kMskN>(td + 8, ta + 8, bm + 2 * lbom16, 1u);
                        tc_commit(dfull0 + 8 * gs);
                        tc_commit(empty0 + 8 * st_i);  // the ring stage has been read
                        issued = true;
                    } else {
                        // The entry ends inside the group: this slot stays empty, its barriers still change phase.  Like
                        // the unpack warps the thread first waits until the groups that used these columns before have
                        // been read out: an arrival must never reach a barrier whose previous phase is still collecting.
                        for (uint32_t q = 0; alive && q < 4; ++q)
                            alive = guard.wait_count(rd0 + 4 * (gs * 4 + q), G / kNG, dempty0 + 8 * gs);
                        if (!alive) break;
                        mbar_arrive_n(afull0 + 8 * (gs * kGroup + w), 4);
                        mbar_arrive(dfull0 + 8 * gs);
                    }
                    kb += kstep;
                    if (kb >= KB) kb -= KB;
                    st_i += kGroup;
                    if (st_i >= S) st_i -= S;
                }
                stage0 += n;
                while (stage0 >= S) stage0 -= S;
            }
            // whatever happened to the other roles: the operations this thread issued are complete before tensor memory
            // is released (this wait also holds in an abandoned kernel)
            if (issued) {
                tc_commit(mdone0 + 8 * w);
                const unsigned long long t0 = Guard::now_ns();
                while (!mbar_try_wait(mdone0 + 8 * w, 0) && Guard::now_ns() - t0 < kDefaultWaitLimitNs) {}
            }
        }
    } else {
        // ======================= producer (one thread) =======================
        if (tid == kProdBase) {
            Cyc rs(p.stages);
            uint32_t issued = 0;
            bool alive = true;
            Walk wk(plan, p.count);
            while (alive && wk.next_entry()) {
                const unsigned char* wbase = p.e[wk.ei].w;
                for (uint32_t u = wk.u0; u < wk.u1; ++u, ++issued) {
                    if (!guard.wait_mbar(empty0 + 8 * rs.idx, rs.ph ^ 1)) {
                        alive = false;
                        break;
                    }
                    mbar_expect_tx(full0 + 8 * rs.idx, kUnitBytes);
                    bulk_g2s(smem_u32(ring + (size_t)rs.idx * kUnitBytes), wbase + (size_t)u * kUnitBytes, kUnitBytes,
                             full0 + 8 * rs.idx);
                    rs.step();
                }
            }
            // every copy issued must have landed before the CTA may retire (rs names the stage after the last one
            // issued; this wait also holds in an abandoned kernel)
            for (uint32_t back = 0; back < (uint32_t)p.stages && back < issued; ++back) {
                if (rs.idx == 0) { rs.idx = p.stages; rs.ph ^= 1; }
                --rs.idx;
                const unsigned long long t0 = Guard::now_ns();
                while (!mbar_try_wait(full0 + 8 * rs.idx, rs.ph) && Guard::now_ns() - t0 < kDefaultWaitLimitNs) {}
            }
        }
    }
    // nobody leaves before every copy has landed and every role is done; then tensor memory is released
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols));
}

// One thread per 32-bit word of the output: 2048 code words + 128 {scale, zero} words per unit.
__global__ void __launch_bounds__(256) pack_stream128_kernel(const uint8_t* __restrict__ codes,
                                                             const uint16_t* __restrict__ scales,
                                                             const uint16_t* __restrict__ zeros, int N, int K, int G,
                                                             uint32_t* __restrict__ out) {
    const int KB = K >> 7, ng = K / G, bpg = G >> 7;
    const int RT = (N + kUnitRows - 1) / kUnitRows;
    const long long total = (long long)RT * KB * (kUnitBytes / 4);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long unit = i / (kUnitBytes / 4);
        const int w = (int)(i % (kUnitBytes / 4));
        const int rt = (int)(unit / KB), kb = (int)(unit % KB);
        uint32_t word = 0;
        if (w < 2048) {
            const int j = w >> 9, r = (w >> 2) & 127, m = w & 3;  // chunk, row, word of the chunk
            const int n = rt * kUnitRows + r;
            if (n < N) {
                const uint2 cc = *reinterpret_cast<const uint2*>(codes + (size_t)n * K + (size_t)kb * 128 + j * 32 + m * 8);
                // byte b: column 8m+b in the low nibble, column 8m+4+b in the high nibble
                word = (cc.x & 0x0F0F0F0Fu) | ((cc.y & 0x0F0F0F0Fu) << 4);
            }
        } else {
            const int n = rt * kUnitRows + (w - 2048);
            if (n < N) {
                const size_t gi = (size_t)n * ng + kb / bpg;
                word = (uint32_t)scales[gi] | ((uint32_t)zeros[gi] << 16);
            }
        }
        out[i] = word;
    }
}


struct SmemPlan {
    int x_rows, xbuf_bytes, stages, xbufs;
    size_t total;
};

constexpr size_t kSmemLimit = 232448;  // 227 KiB per CTA

SmemPlan plan_for(int max_m, int nb_max, int xbufs) {
    SmemPlan pl;
    pl.x_rows = max_m <= 1 ? 1 : max_m <= 2 ? 2 : 4;
    pl.xbuf_bytes = nb_max * 4 * (32 + 48) * pl.x_rows + 512;  // (the last chunk's row window reaches past its own rows)
    const size_t fixed = (size_t)xbufs * pl.xbuf_bytes + (size_t)xbufs * 2 * pl.x_rows * nb_max * 4 +
                         (size_t)kHandDepth * 2 * pl.x_rows * kUnitRows * 4 + (size_t)(3 * kNB + 12 + kGroup + 2 * kHandDepth) * 8 + 16 +
                         16 * kNG + 128 + (size_t)kMaxEntries * 16;
    pl.xbufs = xbufs;
    pl.stages = 0;
    if (fixed < kSmemLimit) {
        long s = (long)((kSmemLimit - fixed) / (kUnitBytes + 16));
        if (s > 24) s = 24;
        s -= s % kNumWg;  // a ring stage is then always consumed by the same unpack warpgroup, which sees each of its phases
        pl.stages = (int)s;
        if (pl.stages <= kGroup) pl.stages = 0;  // (the issuers step through the ring by kGroup)
    }
    pl.total = fixed + (size_t)pl.stages * (kUnitBytes + 16);
    return pl;
}

// All CTAs of the kernel wait on each other (slots, dependency counter), so they must be resident together: the
// launch is cooperative, which the driver refuses when the grid does not fit the device as it is.
template <int kXR>
cudaError_t launch_one(const TcParams& p, int C, size_t smem, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(w4a16_tc_kernel<kXR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, w4a16_tc_kernel<kXR>, kThreads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorCooperativeLaunchTooLarge;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)C);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, w4a16_tc_kernel<kXR>, p);
}

std::atomic<unsigned long long> g_wait_ns{kDefaultWaitLimitNs};

}  // namespace

bool w4a16_tc_supported(int M, int N, int K, int G) {
    if (M < 1 || M > kMaxRows || N < 1 || K % 128 != 0 || G % 128 != 0) return false;
    // an activation buffer holds the 128-column blocks one CTA touches in this linear
    const uint32_t units = (uint32_t)((N + kUnitRows - 1) / kUnitRows) * (uint32_t)(K / 128);
    const uint32_t nb = std::min<uint32_t>((uint32_t)(K / 128), units / (uint32_t)num_sms() + 1u);
    if (units / (uint32_t)num_sms() >= 65535u || K / 128 >= 65536) return false;  // (16-bit fields of the slice table)
    return plan_for(M, (int)nb, 2).stages >= 4;
}

size_t w4a16_tc_weight_bytes(int N, int K) { return (size_t)((N + kUnitRows - 1) / kUnitRows) * (K / 128) * kUnitBytes; }

size_t w4a16_tc_workspace() { return (size_t)kWsHeader + (size_t)num_sms() * 2 * kSlotDepth * kSlotElems * 8; }

qil_status launch_pack_stream128_w4(const uint8_t* codes, const void* scales, const void* zeros, int N, int K, int G,
                                    void* out, cudaStream_t st) {
    const long long words = (long long)(w4a16_tc_weight_bytes(N, K) / 4);
    long long blocks = (words + 255) / 256;
    const long long cap = (long long)num_sms() * 16;
    if (blocks > cap) blocks = cap;
    pack_stream128_kernel<<<(int)blocks, 256, 0, st>>>(codes, reinterpret_cast<const uint16_t*>(scales),
                                                       reinterpret_cast<const uint16_t*>(zeros), N, K, G,
                                                       reinterpret_cast<uint32_t*>(out));
    return launch_status();
}

void w4a16_tc_set_wait_limit(unsigned long long ns) { g_wait_ns.store(ns ? ns : kDefaultWaitLimitNs); }

// Every entry must satisfy w4a16_tc_supported().  entries[i].flags: QIL_DEP_PREVIOUS, QIL_DEP_NEVER.
//
// How the units are dealt out.  A phase is a maximal run of entries of which only the first may carry
// QIL_DEP_PREVIOUS: its entries do not depend on each other, so their units form one stream that is cut into one
// contiguous, balanced slice per CTA.  A CTA then meets few entries per phase (on a list without dependencies: two or
// three in the whole launch), and the cost a CTA pays per entry it takes part in - activation conversion, row tiles
// shared with its neighbours - is paid rarely.  The price is an activation buffer that holds all K / 128 blocks of
// an entry; where that leaves too shallow a weight ring every entry is its own phase.
qil_status launch_w4a16_tc(const qil_linear_desc* entries, int count, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (ws == nullptr || ws_bytes < w4a16_tc_workspace()) return QIL_ERR_WORKSPACE;
    static TcParams p;  // 14 KiB: kept off the caller's stack; guarded by the mutex below
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    const uint32_t C = (uint32_t)num_sms();
    for (int first = 0; first < count; first += kMaxEntries) {
        const int n = count - first < kMaxEntries ? count - first : kMaxEntries;
        int max_m = 1;
        bool any_dep = false;
        uint32_t tiles = 0;
        uint32_t units[kMaxEntries];
        for (int i = 0; i < n; ++i) {
            const qil_linear_desc& d = entries[first + i];
            TcEntry& e = p.e[i];
            e.x = reinterpret_cast<const uint16_t*>(d.x);
            e.w = reinterpret_cast<const unsigned char*>(d.qweight);
            e.y = reinterpret_cast<__nv_bfloat16*>(d.y);
            e.N = d.N; e.K = d.K; e.M = d.M;
            e.flags = (i > 0) ? (d.flags & (kFlagDep | kFlagNever)) : 0;  // earlier launches are ordered by the stream
            if (e.flags & kFlagNever) e.flags |= kFlagDep;
            e.tiles_before = tiles;
            const uint32_t row_tiles = (uint32_t)((d.N + kUnitRows - 1) / kUnitRows);
            units[i] = row_tiles * (uint32_t)(d.K / 128);
            if (d.K / 128 >= 65536) return QIL_ERR_UNSUPPORTED;  // (16-bit fields of the slice table)
            tiles += row_tiles;
            any_dep |= (e.flags & kFlagDep) != 0;
            if (d.M > max_m) max_m = d.M;
        }
        // slices per phase (merged) or per entry; returns the blocks an activation buffer must hold, 0 if a field overflows
        auto deal = [&](bool merged) -> int {
            int nb_max = 1;
            for (int i = 0; i < n;) {
                int j = i + 1;
                while (merged && j < n && !(p.e[j].flags & kFlagDep)) ++j;
                uint64_t total = 0;
                for (int k = i; k < j; ++k) total += units[k];
                if (total > 0xFFFFFFFFull) return 0;
                const uint32_t q = (uint32_t)total / C, rem = (uint32_t)total % C;
                uint32_t base = 0;
                for (int k = i; k < j; ++k) {
                    p.e[k].q = q; p.e[k].rem = rem; p.e[k].base = base;
                    base += units[k];
                    const uint32_t most = std::min<uint32_t>(units[k], q + (rem ? 1u : 0u));  // units one CTA holds of the entry
                    if (most >= 65536u) return 0;
                    const int nb = (int)std::min<uint32_t>((uint32_t)(entries[first + k].K / 128), most);
                    if (nb > nb_max) nb_max = nb;
                }
                i = j;
            }
            return nb_max;
        };
        // as many activation buffers as leave a deep weight ring
        auto best_plan = [&](int nb_max) {
            SmemPlan pl = plan_for(max_m, nb_max, kMaxXBufs);
            for (int xb = kMaxXBufs - 1; xb >= 2 && pl.stages < 12; --xb) pl = plan_for(max_m, nb_max, xb);
            return pl;
        };
        int nb_max = deal(true);
        SmemPlan pl = nb_max > 0 ? best_plan(nb_max) : SmemPlan{};
        if (nb_max == 0 || pl.stages < 12) {
            nb_max = deal(false);
            if (nb_max == 0) return QIL_ERR_UNSUPPORTED;
            pl = best_plan(nb_max);
        }
        if (pl.stages < 4) return QIL_ERR_UNSUPPORTED;
        p.count = n;
        p.stages = pl.stages;
        p.nb_max = nb_max;
        p.xbufs = pl.xbufs;
        p.xbuf_bytes = pl.xbuf_bytes;
        p.wait_ns = g_wait_ns.load();
        p.status = reinterpret_cast<int*>(ws);
        p.tiles_done = any_dep ? reinterpret_cast<unsigned int*>(ws) + 1 : nullptr;
        p.slots = reinterpret_cast<unsigned char*>(ws) + kWsHeader;
        if (any_dep && cudaMemsetAsync(reinterpret_cast<unsigned int*>(ws) + 1, 0, 4, st) != cudaSuccess) {
            (void)cudaGetLastError();
            return QIL_ERR_CUDA;
        }
        const cudaError_t err = pl.x_rows == 1   ? launch_one<1>(p, (int)C, pl.total, st)
                                : pl.x_rows == 2 ? launch_one<2>(p, (int)C, pl.total, st)
                                                 : launch_one<4>(p, (int)C, pl.total, st);
        if (err != cudaSuccess) {
            (void)cudaGetLastError();
            return err == cudaErrorCooperativeLaunchTooLarge ? QIL_ERR_UNSUPPORTED : QIL_ERR_CUDA;
        }
    }
    return QIL_OK;
}

}  // namespace qil

