// Weight-only 4-bit decode linears on the 5th-generation tensor cores (tcgen05), as one
// persistent kernel over a list of linears (the memory-bound decode stage of the paper's
// OpenVLA deployment, Sec. 5.4 / App. A.4.2; M <= 4 activation rows).
//
// CUDA cores only unpack: a thread turns 64 bytes of packed codes (one weight row x 128
// columns) into int8 with three integer instructions per 8 weights and writes them to
// tensor memory (tcgen05.st), where they are the A operand (128 rows x 32 int8 per
// instruction) of tcgen05.mma kind::i8.  The B operand is the activation block, converted
// once per linear to 16-bit block fixed point - per 128 columns a power-of-two scale and
// two int8 planes (v = 256 hi + lo) - and laid out K-major in shared memory so that the
// 8 "columns" of the instruction are {row0 hi, row0 lo, row1 hi, ...}.  Accumulators are
// int32 in tensor memory (exact); per 128-column block the owner thread of a weight row
// reads them back (tcgen05.ld) and folds scale and zero point once:
//     y += s_w * 2^e * ((256 D_hi + D_lo) - z * X),   X = sum of the block's integers.
//
// Data layout (QIL_LAYOUT_STREAM128): unit u = (row tile of 128 rows, column block of 128)
// is 8704 bytes: 4 chunks (32 columns each) x 128 rows x 16 bytes of codes, byte b of
// word m of a chunk holding column 8m+b (low nibble) and 8m+4+b (high nibble); then
// 128 x {fp16 scale, fp16 zero}.  Rows beyond N are zero.  A linear is one contiguous
// stream of units.
//
// Roles in a CTA (one CTA per SM): a producer thread streams the CTA's slice of units
// through a shared-memory ring (cp.async.bulk + mbarrier); the unpack warpgroups alternate units
// (unpack -> tensor memory, later the epilogue of the same unit; three of them take turns); one thread per
// warpgroup issues its MMAs; four stager warps convert the next activations; four finalizer warps combine the
// warpgroups' partial sums, write outputs and complete row tiles shared with other CTAs
// through {value, tag} pairs in the workspace (one 8-byte store each, fixed summation order).
// Every wait is bounded (2 s); on expiry QIL_ERR_TIMEOUT is recorded in the workspace
// status word, waiting stops, tensor memory is released and the kernel returns.
#include <mutex>

#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kUnitRows = 128;
constexpr int kUnitBytes = 8192 + 512;
constexpr int kWgThreads = 128;
constexpr int kNumWg = 3;
constexpr int kStagerThreads = 128;
constexpr int kFinThreads = 128;
// thread ranges: kNumWg unpack/epilogue warpgroups, then the MMA warp, the producer warp, the stager, the finalizer
constexpr int kMmaBase = kNumWg * kWgThreads;
constexpr int kProdBase = kMmaBase + 32 * kNumWg;  // one MMA-issuing warp per warpgroup
constexpr int kStagerBase = kProdBase + 32;
constexpr int kFinBase = kStagerBase + kStagerThreads;
constexpr int kThreads = kFinBase + kFinThreads;
constexpr int kNumBuf = 3 * kNumWg;  // A buffers (32 columns each) and accumulator buffers (8 columns each)
constexpr int kTmemCols = 512;       // A at columns [0, 32 kNumBuf), D behind them
constexpr int kColD = 32 * kNumBuf;
static_assert(kColD + 8 * kNumBuf <= kTmemCols, "tensor memory budget");
constexpr int kMaxTiles = 2;    // row tiles per pass
constexpr int kPartBufs = 4;    // partial-sum buffers between the warpgroups and the finalizer
constexpr int kMaxEntries = 256;
constexpr int kMaxRows = 4;     // activation rows
constexpr int kSlotDepth = 4;                      // ring of slots per (CTA, first/last tile)
constexpr int kSlotElems = kMaxRows * kUnitRows;   // {value, tag} pairs of 8 bytes
constexpr int kWsHeader = 256;
constexpr int kFlagDep = 1;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct TcEntry {  // 48 bytes
    const uint16_t* x;
    const unsigned char* w;
    __nv_bfloat16* y;
    int N, K, M, flags;
    uint32_t tiles_before;
    uint32_t pad;
};

struct TcParams {
    TcEntry e[kMaxEntries];
    int count;
    int stages;
    int x_rows;     // activation rows staged: 1, 2 or 4 (>= every M)
    int kb_max;     // max K / 128
    int lbo;        // byte distance between 16-column chunks of the activation operand = 32 * x_rows
    int xbuf_bytes; // one activation buffer
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
template <int kId, int kCount>
__device__ __forceinline__ void group_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(kId), "n"(kCount) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// shared-memory operand descriptor: K-major, no swizzle, 8-row x 16-byte core matrices `lbo` bytes apart along K
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo) {
    uint64_t d = (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(128u >> 4) << 32;  // stride between 8-row groups: unused with 8 columns
    d |= (uint64_t)1 << 46;            // descriptor version of this architecture
    return d;
}
// D[128 x 8] (+)= A[128 x 32 u8, tensor memory] * B[8 x 32 s8, shared memory]^T, int32 accumulate
__device__ __forceinline__ void mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t accumulate) {
    // instruction descriptor: D = s32 (2 at bit 4), A = u8 (0 at bit 7), B = s8 (1 at bit 10), both K-major,
    // N >> 3 at bit 17, M >> 4 at bit 24
    constexpr uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | ((8u >> 3) << 17) | ((128u >> 4) << 24);
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// ---- bounded waits ----------------------------------------------------------------------------
struct Guard {
    int* status;
    volatile int* poisoned;
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
            if (mbar_try_wait(bar, parity)) return;
            if ((i & 15u) == 0 && (*poisoned || now_ns() - t0 > kWaitLimitNs)) break;
        }
        fail();
    }
    template <typename Pred>
    __device__ __forceinline__ void wait_flag(Pred done) const {
        if (done()) return;
        if (*poisoned) return;
        const unsigned long long t0 = now_ns();
        for (uint32_t i = 1;; ++i) {
            if (done()) return;
            __nanosleep(i < 64 ? 20 : 200);
            if ((i & 63u) == 0 && (*poisoned || now_ns() - t0 > kWaitLimitNs)) break;
        }
        fail();
    }
};

__device__ __forceinline__ void slice_of(uint32_t units, uint32_t c, uint32_t C, uint32_t& u0, uint32_t& u1) {
    u0 = (uint32_t)(((uint64_t)c * units) / C);
    u1 = (uint32_t)(((uint64_t)(c + 1) * units) / C);
}
__device__ __forceinline__ uint32_t owner_of(uint32_t u, uint32_t units, uint32_t C) {
    return (uint32_t)((((uint64_t)(u + 1)) * C - 1) / units);
}
__device__ __forceinline__ bool contributor_slot(uint32_t cc, uint32_t rt, uint32_t units, uint32_t KB, uint32_t C,
                                                 uint32_t& which) {
    uint32_t cu0, cu1;
    slice_of(units, cc, C, cu0, cu1);
    which = (cu0 / KB == rt) ? 0u : 1u;
    return cu0 != cu1;
}

// The work of one CTA: entries in which it owns units, cut into passes of at most kMaxTiles row tiles.
struct Walk {
    const TcParams& p;
    uint32_t C, c;
    int ei;
    uint32_t KB, units, u0, u1, t_first, t_last;
    __device__ Walk(const TcParams& p_, uint32_t C_, uint32_t c_) : p(p_), C(C_), c(c_), ei(-1) {}
    __device__ bool next_entry() {
        for (++ei; ei < p.count; ++ei) {
            KB = (uint32_t)p.e[ei].K >> 7;
            units = (((uint32_t)p.e[ei].N + kUnitRows - 1) / kUnitRows) * KB;
            slice_of(units, c, C, u0, u1);
            if (u0 != u1) {
                t_first = u0 / KB;
                t_last = (u1 - 1) / KB;
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

__global__ void __launch_bounds__(kThreads, 1) w4a16_tc_kernel(const __grid_constant__ TcParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x;
    const uint32_t C = gridDim.x, c = blockIdx.x;
    const int XR = p.x_rows;

    // ---- carve shared memory ----
    unsigned char* ring = smem;                                                          // [stages][kUnitBytes]
    unsigned char* xs = ring + (size_t)p.stages * kUnitBytes;                            // [2][xbuf_bytes]
    unsigned char* xraw = xs + (size_t)2 * p.xbuf_bytes;                                 // [XR][kb_max*256] bf16
    int* xsum = reinterpret_cast<int*>(xraw + (size_t)XR * p.kb_max * 256);              // [2][XR][kb_max]
    float* xscale = reinterpret_cast<float*>(xsum + 2 * XR * p.kb_max);                  // [2][XR][kb_max]
    float* part = xscale + 2 * XR * p.kb_max;                       // [kPartBufs][kNumWg][kMaxTiles][XR][128]
    const int part_floats = kNumWg * kMaxTiles * XR * kUnitRows;
    uint64_t* bars = reinterpret_cast<uint64_t*>(part + (size_t)kPartBufs * part_floats);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + p.stages);
    uint64_t* b2 = bars + 2 * p.stages;
    const uint32_t afull0 = smem_u32(b2);
    const uint32_t dfull0 = smem_u32(b2 + 2 * kNumBuf), dempty0 = smem_u32(b2 + 3 * kNumBuf);
    uint64_t* b3 = b2 + 4 * kNumBuf;
    const uint32_t xfull0 = smem_u32(b3), xempty0 = smem_u32(b3 + 2), xraw0 = smem_u32(b3 + 4);
    const uint32_t pfull0 = smem_u32(b3 + 5), pempty0 = smem_u32(b3 + 5 + kPartBufs);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(b3 + 5 + 2 * kPartBufs);
    volatile int* poisoned = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 4);
        }
        for (int i = 0; i < kNumBuf; ++i) {
            mbar_init(afull0 + 8 * i, 4);
            mbar_init(dfull0 + 8 * i, 1);
            mbar_init(dempty0 + 8 * i, 4);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(xfull0 + 8 * i, 1);
            mbar_init(xempty0 + 8 * i, kNumWg * 4);
        }
        mbar_init(xraw0, 1);
        for (int i = 0; i < kPartBufs; ++i) {
            mbar_init(pfull0 + 8 * i, kNumWg * 4);
            mbar_init(pempty0 + 8 * i, 1);
        }
        *poisoned = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < kPartBufs * part_floats; i += kThreads) part[i] = 0.f;
    for (int i = tid; i < 2 * p.xbuf_bytes / 4; i += kThreads) reinterpret_cast<uint32_t*>(xs)[i] = 0u;
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
    const Guard guard{p.status, poisoned};

    if (tid < kMmaBase) {
        // ======================= unpack + epilogue warpgroups =======================
        const int wg = tid / kWgThreads, r = tid % kWgThreads, lane = tid & 31;
        const uint32_t lane_base = (uint32_t)(r & ~31) << 16;  // this warp's quarter of the tensor-memory lanes
        Cyc rs(p.stages), pb(kPartBufs), ab(kNumBuf), turn(kNumWg);  // all advance once per unit of the CTA
        uint32_t xe = 0;
        Walk wk(p, C, c);
        while (wk.next_entry()) {
            const int M = p.e[wk.ei].M;
            const uint32_t KB = wk.KB;
            const uint32_t xb = xe & 1;
            guard.wait_mbar(xfull0 + 8 * xb, (xe >> 1) & 1);
            ++xe;
            const int* xsum_b = xsum + (size_t)xb * XR * p.kb_max;
            const float* xscale_b = xscale + (size_t)xb * XR * p.kb_max;
            for (uint32_t tp = wk.t_first; tp <= wk.t_last; tp += kMaxTiles) {
                const uint32_t pu0 = max(wk.u0, tp * KB), pu1 = min(wk.u1, (tp + kMaxTiles) * KB);
                guard.wait_mbar(pempty0 + 8 * pb.idx, pb.ph ^ 1);
                float* my_part = part + (size_t)pb.idx * part_floats + (size_t)wg * kMaxTiles * XR * kUnitRows + r;
                float fin[kMaxRows] = {0.f, 0.f, 0.f, 0.f};
                int cur_tile = -1;
                // units whose MMAs are in flight: the accumulators of a unit are read after the next two units of
                // this warpgroup have been written to tensor memory (the oldest record is pend_*, the newer next_*)
                int npend = 0;
                uint32_t pend_d = 0, pend_dph = 0, pend_kb = 0, next_d = 0, next_dph = 0, next_kb = 0;
                int pend_tl = 0, next_tl = 0;
                float pend_s = 0.f, next_s = 0.f;
                int pend_z = 0, next_z = 0;
                uint32_t d[8];
                auto epilogue_load = [&]() {   // start reading the accumulators of the pending unit
                    guard.wait_mbar(dfull0 + 8 * pend_d, pend_dph);
                    tc_fence_after();
                    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]),
                                   "=r"(d[7])
                                 : "r"(tmem + lane_base + kColD + 8 * pend_d));
                };
                auto epilogue_math = [&]() {   // ... and fold them into this thread's row sums
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(dempty0 + 8 * pend_d);
                    if (pend_tl != cur_tile) {
                        if (cur_tile >= 0) {
#pragma unroll
                            for (int t = 0; t < kMaxRows; ++t)
                                if (t < XR) my_part[((size_t)cur_tile * XR + t) * kUnitRows] = fin[t];
                        }
                        fin[0] = fin[1] = fin[2] = fin[3] = 0.f;
                        cur_tile = pend_tl;
                    }
#pragma unroll
                    for (int t = 0; t < kMaxRows; ++t)
                        if (t < M) {
                            const int acc = (int)d[2 * t] * 256 + (int)d[2 * t + 1];
                            const int v = acc - pend_z * xsum_b[t * p.kb_max + pend_kb];
                            fin[t] = fmaf((float)v, pend_s * xscale_b[t * p.kb_max + pend_kb], fin[t]);
                        }
                };
                uint32_t tl = pu0 / KB - tp, kb = pu0 % KB;
                for (uint32_t cu = pu0; cu < pu1; ++cu) {
                    if (turn.idx == (uint32_t)wg) {
                        const uint32_t a = ab.idx;
                        guard.wait_mbar(full0 + 8 * rs.idx, rs.ph);
                        const unsigned char* ub = ring + (size_t)rs.idx * kUnitBytes;
                        tc_fence_after();
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 w = *reinterpret_cast<const uint4*>(ub + ((size_t)j * kUnitRows + r) * 16);
                            const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
                            uint32_t q[8];
#pragma unroll
                            for (int m = 0; m < 4; ++m) {
                                q[2 * m] = ws[m] & 0x0F0F0F0Fu;
                                q[2 * m + 1] = (ws[m] >> 4) & 0x0F0F0F0Fu;
                            }
                            asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(
                                             tmem + lane_base + 32 * a + 8 * j),
                                         "r"(q[0]), "r"(q[1]), "r"(q[2]), "r"(q[3]), "r"(q[4]), "r"(q[5]), "r"(q[6]), "r"(q[7])
                                         : "memory");
                        }
                        const __half2 meta = *reinterpret_cast<const __half2*>(ub + 8192 + 4 * r);
                        const bool drain = npend == 2;
                        if (drain) epilogue_load();  // overlaps with the stores above
                        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            mbar_arrive(afull0 + 8 * a);
                            mbar_arrive(empty0 + 8 * rs.idx);
                        }
                        if (drain) {
                            epilogue_math();
                            pend_d = next_d; pend_dph = next_dph; pend_kb = next_kb; pend_tl = next_tl;
                            pend_s = next_s; pend_z = next_z;
                            npend = 1;
                        }
                        if (npend == 0) {
                            pend_d = a; pend_dph = ab.ph; pend_kb = kb; pend_tl = (int)tl;
                            pend_s = __low2float(meta); pend_z = (int)__high2float(meta);
                        } else {
                            next_d = a; next_dph = ab.ph; next_kb = kb; next_tl = (int)tl;
                            next_s = __low2float(meta); next_z = (int)__high2float(meta);
                        }
                        ++npend;
                    }
                    rs.step();
                    ab.step();
                    turn.step();
                    if (++kb == KB) { kb = 0; ++tl; }
                }
                while (npend > 0) {
                    epilogue_load();
                    epilogue_math();
                    pend_d = next_d; pend_dph = next_dph; pend_kb = next_kb; pend_tl = next_tl;
                    pend_s = next_s; pend_z = next_z;
                    --npend;
                }
                if (cur_tile >= 0) {
#pragma unroll
                    for (int t = 0; t < kMaxRows; ++t)
                        if (t < XR) my_part[((size_t)cur_tile * XR + t) * kUnitRows] = fin[t];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(pfull0 + 8 * pb.idx);
                pb.step();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(xempty0 + 8 * xb);
        }
    } else if (tid < kProdBase) {
        // ======================= MMA issuers (one thread per warpgroup) =======================
        if (((tid - kMmaBase) & 31) == 0) {
            const uint32_t g = (uint32_t)(tid - kMmaBase) >> 5;  // serves the units of warpgroup g
            uint32_t xe = 0;
            Cyc ab(kNumBuf), turn(kNumWg);
            Walk wk(p, C, c);
            const uint64_t desc_hi = smem_desc(0, p.lbo);
            while (wk.next_entry()) {
                const uint32_t KB = wk.KB;
                const uint32_t xb = xe & 1;
                guard.wait_mbar(xfull0 + 8 * xb, (xe >> 1) & 1);
                ++xe;
                const uint32_t xs16 = smem_u32(xs + (size_t)xb * p.xbuf_bytes) >> 4, lbo16 = (uint32_t)p.lbo >> 4;
                uint32_t kb = wk.u0 % KB;
                for (uint32_t cu = wk.u0; cu < wk.u1; ++cu) {
                    if (turn.idx == g) {
                        const uint32_t a = ab.idx;
                        guard.wait_mbar(afull0 + 8 * a, ab.ph);
                        guard.wait_mbar(dempty0 + 8 * a, ab.ph ^ 1);
                        tc_fence_after();
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            mma_i8_ts(tmem + kColD + 8 * a, tmem + 32 * a + 8 * j,
                                      desc_hi | (uint64_t)(xs16 + (kb * 8 + 2 * j) * lbo16), j > 0 ? 1u : 0u);
                        // accumulators complete -> epilogue; it also means the A buffer has been read, and the same
                        // warpgroup reuses it only after that epilogue
                        tc_commit(dfull0 + 8 * a);
                    }
                    ab.step();
                    turn.step();
                    if (++kb == KB) kb = 0;
                }
            }
        }
    } else if (tid < kStagerBase) {
        // ======================= producer (one thread) =======================
        if (tid == kProdBase) {
            Cyc rs(p.stages);
            uint32_t issued = 0;
            Walk wk(p, C, c);
            while (wk.next_entry()) {
                const unsigned char* wbase = p.e[wk.ei].w;
                for (uint32_t cu = wk.u0; cu < wk.u1; ++cu, ++issued) {
                    guard.wait_mbar(empty0 + 8 * rs.idx, rs.ph ^ 1);
                    mbar_expect_tx(full0 + 8 * rs.idx, kUnitBytes);
                    bulk_g2s_plain(smem_u32(ring + (size_t)rs.idx * kUnitBytes), wbase + (size_t)cu * kUnitBytes, kUnitBytes,
                                   full0 + 8 * rs.idx);
                    rs.step();
                }
            }
            // every copy issued must have landed before the CTA may retire
            for (uint32_t back = 0; back < (uint32_t)p.stages && back < issued; ++back) {
                if (rs.idx == 0) { rs.idx = p.stages; rs.ph ^= 1; }
                --rs.idx;
                guard.wait_mbar(full0 + 8 * rs.idx, rs.ph);
            }
        }
    } else if (tid < kFinBase) {
        // ======================= activation stager (4 warps) =======================
        // bf16 row -> per 128 columns: e with max|x| / 2^e <= 32639, v = rint(x / 2^e) = 256 hi + lo (both int8),
        // X = sum v.  hi / lo planes go to rows 2t / 2t+1 of every 16-column chunk of the operand.
        const int st = tid - kStagerBase;
        uint32_t xe = 0;
        Walk wk(p, C, c);
        while (wk.next_entry()) {
            const TcEntry& E = p.e[wk.ei];
            const uint32_t KB = wk.KB;
            const uint32_t xb = xe & 1;
            unsigned char* xs_b = xs + (size_t)xb * p.xbuf_bytes;
            int* xsum_b = xsum + (size_t)xb * XR * p.kb_max;
            float* xscale_b = xscale + (size_t)xb * XR * p.kb_max;
            if (st == 0) {
                guard.wait_mbar(xempty0 + 8 * xb, ((xe >> 1) & 1) ^ 1);
                if (E.flags & kFlagDep) {
                    const unsigned int need = E.tiles_before;
                    guard.wait_flag([&] { return ld_acquire(p.tiles_done) >= need; });
                    asm volatile("fence.proxy.async;" ::: "memory");
                }
                mbar_expect_tx(xraw0, (uint32_t)E.M * (uint32_t)E.K * 2u);
                for (int t = 0; t < E.M; ++t)
                    bulk_g2s_plain(smem_u32(xraw + (size_t)t * p.kb_max * 256), E.x + (size_t)t * E.K, (uint32_t)E.K * 2u, xraw0);
            }
            guard.wait_mbar(xraw0, xe & 1);
            // Two passes over the row, 8 columns (one 16-byte piece) per thread and step, no cross-thread
            // shuffles: pass 1 leaves max|x| of every 128-column block in shared memory (atomicMax on the bit
            // patterns), pass 2 converts with the block's scale and adds up the integers (atomicAdd).
            const int pieces = (int)KB * 16;  // 16-byte pieces per row
            for (int t = 0; t < E.M; ++t) {
                unsigned int* bmax = reinterpret_cast<unsigned int*>(xscale_b + t * p.kb_max);  // reused as scratch
                for (int kb = st; kb < (int)KB; kb += kStagerThreads) {
                    bmax[kb] = 0u;
                    xsum_b[t * p.kb_max + kb] = 0;
                }
            }
            group_sync<1, kStagerThreads>();
            for (int t = 0; t < E.M; ++t) {
                const unsigned char* xrow = xraw + (size_t)t * p.kb_max * 256;
                unsigned int* bmax = reinterpret_cast<unsigned int*>(xscale_b + t * p.kb_max);
#pragma unroll 4
                for (int pc = st; pc < pieces; pc += kStagerThreads) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(xrow + (size_t)pc * 16);
                    const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
                    uint32_t amax = 0;  // bf16 magnitudes order like unsigned integers
#pragma unroll
                    for (int i = 0; i < 4; ++i) amax = max(amax, max((u[i] << 16) & 0x7FFFFFFFu, u[i] & 0x7FFF0000u));
                    atomicMax(bmax + (pc >> 4), amax);
                }
            }
            group_sync<1, kStagerThreads>();
            for (int t = 0; t < E.M; ++t) {
                const unsigned char* xrow = xraw + (size_t)t * p.kb_max * 256;
                const unsigned int* bmax = reinterpret_cast<const unsigned int*>(xscale_b + t * p.kb_max);
                unsigned char* xdst = xs_b + (size_t)(2 * t) * 16;
#pragma unroll 4
                for (int pc = st; pc < pieces; pc += kStagerThreads) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(xrow + (size_t)pc * 16);
                    const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
                    const uint32_t amax = bmax[pc >> 4];
                    // 2^e = smallest power of two with max|x| / 2^e <= 32639: exponent field E -> e = E - 127 - 14, one
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
                    // piece pc = 8 columns: 16-column chunk pc/2, first or second half of its 16-byte row
                    unsigned char* dst = xdst + (size_t)(pc >> 1) * p.lbo + (pc & 1) * 8;
                    *reinterpret_cast<uint2*>(dst) = hi;
                    *reinterpret_cast<uint2*>(dst + 16) = lo;
                    atomicAdd(xsum_b + t * p.kb_max + (pc >> 4), sum);
                }
            }
            group_sync<1, kStagerThreads>();
            for (int t = 0; t < E.M; ++t)  // replace the block maxima by the scales 2^e
                for (int kb = st; kb < (int)KB; kb += kStagerThreads) {
                    const uint32_t amax = reinterpret_cast<const unsigned int*>(xscale_b + t * p.kb_max)[kb];
                    int ef = (int)(amax >> 23);
                    if (ef < 1 || ef >= 255) ef = 127 + 14;
                    int e = ef - 127 - 14 + (((amax & 0x7FFFFFu) > 0x7EFE00u) ? 1 : 0);
                    if (e < -126) e = -126;
                    xscale_b[t * p.kb_max + kb] = __uint_as_float((uint32_t)(127 + e) << 23);
                }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMAs read xs through the async proxy
            group_sync<1, kStagerThreads>();
            if (st == 0) mbar_arrive(xfull0 + 8 * xb);
            ++xe;
        }
    } else {
        // ======================= finalizer (4 warps; thread = row of the tile) =======================
        // Row tiles shared with other CTAs are completed through the workspace: each contributor writes
        // {value, tag} pairs (one 8-byte store per element, tag = entry index + 1) into a ring of kSlotDepth
        // slots; the CTA owning the end of the tile polls the pairs, adds them in CTA order and clears the tags.
        const int r = tid - kFinBase;
        Cyc pb(kPartBufs);
        Walk wk(p, C, c);
        while (wk.next_entry()) {
            const TcEntry& E = p.e[wk.ei];
            const int M = E.M, N = E.N;
            const uint32_t KB = wk.KB, u0 = wk.u0, u1 = wk.u1, units = wk.units;
            const uint32_t tag = (uint32_t)wk.ei + 1u, ring_i = (uint32_t)wk.ei % kSlotDepth;
            // slice geometry: is the last tile cut at its end (this CTA contributes), the first at its beginning
            // (this CTA completes it)?
            const bool have_last = (wk.t_last + 1) * KB > u1;
            const bool have_first = wk.t_first * KB < u0 && (wk.t_first + 1) * KB <= u1;
            unsigned long long* my_slot = nullptr;
            if (have_last) {
                const uint32_t which = (wk.t_last == wk.t_first) ? 0u : 1u;
                my_slot = reinterpret_cast<unsigned long long*>(p.slots) +
                          (((size_t)c * 2 + which) * kSlotDepth + ring_i) * kSlotElems;
                // the slot must have been consumed (tags cleared) by whoever completed the tile it last served;
                // checked now, while the warpgroups are still computing
#pragma unroll
                for (int t = 0; t < kMaxRows; ++t)
                    if (t < M) {
                        const unsigned long long* q = my_slot + t * kUnitRows + r;
                        guard.wait_flag([&] { return (uint32_t)(__ldcg(q) >> 32) == 0u; });
                    }
            }
            uint32_t n_full = 0;
            float first_v[kMaxRows] = {0.f, 0.f, 0.f, 0.f};
            for (uint32_t tp = wk.t_first; tp <= wk.t_last; tp += kMaxTiles) {
                const uint32_t ntiles = min((uint32_t)kMaxTiles, wk.t_last - tp + 1);
                guard.wait_mbar(pfull0 + 8 * pb.idx, pb.ph);
                float* buf = part + (size_t)pb.idx * part_floats;
                for (uint32_t tl = 0; tl < ntiles; ++tl) {
                    const uint32_t rt = tp + tl;
                    const bool cb = u0 <= rt * KB, ce = (rt + 1) * KB <= u1;
                    float v[kMaxRows];
#pragma unroll
                    for (int t = 0; t < kMaxRows; ++t) {
                        v[t] = 0.f;
                        if (t < XR) {
#pragma unroll
                            for (int g = 0; g < kNumWg; ++g) {  // fixed order
                                float* a = buf + ((size_t)(g * kMaxTiles + tl) * XR + t) * kUnitRows + r;
                                v[t] += *a;
                                *a = 0.f;
                            }
                        }
                    }
                    const int row = (int)rt * kUnitRows + r;
                    if (cb && ce) {
                        ++n_full;
                        if (row < N) {
#pragma unroll
                            for (int t = 0; t < kMaxRows; ++t)
                                if (t < M) E.y[(size_t)t * N + row] = __float2bfloat16_rn(v[t]);
                        }
                    } else if (ce) {
#pragma unroll
                        for (int t = 0; t < kMaxRows; ++t) first_v[t] = v[t];
                    } else {  // publish this CTA's share: value and tag travel in one store
#pragma unroll
                        for (int t = 0; t < kMaxRows; ++t)
                            if (t < M)
                                __stcg(my_slot + t * kUnitRows + r,
                                       ((unsigned long long)tag << 32) | (unsigned long long)__float_as_uint(v[t]));
                    }
                }
                group_sync<2, kFinThreads>();
                if (r == 0) mbar_arrive(pempty0 + 8 * pb.idx);
                pb.step();
            }
            if (have_first) {  // complete the tile whose beginning belongs to earlier CTAs
                const uint32_t rt = wk.t_first;
                const uint32_t c_lo = owner_of(rt * KB, units, C);
                float sum[kMaxRows] = {0.f, 0.f, 0.f, 0.f};
                for (uint32_t cc = c_lo; cc < c; ++cc) {
                    uint32_t which;
                    if (!contributor_slot(cc, rt, units, KB, C, which)) continue;
                    unsigned long long* src = reinterpret_cast<unsigned long long*>(p.slots) +
                                              (((size_t)cc * 2 + which) * kSlotDepth + ring_i) * kSlotElems + r;
                    unsigned long long got[kMaxRows] = {0ull, 0ull, 0ull, 0ull};
                    guard.wait_flag([&] {
                        bool all = true;
#pragma unroll
                        for (int t = 0; t < kMaxRows; ++t)
                            if (t < M) {
                                got[t] = __ldcg(src + t * kUnitRows);
                                all &= (uint32_t)(got[t] >> 32) == tag;
                            }
                        return all;
                    });
#pragma unroll
                    for (int t = 0; t < kMaxRows; ++t)
                        if (t < M) {
                            sum[t] += __uint_as_float((uint32_t)got[t]);
                            __stcg(src + t * kUnitRows, 0ull);  // consumed: the slot may be reused
                        }
                }
                const int row = (int)rt * kUnitRows + r;
                if (row < N) {
#pragma unroll
                    for (int t = 0; t < kMaxRows; ++t)
                        if (t < M) E.y[(size_t)t * N + row] = __float2bfloat16_rn(sum[t] + first_v[t]);
                }
                ++n_full;
            }
            if (n_full && p.tiles_done) {
                group_sync<2, kFinThreads>();  // every row of the tiles is written
                if (r == 0) {
                    __threadfence();
                    red_release_add(p.tiles_done, n_full);
                }
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
    int x_rows, lbo, xbuf_bytes, stages;
    size_t total;
};

constexpr size_t kSmemLimit = 232448;  // 227 KiB per CTA

SmemPlan plan_for(int max_m, int kb_max) {
    SmemPlan pl;
    pl.x_rows = max_m <= 1 ? 1 : max_m <= 2 ? 2 : 4;
    pl.lbo = 32 * pl.x_rows;
    pl.xbuf_bytes = kb_max * 8 * pl.lbo + 128;  // the last chunk's 8-row window reaches past its own rows
    const size_t fixed = (size_t)2 * pl.xbuf_bytes + (size_t)pl.x_rows * kb_max * 256 + (size_t)2 * 2 * pl.x_rows * kb_max * 4 +
                         (size_t)kPartBufs * kNumWg * kMaxTiles * pl.x_rows * kUnitRows * 4 +
                         (size_t)(4 * kNumBuf + 5 + 2 * kPartBufs) * 8 + 16 + 128;
    pl.stages = 0;
    if (fixed < kSmemLimit) {
        long s = (long)((kSmemLimit - fixed) / (kUnitBytes + 16));
        if (s > 20) s = 20;
        pl.stages = (int)s;
    }
    pl.total = fixed + (size_t)pl.stages * (kUnitBytes + 16);
    return pl;
}

}  // namespace

bool w4a16_tc_supported(int M, int N, int K, int G) {
    if (M < 1 || M > kMaxRows || N < 1 || K % 128 != 0 || G % 128 != 0) return false;
    return plan_for(M, K / 128).stages >= 4;
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

// Every entry must satisfy w4a16_tc_supported().  entries[i].flags bit 0 = QIL_DEP_PREVIOUS.
qil_status launch_w4a16_tc(const qil_linear_desc* entries, int count, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (ws == nullptr || ws_bytes < w4a16_tc_workspace()) return QIL_ERR_WORKSPACE;
    static TcParams p;  // 12 KiB: kept off the caller's stack; guarded by the mutex below
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    const int C = num_sms();
    for (int base = 0; base < count; base += kMaxEntries) {
        const int n = count - base < kMaxEntries ? count - base : kMaxEntries;
        int max_m = 1, kmax = 128;
        bool any_dep = false;
        uint32_t tiles = 0;
        for (int i = 0; i < n; ++i) {
            const qil_linear_desc& d = entries[base + i];
            TcEntry& e = p.e[i];
            e.x = reinterpret_cast<const uint16_t*>(d.x);
            e.w = reinterpret_cast<const unsigned char*>(d.qweight);
            e.y = reinterpret_cast<__nv_bfloat16*>(d.y);
            e.N = d.N; e.K = d.K; e.M = d.M;
            e.flags = (i > 0) ? (d.flags & kFlagDep) : 0;  // earlier launches are ordered by the stream
            e.tiles_before = tiles;
            e.pad = 0;
            tiles += (uint32_t)((d.N + kUnitRows - 1) / kUnitRows);
            any_dep |= (e.flags & kFlagDep) != 0;
            if (d.M > max_m) max_m = d.M;
            if (d.K > kmax) kmax = d.K;
        }
        const SmemPlan pl = plan_for(max_m, kmax / 128);
        if (pl.stages < 4) return QIL_ERR_UNSUPPORTED;
        p.count = n;
        p.stages = pl.stages;
        p.x_rows = pl.x_rows;
        p.kb_max = kmax / 128;
        p.lbo = pl.lbo;
        p.xbuf_bytes = pl.xbuf_bytes;
        p.status = reinterpret_cast<int*>(ws);
        p.tiles_done = any_dep ? reinterpret_cast<unsigned int*>(ws) + 1 : nullptr;
        p.slots = reinterpret_cast<unsigned char*>(ws) + kWsHeader;
        if (any_dep && cudaMemsetAsync(reinterpret_cast<unsigned int*>(ws) + 1, 0, 4, st) != cudaSuccess) {
            (void)cudaGetLastError();
            return QIL_ERR_CUDA;
        }
        if (cudaFuncSetAttribute(w4a16_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.total) != cudaSuccess) {
            (void)cudaGetLastError();
            return QIL_ERR_CUDA;
        }
        w4a16_tc_kernel<<<C, kThreads, pl.total, st>>>(p);
        const qil_status s = launch_status();
        if (s != QIL_OK) return s;
    }
    return QIL_OK;
}

}  // namespace qil
