// Weight-only 4-bit decode linears as ONE persistent kernel over a list of linears
// (the memory-bound decode stage of the paper's OpenVLA deployment, Sec. 5.4 /
// App. A.4.2: q, k, v, o, gate, up, down of every decoder layer, M <= 8 rows).
//
// Data layout (QIL_LAYOUT_STREAM): the weight matrix is a sequence of self-contained
// 1088-byte units, unit u = (row tile rt = u / (K/128), column block kb = u % (K/128)):
// 1024 bytes of packed codes of 16 output features x 128 input features (16 rows of 64
// bytes) followed by 16 x {fp16 scale, fp16 zero} of those rows for that block.  A
// linear is therefore one contiguous byte stream, and any slice of units is too.
//
// Execution: one CTA per SM, alive for the whole list.  For every linear each CTA
// owns a contiguous slice of its units (balanced to +-1 unit).  A producer thread
// streams the slice through a shared-memory ring with bulk asynchronous copies
// (cp.async.bulk + mbarrier transaction counts), running ahead across linears as far
// as the ring allows, so HBM stays busy while the consumers finish a linear.
// Sixteen consumer warps each take one unit per ring stage: nibbles -> bf16 (128+q)
// by mask/or, mma.sync m16n8k16 against the activation rows staged in shared memory,
// scale/zero folded once per unit (y += s*(acc - (128+z)*X), X = block sum of x).
// Row tiles cut by a slice boundary are completed through small fp32 slots in the
// workspace: every CTA first publishes its contribution to the tile it shares with
// the next CTA, then completes the tile it shares with previous CTAs, adding the
// contributions in CTA order - so results do not depend on timing.  A slot's flag
// carries the index of the entry it was filled for (0 = free), because the CTA that
// completes a tile differs from entry to entry.  An entry flagged
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

constexpr int kConsumerWarps = 16;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;  // + one producer warp
constexpr int kUnitBytes = 1088;
constexpr int kStageUnits = kConsumerWarps;
constexpr int kStageBytes = kStageUnits * kUnitBytes;
constexpr int kMaxTiles = 8;    // row tiles handled per pass
constexpr int kElems = 128;     // fp32 values of one row tile: 16 rows x 8 activation rows
constexpr int kMaxEntries = 256;
constexpr int kSlotBytes = kElems * 4 + 16;  // data + flag word (padded)
constexpr int kWsHeader = 256;
constexpr int kRowPad = 16;
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
    int x_row_bytes;  // max K * 2 + pad
    int kb_max;       // max K / 128
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
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const unsigned int* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(unsigned int* p, uint32_t v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(unsigned int* p, uint32_t v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t nib_pair(uint32_t w, int i) {
    return ((w >> (4 * i)) & 0x000F000Fu) | 0x43004300u;  // bf16x2 {128 + nibble i, 128 + nibble i+4}
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
        if (*poisoned) return;
        if (mbar_try_wait(bar, parity)) return;
        const unsigned long long t0 = now_ns();
        for (uint32_t i = 1;; ++i) {
            if (mbar_try_wait(bar, parity)) return;
            if ((i & 63u) == 0 && (*poisoned || now_ns() - t0 > kWaitLimitNs)) break;
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

__global__ void __launch_bounds__(kThreads, 1) w4a16_stream_kernel(const __grid_constant__ StreamParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x;
    const uint32_t C = gridDim.x, c = blockIdx.x;

    // ---- carve shared memory ----
    unsigned char* ring = smem;
    float* tile_part = reinterpret_cast<float*>(ring + (size_t)p.stages * kStageBytes);  // [kMaxTiles][16 warps][128]
    float* stash_first = tile_part + kMaxTiles * kConsumerWarps * kElems;                // [128]
    float* stash_last = stash_first + kElems;                                            // [128]
    unsigned char* xs = reinterpret_cast<unsigned char*>(stash_last + kElems);           // [x_rows][x_row_bytes]
    float* xsum = reinterpret_cast<float*>(xs + (size_t)p.x_rows * p.x_row_bytes);       // [8][kb_max]
    uint64_t* bars = reinterpret_cast<uint64_t*>(xsum + 8 * p.kb_max);                   // full[S], empty[S]
    volatile int* poisoned = reinterpret_cast<volatile int*>(bars + 2 * p.stages);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + p.stages);

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kConsumerWarps);
        }
        *poisoned = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const Guard guard{p.status, poisoned};

    if (tid >= kConsumerThreads) {
        // =============================== producer ===============================
        if (tid == kConsumerThreads) {
            uint64_t policy;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
            uint32_t ctr = 0;
            for (int ei = 0; ei < p.count; ++ei) {
                const StreamEntry& E = p.e[ei];
                const uint32_t KB = E.K >> 7, units = (uint32_t)(E.N >> 4) * KB;
                uint32_t u0, u1;
                slice_of(units, c, C, u0, u1);
                if (u0 == u1) continue;
                const uint32_t t_first = u0 / KB, t_last = (u1 - 1) / KB;
                for (uint32_t tp = t_first; tp <= t_last; tp += kMaxTiles) {
                    const uint32_t pu0 = max(u0, tp * KB), pu1 = min(u1, (tp + kMaxTiles) * KB);
                    for (uint32_t cu = pu0; cu < pu1; cu += kStageUnits, ++ctr) {
                        const uint32_t n = min((uint32_t)kStageUnits, pu1 - cu);
                        const uint32_t s = ctr % p.stages, round = ctr / p.stages;
                        guard.wait_mbar(empty0 + 8 * s, (round & 1) ^ 1);
                        mbar_expect_tx(full0 + 8 * s, n * kUnitBytes);
                        bulk_g2s(smem_u32(ring + (size_t)s * kStageBytes), E.w + (size_t)cu * kUnitBytes, n * kUnitBytes,
                                 full0 + 8 * s, policy);
                    }
                }
            }
            // every copy this thread issued must have landed before the CTA may retire
            const uint32_t issued = ctr;
            for (uint32_t back = 0; back < (uint32_t)p.stages && back < issued; ++back) {
                const uint32_t k = issued - 1 - back;
                guard.wait_mbar(full0 + 8 * (k % p.stages), (k / p.stages) & 1);
            }
        }
    } else {
        // =============================== consumers ===============================
        const int lane = tid & 31, warp = tid >> 5;
        const int g = lane >> 2, t = lane & 3;
        uint32_t ctr = 0;
        for (int ei = 0; ei < p.count; ++ei) {
            const StreamEntry& E = p.e[ei];
            const uint32_t KB = E.K >> 7, RT = E.N >> 4, units = RT * KB;
            const int M = E.M, N = E.N;
            uint32_t u0, u1;
            slice_of(units, c, C, u0, u1);
            if (u0 == u1) continue;  // this CTA has nothing of this entry (fewer units than CTAs)

            // ---- dependency on earlier entries ----
            if (E.flags & 1) {
                if (tid == 0) {
                    const unsigned int need = E.tiles_before;
                    guard.wait_flag([&] { return ld_acquire(p.tiles_done) >= need; });
                }
                consumer_sync();
            }
            // ---- stage x (pair-permuted) and its 128-column block sums ----
            for (int i = tid; i < 8 * (int)KB; i += kConsumerThreads) xsum[(i / KB) * p.kb_max + (i % KB)] = 0.f;
            consumer_sync();
            {
                const int items = M * (int)KB * 16;  // one item = 8 consecutive k of one row
                for (int it = tid; it < ((items + 31) & ~31); it += kConsumerThreads) {
                    float s = 0.f;
                    int r = 0, b8 = 0;
                    if (it < items) {
                        r = it / ((int)KB * 16);
                        b8 = it % ((int)KB * 16);
                        const uint4 v = __ldcg(reinterpret_cast<const uint4*>(E.x + (size_t)r * E.K + (size_t)b8 * 8));
                        uint4 o;
                        o.x = __byte_perm(v.x, v.z, 0x5410);  // (x0, x4)
                        o.y = __byte_perm(v.x, v.z, 0x7632);  // (x1, x5)
                        o.z = __byte_perm(v.y, v.w, 0x5410);  // (x2, x6)
                        o.w = __byte_perm(v.y, v.w, 0x7632);  // (x3, x7)
                        *reinterpret_cast<uint4*>(xs + (size_t)r * p.x_row_bytes + (size_t)b8 * 16) = o;
                        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            s += __uint_as_float(u[j] << 16) + __uint_as_float(u[j] & 0xFFFF0000u);
                    }
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    if ((lane & 15) == 0 && it < items) xsum[r * p.kb_max + (b8 >> 4)] = s;
                }
            }
            consumer_sync();

            const uint32_t t_first = u0 / KB, t_last = (u1 - 1) / KB;
            bool have_first = false;  // a cut first tile that this CTA completes at the end of the entry
            for (uint32_t tp = t_first; tp <= t_last; tp += kMaxTiles) {
                const uint32_t pu0 = max(u0, tp * KB), pu1 = min(u1, (tp + kMaxTiles) * KB);
                const uint32_t ntiles = min((uint32_t)kMaxTiles, t_last - tp + 1);
                for (int i = tid; i < (int)ntiles * kConsumerWarps * kElems / 4; i += kConsumerThreads)
                    reinterpret_cast<float4*>(tile_part)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                consumer_sync();

                float fin[4] = {0.f, 0.f, 0.f, 0.f};
                int cur_tile = -1;
                for (uint32_t cu = pu0; cu < pu1; cu += kStageUnits, ++ctr) {
                    const uint32_t n = min((uint32_t)kStageUnits, pu1 - cu);
                    const uint32_t s = ctr % p.stages, round = ctr / p.stages;
                    guard.wait_mbar(full0 + 8 * s, round & 1);
                    if ((uint32_t)warp < n) {
                        const uint32_t u = cu + warp;
                        const int tl = (int)(u / KB - tp);
                        const uint32_t kb = u % KB;
                        if (tl != cur_tile) {
                            if (cur_tile >= 0)
                                *reinterpret_cast<float4*>(tile_part + ((size_t)cur_tile * kConsumerWarps + warp) * kElems +
                                                           lane * 4) = make_float4(fin[0], fin[1], fin[2], fin[3]);
                            fin[0] = fin[1] = fin[2] = fin[3] = 0.f;
                            cur_tile = tl;
                        }
                        const unsigned char* ub = ring + (size_t)s * kStageBytes + (size_t)warp * kUnitBytes;
                        const uint4 wa = *reinterpret_cast<const uint4*>(ub + lane * 16);
                        const uint4 wb = *reinterpret_cast<const uint4*>(ub + 512 + lane * 16);
                        const __half2 ma = *reinterpret_cast<const __half2*>(ub + 1024 + 4 * g);
                        const __half2 mb = *reinterpret_cast<const __half2*>(ub + 1024 + 4 * (g + 8));
                        float acc[4][4];
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int q = 0; q < 4; ++q) acc[j][q] = 0.f;
                        const uint32_t was[4] = {wa.x, wa.y, wa.z, wa.w};
                        const uint32_t wbs[4] = {wb.x, wb.y, wb.z, wb.w};
                        const unsigned char* xrow = xs + (size_t)g * p.x_row_bytes + (size_t)(kb * 16 + t * 4) * 16;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 b = make_uint4(0, 0, 0, 0);
                            if (g < M) b = *reinterpret_cast<const uint4*>(xrow + j * 16);
                            mma_bf16_16816(acc[j], nib_pair(was[j], 0), nib_pair(wbs[j], 0), nib_pair(was[j], 1),
                                           nib_pair(wbs[j], 1), b.x, b.y);
                            mma_bf16_16816(acc[j], nib_pair(was[j], 2), nib_pair(wbs[j], 2), nib_pair(was[j], 3),
                                           nib_pair(wbs[j], 3), b.z, b.w);
                        }
                        const float sa = __low2float(ma), za = 128.f + __high2float(ma);
                        const float sb = __low2float(mb), zb = 128.f + __high2float(mb);
                        const float x0 = xsum[(2 * t) * p.kb_max + kb], x1 = xsum[(2 * t + 1) * p.kb_max + kb];
                        const float a0 = (acc[0][0] + acc[1][0]) + (acc[2][0] + acc[3][0]);
                        const float a1 = (acc[0][1] + acc[1][1]) + (acc[2][1] + acc[3][1]);
                        const float a2 = (acc[0][2] + acc[1][2]) + (acc[2][2] + acc[3][2]);
                        const float a3 = (acc[0][3] + acc[1][3]) + (acc[2][3] + acc[3][3]);
                        fin[0] = fmaf(sa, fmaf(-za, x0, a0), fin[0]);
                        fin[1] = fmaf(sa, fmaf(-za, x1, a1), fin[1]);
                        fin[2] = fmaf(sb, fmaf(-zb, x0, a2), fin[2]);
                        fin[3] = fmaf(sb, fmaf(-zb, x1, a3), fin[3]);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty0 + 8 * s);
                }
                if (cur_tile >= 0)
                    *reinterpret_cast<float4*>(tile_part + ((size_t)cur_tile * kConsumerWarps + warp) * kElems + lane * 4) =
                        make_float4(fin[0], fin[1], fin[2], fin[3]);
                consumer_sync();

                // ---- combine the warps (fixed order) and route every tile of the pass ----
                uint32_t n_full = 0;
                bool have_last = false;
                uint32_t last_rt = 0;
                for (uint32_t tl = 0; tl < ntiles; ++tl) {
                    const uint32_t rt = tp + tl;
                    const bool covers_begin = u0 <= rt * KB, covers_end = (rt + 1) * KB <= u1;
                    float sum = 0.f;
                    if (tid < kElems) {
#pragma unroll
                        for (int w = 0; w < kConsumerWarps; ++w) sum += tile_part[((size_t)tl * kConsumerWarps + w) * kElems + tid];
                    }
                    if (covers_begin && covers_end) {
                        ++n_full;
                        if (tid < kElems) {
                            // element tid = lane*4 + q of a warp fragment: q -> (row half, token parity)
                            const int ln = tid >> 2, q = tid & 3;
                            const int row = (ln >> 2) + ((q & 2) ? 8 : 0), tok = 2 * (ln & 3) + (q & 1);
                            if (tok < M) E.y[(size_t)tok * N + rt * 16 + row] = __float2bfloat16_rn(sum);
                        }
                    } else if (covers_end) {  // cut at its beginning: completed by this CTA later
                        have_first = true;
                        if (tid < kElems) stash_first[tid] = sum;
                    } else {  // the tile continues in the next CTA: publish the contribution
                        have_last = true;
                        last_rt = rt;
                        if (tid < kElems) stash_last[tid] = sum;
                    }
                }
                if (n_full && p.tiles_done) {
                    __threadfence();
                    consumer_sync();
                    if (tid == 0) red_release_add(p.tiles_done, n_full);
                }
                if (have_last) {
                    const uint32_t which = (last_rt == t_first) ? 0u : 1u;
                    unsigned char* slot = p.slots + ((size_t)c * 2 + which) * kSlotBytes;
                    unsigned int* flag = reinterpret_cast<unsigned int*>(slot + kElems * 4);
                    if (tid == 0) guard.wait_flag([&] { return ld_acquire(flag) == 0u; });
                    consumer_sync();
                    if (tid < kElems) reinterpret_cast<float*>(slot)[tid] = stash_last[tid];
                    __threadfence();
                    consumer_sync();
                    if (tid == 0) st_release(flag, (uint32_t)ei + 1u);  // the tag names the entry the data belongs to
                }
                consumer_sync();  // tile_part and the stashes are free again
            }

            // ---- complete the first tile of the slice from the contributions of earlier CTAs ----
            if (have_first) {
                const uint32_t rt = t_first;
                const uint32_t c_lo = owner_of(rt * KB, units, C);
                const uint32_t ncontrib = c - c_lo;
                for (uint32_t i = tid; i < ncontrib; i += kConsumerThreads) {
                    uint32_t which;
                    if (!contributor_slot(c_lo + i, rt, units, KB, C, which)) continue;
                    const unsigned int* flag = reinterpret_cast<const unsigned int*>(
                        p.slots + ((size_t)(c_lo + i) * 2 + which) * kSlotBytes + kElems * 4);
                    const uint32_t tag = (uint32_t)ei + 1u;
                    guard.wait_flag([&] { return ld_acquire(flag) == tag; });
                }
                consumer_sync();
                if (tid < kElems) {
                    float sum = 0.f;
                    for (uint32_t cc = c_lo; cc < c; ++cc) {
                        uint32_t which;
                        if (!contributor_slot(cc, rt, units, KB, C, which)) continue;
                        sum += __ldcg(reinterpret_cast<const float*>(p.slots + ((size_t)cc * 2 + which) * kSlotBytes) + tid);
                    }
                    sum += stash_first[tid];
                    const int ln = tid >> 2, q = tid & 3;
                    const int row = (ln >> 2) + ((q & 2) ? 8 : 0), tok = 2 * (ln & 3) + (q & 1);
                    if (tok < M) E.y[(size_t)tok * N + rt * 16 + row] = __float2bfloat16_rn(sum);
                }
                __threadfence();
                consumer_sync();
                for (uint32_t i = tid; i < ncontrib; i += kConsumerThreads) {
                    uint32_t which;
                    if (!contributor_slot(c_lo + i, rt, units, KB, C, which)) continue;
                    st_release(reinterpret_cast<unsigned int*>(p.slots + ((size_t)(c_lo + i) * 2 + which) * kSlotBytes +
                                                               kElems * 4), 0u);
                }
                if (tid == 0 && p.tiles_done) red_release_add(p.tiles_done, 1u);
                consumer_sync();
            }
        }
    }
    // nobody leaves before every copy has landed and every consumer is done with shared memory
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
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                word |= ((cc.x >> (8 * j)) & 0xFu) << (4 * j);
                word |= ((cc.y >> (8 * j)) & 0xFu) << (4 * (j + 4));
            }
        } else {
            const size_t gi = (size_t)(rt * 16 + (w - 256)) * ng + kb / bpg;
            word = (uint32_t)scales[gi] | ((uint32_t)zeros[gi] << 16);
        }
        out[i] = word;
    }
}

size_t smem_fixed_bytes(int x_rows, int x_row_bytes, int kb_max) {
    return (size_t)kMaxTiles * kConsumerWarps * kElems * 4 + 2 * kElems * 4 + (size_t)x_rows * x_row_bytes +
           (size_t)8 * kb_max * 4 + 64 /* poisoned flag + slack */;
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
    if (M < 1 || M > 8 || N < 16 || N % 16 != 0 || K % 128 != 0 || G % 128 != 0) return false;
    return stages_for(M, 2 * K + kRowPad, K / 128) >= 3;
}

size_t w4a16_stream_weight_bytes(int N, int K) { return (size_t)(N / 16) * (K / 128) * kUnitBytes; }

size_t w4a16_stream_workspace() { return (size_t)kWsHeader + (size_t)num_sms() * 2 * kSlotBytes; }

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
            e.flags = (i > 0) ? (d.flags & 1) : 0;
            e.tiles_before = tiles;
            e.pad = 0;
            tiles += (uint32_t)(d.N / 16);
            any_dep |= (e.flags & 1) != 0;
            if (d.M > x_rows) x_rows = d.M;
            if (d.K > kmax) kmax = d.K;
        }
        p.count = n;
        p.x_rows = x_rows;
        p.x_row_bytes = 2 * kmax + kRowPad;
        p.kb_max = kmax / 128;
        p.stages = stages_for(p.x_rows, p.x_row_bytes, p.kb_max);
        if (p.stages < 3) return QIL_ERR_UNSUPPORTED;
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
