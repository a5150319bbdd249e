// A list of independent W4A4 / W8A8 integer GEMMs as ONE persistent launch (the conv stages of the paper's driving
// policy, Sec. 5.1 / Sec. 5.4, Table "CILRS performance", are GEMMs of 2.6 to 3.2 G operations each: at the rate of
// the tensor cores each lasts well under a microsecond, less than a kernel needs to start, so what a GEMM costs is the
// start-up of its kernel unless several share one).
//
// Every GEMM is cut into output tiles of 128 x 64; the host deals the tiles of all GEMMs out to one CTA per SM,
// longest first, each to the CTA with the least work so far (K steps).  A CTA walks its tiles without stopping:
//   * 4 loader warps read the packed operands from global memory (three steps of loads in flight per thread), split
//     nibbles into signed bytes x 16 (8-bit operands are stored as they are) and store them as K-major operands,
//   * 1 thread issues the tcgen05.mma kind::i8 (128 x 64 x 32) of a step; tcgen05.commit recycles the stage (6 stages),
//     and after a tile's last step hands its accumulator to the read-out,
//   * 4 read-out warps (thread = output row) rescale and store; there are two accumulators in tensor memory, so the
//     read-out of a tile overlaps the steps of the next one.
// Arithmetic and operand layout are those of the single-GEMM kernel (w4a4.cu).  Every wait is bounded.
#include <algorithm>
#include <mutex>
#include <vector>

#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kTileM = 128, kTileN = 64;
constexpr int kStepBytes = 64;                 // operand bytes per row and step: 128 four-bit or 64 eight-bit elements
constexpr int kStages = 6;
constexpr int kALbo = kTileM * 16 + 16, kBLbo = kTileN * 16 + 16;  // (padded against bank conflicts, as in w4a4.cu)
constexpr int kAStage = 8 * kALbo, kBStage = 8 * kBLbo;
constexpr int kPre = 3;
constexpr int kThreads = 288;                  // 4 loader warps, the MMA warp, 4 read-out warps
constexpr int kMaxGemms = 8, kMaxTiles = 1200, kMaxCtas = 320;
constexpr int kCtasPerSm = 1;                  // (two CTAs per SM with half the stages measured slower)
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct Gemm {  // 72 bytes
    const uint32_t* qx;
    const uint32_t* qw;
    const float* sx;
    const float* sw;
    __nv_bfloat16* y;
    int32_t* acc_out;
    int M, N, K, bits;
    int tiles_n;     // column tiles
    int tile_base;   // number of this GEMM's first tile in the list
};

struct ListParams {
    Gemm g[kMaxGemms];
    unsigned short tile[kMaxTiles];     // tile numbers, grouped by CTA
    unsigned short first[kMaxCtas + 1]; // CTA c walks tile[first[c] .. first[c + 1])
    int count;
    int* status;
};

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
// D[128 x 64] (+)= A[128 x 32 s8] * B[64 x 32 s8]^T, int32 accumulate, operands in shared memory
__device__ __forceinline__ void mma_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
    constexpr uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)kTileN >> 3) << 17) | (((uint32_t)kTileM >> 4) << 24);
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 packed codes (one uint4) -> 32 signed bytes (x16) = two 16-byte K chunks
__device__ __forceinline__ void split32(const uint4& w, uint4& c0, uint4& c1) {
    constexpr uint32_t m = 0xF0F0F0F0u;
    c0 = make_uint4((w.x << 4) & m, w.x & m, (w.y << 4) & m, w.y & m);
    c1 = make_uint4((w.z << 4) & m, w.z & m, (w.w << 4) & m, w.w & m);
}

struct TileRef {
    int g, m0, n0, steps;
};
__device__ __forceinline__ TileRef tile_ref(const ListParams& p, int t) {
    int g = 0;
    while (g + 1 < p.count && t >= p.g[g + 1].tile_base) ++g;
    const Gemm& G = p.g[g];
    const int local = t - G.tile_base;
    TileRef r;
    r.g = g;
    r.m0 = (local / G.tiles_n) * kTileM;
    r.n0 = (local % G.tiles_n) * kTileN;
    const int step_k = kStepBytes * 8 / G.bits;
    r.steps = (G.K + step_k - 1) / step_k;
    return r;
}

__global__ void __launch_bounds__(kThreads, kCtasPerSm) igemm_list_kernel(const __grid_constant__ ListParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sa = smem;                                  // [kStages][kAStage]
    unsigned char* sb = smem + (size_t)kStages * kAStage;      // [kStages][kBStage]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sb + (size_t)kStages * kBStage);
    const uint32_t full0 = smem_u32(bars), free0 = smem_u32(bars + kStages);
    const uint32_t acc_full0 = smem_u32(bars + 2 * kStages), acc_free0 = smem_u32(bars + 2 * kStages + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int t_begin = p.first[blockIdx.x], t_end = p.first[blockIdx.x + 1];

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8 * s, 4);     // the loader warps
            mbar_init(free0 + 8 * s, 1);     // the commit of the MMAs that read the stage
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(acc_full0 + 8 * a, 1);   // the commit after the tile's last step
            mbar_init(acc_free0 + 8 * a, 4);   // the read-out warps
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * kTileN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (warp < 4) {
        // ---------------- loaders: lane = 16-byte piece tid % 4 of the step's 64 operand bytes of token rows tid / 4 + 32 j
        // (j < 4) and weight rows tid / 4 + 32 j (j < 2) ----------------
        const int pq = tid & 3, pr = tid >> 2;
        uint32_t s = 0, ph = 1;  // stage and the parity of "stage free" to wait for
        for (int ti = t_begin; ok && ti < t_end; ++ti) {
            const TileRef T = tile_ref(p, p.tile[ti]);
            const Gemm& G = p.g[T.g];
            const int row_words = G.K * G.bits / 32;
            const bool four = G.bits == 4;
            const uint32_t* xa = G.qx + (size_t)T.m0 * row_words + 4 * pq;
            const uint32_t* wb = G.qw + (size_t)T.n0 * row_words + 4 * pq;
            uint4 pa[kPre][4], pb[kPre][2];
            auto fetch = [&](uint4 (&da)[4], uint4 (&db)[2], int step) {  // operand words of one step (zeros beyond the matrix)
                const int w0 = step * (kStepBytes / 4);
                const bool in_k = w0 + 4 * pq < row_words;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int row = pr + 32 * j;
                    da[j] = (in_k && T.m0 + row < G.M) ? __ldg(reinterpret_cast<const uint4*>(xa + (size_t)row * row_words + w0))
                                                       : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int row = pr + 32 * j;
                    db[j] = (in_k && T.n0 + row < G.N) ? __ldg(reinterpret_cast<const uint4*>(wb + (size_t)row * row_words + w0))
                                                       : make_uint4(0, 0, 0, 0);
                }
            };
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
#pragma unroll
                for (int j = 0; j < 4; ++j) pa[u][j] = make_uint4(0, 0, 0, 0);
                pb[u][0] = pb[u][1] = make_uint4(0, 0, 0, 0);
                if (u < T.steps) fetch(pa[u], pb[u], u);
            }
            for (int step0 = 0; ok && step0 < T.steps; step0 += kPre) {
#pragma unroll
                for (int u = 0; u < kPre; ++u) {
                    const int step = step0 + u;
                    if (step >= T.steps) break;
                    ok = mbar_wait(free0 + 8 * s, ph);  // the MMAs that read this stage last are complete
                    if (!ok) break;
                    // 4-bit: piece pq = K chunks 2 pq, 2 pq + 1 of the step; 8-bit: piece pq = chunk pq
                    const int per = four ? 2 : 1;
                    unsigned char* a_st = sa + (size_t)s * kAStage + (size_t)(per * pq) * kALbo + (size_t)pr * 16;
                    unsigned char* b_st = sb + (size_t)s * kBStage + (size_t)(per * pq) * kBLbo + (size_t)pr * 16;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (four) {
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
                        if (four) {
                            uint4 c0, c1;
                            split32(pb[u][j], c0, c1);
                            *reinterpret_cast<uint4*>(b_st + (size_t)j * (32 * 16)) = c0;
                            *reinterpret_cast<uint4*>(b_st + (size_t)j * (32 * 16) + kBLbo) = c1;
                        } else {
                            *reinterpret_cast<uint4*>(b_st + (size_t)j * (32 * 16)) = pb[u][j];
                        }
                    }
                    if (step + kPre < T.steps) fetch(pa[u], pb[u], step + kPre);  // kPre steps stay in flight
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMAs read through the async proxy
                    __syncwarp();
                    if (lane == 0) mbar_arrive(full0 + 8 * s);
                    if (++s == kStages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 4) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            uint32_t s = 0, ph = 0;   // stage and the parity of "stage full" to wait for
            bool issued = false;
            int n_tile = 0;
            for (int ti = t_begin; ok && ti < t_end; ++ti, ++n_tile) {
                const TileRef T = tile_ref(p, p.tile[ti]);
                const int chunks = p.g[T.g].bits == 4 ? 8 : 4;
                const uint32_t acc = (uint32_t)(n_tile & 1), use = (uint32_t)(n_tile >> 1);
                ok = mbar_wait(acc_free0 + 8 * acc, (use & 1u) ^ 1u);  // the tile that used this accumulator has been read out
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int step = 0; step < T.steps; ++step) {
                    ok = mbar_wait(full0 + 8 * s, ph);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = smem_u32(sa + (size_t)s * kAStage), b_addr = smem_u32(sb + (size_t)s * kBStage);
                    for (int i = 0; i < chunks / 2; ++i)  // K = 32 each: chunks 2i, 2i + 1
                        mma_i8_ss(tmem + kTileN * acc, smem_desc(a_addr + 2 * i * kALbo, kALbo, 128),
                                  smem_desc(b_addr + 2 * i * kBLbo, kBLbo, 128), (step > 0 || i > 0) ? 1u : 0u);
                    tc_commit(free0 + 8 * s);
                    issued = true;
                    if (++s == kStages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                tc_commit(acc_full0 + 8 * acc);  // arrives when every MMA of the tile is complete
            }
            // every MMA issued is complete before tensor memory is released, whatever happened to the other roles
            if (issued) {
                const uint32_t last = smem_u32(bars + 2 * kStages + 5);  // (a barrier of its own for this last wait)
                mbar_init(last, 1);
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                tc_commit(last);
                (void)mbar_wait(last, 0);
            }
        }
    } else {
        // ---------------- read-out: thread r = accumulator row r ----------------
        const int r = (warp & 3) * 32 + lane;  // (a warp reads the quarter warp % 4 of the tensor-memory lanes)
        const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
        int n_tile = 0;
        for (int ti = t_begin; ok && ti < t_end; ++ti, ++n_tile) {
            const TileRef T = tile_ref(p, p.tile[ti]);
            const Gemm& G = p.g[T.g];
            const uint32_t acc = (uint32_t)(n_tile & 1), use = (uint32_t)(n_tile >> 1);
            const int m = T.m0 + r, N = G.N;
            const bool a_row = m < G.M;
            const float sxm = a_row ? __ldg(G.sx + m) : 0.f;
            const bool vec = (N % 8) == 0;
            ok = mbar_wait(acc_full0 + 8 * acc, use & 1u);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
            for (int c0 = 0; c0 < kTileN; c0 += 16) {
                uint32_t d[16];
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                    : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]), "=r"(d[8]),
                      "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15])
                    : "r"(tmem + lane_base + kTileN * acc + (uint32_t)c0));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int j = 0; j < 16; ++j) asm volatile("" : "+r"(d[j]));
                if (c0 + 16 >= kTileN) {  // the accumulator is in registers: the MMA warp may reuse it
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_free0 + 8 * acc);
                }
                if (!a_row) continue;
#pragma unroll
                for (int h = 0; h < 2; ++h) {  // 8 outputs = one 16-byte piece of the row
                    const int nb = T.n0 + c0 + 8 * h;
                    if (nb >= N) continue;
                    int a[8];
                    float sc[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        a[j] = G.bits == 4 ? ((int)d[8 * h + j] >> 8) : (int)d[8 * h + j];  // (4-bit: exact, a multiple of 256)
                        sc[j] = nb + j < N ? sxm * __ldg(G.sw + nb + j) : 0.f;
                    }
                    if (vec) {
                        uint32_t pk[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const __nv_bfloat162 v = __floats2bfloat162_rn((float)a[2 * j] * sc[2 * j], (float)a[2 * j + 1] * sc[2 * j + 1]);
                            pk[j] = *reinterpret_cast<const uint32_t*>(&v);
                        }
                        *reinterpret_cast<uint4*>(G.y + (size_t)m * N + nb) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        if (G.acc_out) {
                            *reinterpret_cast<int4*>(G.acc_out + (size_t)m * N + nb) = make_int4(a[0], a[1], a[2], a[3]);
                            *reinterpret_cast<int4*>(G.acc_out + (size_t)m * N + nb + 4) = make_int4(a[4], a[5], a[6], a[7]);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            if (nb + j < N) {
                                if (G.acc_out) G.acc_out[(size_t)m * N + nb + j] = a[j];
                                G.y[(size_t)m * N + nb + j] = __float2bfloat16_rn((float)a[j] * sc[j]);
                            }
                    }
                }
            }
        }
    }
    if (!ok && p.status) atomicOr(p.status, (int)QIL_ERR_TIMEOUT);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 4) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * kTileN));
}

constexpr size_t kSmemBytes = (size_t)kStages * (kAStage + kBStage) + (2 * kStages + 6) * 8 + 16;

}  // namespace

bool igemm_list_supported(const qil_igemm_desc* d, int count) {
    if (count < 1 || count > kMaxGemms) return false;
    long long tiles = 0;
    for (int i = 0; i < count; ++i)
        tiles += (long long)((d[i].M + kTileM - 1) / kTileM) * ((d[i].N + kTileN - 1) / kTileN);
    return tiles <= kMaxTiles && kCtasPerSm * num_sms() <= kMaxCtas;
}

// Every entry validated by the caller; entries are independent (no entry reads another entry's output).
qil_status launch_igemm_list(const qil_igemm_desc* d, int count, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (ws == nullptr || ws_bytes < 16) return QIL_ERR_WORKSPACE;
    static ListParams p;  // kept off the caller's stack; guarded by the mutex below
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    struct T { int id, steps; };
    std::vector<T> tiles;
    int base = 0;
    for (int i = 0; i < count; ++i) {
        Gemm& g = p.g[i];
        g.qx = reinterpret_cast<const uint32_t*>(d[i].qx);
        g.qw = reinterpret_cast<const uint32_t*>(d[i].qw);
        g.sx = d[i].sx; g.sw = d[i].sw;
        g.y = reinterpret_cast<__nv_bfloat16*>(d[i].y);
        g.acc_out = d[i].acc_out;
        g.M = d[i].M; g.N = d[i].N; g.K = d[i].K; g.bits = d[i].bits;
        g.tiles_n = (d[i].N + kTileN - 1) / kTileN;
        g.tile_base = base;
        const int n = ((d[i].M + kTileM - 1) / kTileM) * g.tiles_n;
        const int step_k = kStepBytes * 8 / d[i].bits;
        const int steps = (d[i].K + step_k - 1) / step_k;
        for (int t = 0; t < n; ++t) tiles.push_back({base + t, steps});
        base += n;
    }
    // longest first, each to the CTA with the least work so far (a tile costs its steps plus a constant)
    const int C = std::min(kCtasPerSm * num_sms(), (int)tiles.size());
    std::stable_sort(tiles.begin(), tiles.end(), [](const T& a, const T& b) { return a.steps > b.steps; });
    std::vector<std::vector<int>> per(C);
    std::vector<long> load(C, 0);
    for (const T& t : tiles) {
        int best = 0;
        for (int c = 1; c < C; ++c)
            if (load[c] < load[best]) best = c;
        per[best].push_back(t.id);
        load[best] += t.steps + 3;
    }
    int k = 0;
    for (int c = 0; c < C; ++c) {
        p.first[c] = (unsigned short)k;
        for (int id : per[c]) p.tile[k++] = (unsigned short)id;
    }
    p.first[C] = (unsigned short)k;
    p.count = count;
    p.status = reinterpret_cast<int*>(ws);
    if (cudaFuncSetAttribute(igemm_list_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    igemm_list_kernel<<<C, kThreads, kSmemBytes, st>>>(p);
    return launch_status();
}

}  // namespace qil
