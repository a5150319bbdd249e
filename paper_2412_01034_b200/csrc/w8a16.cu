// Weight-only 8-bit linears (the INT8 deployment point of the paper's OpenVLA table, Sec. 5.4: weights as uint8
// codes with an fp16 scale and zero point per group, bf16 activations): y = x . dequant(W)^T.
//
// Decode (few activation rows) is bound by HBM at one byte per weight, and the arithmetic is kept off the critical
// path by integer dot products on the CUDA cores:
//   * per 128 columns the activations become 16-bit block fixed point, x ~ 2^e v with |v| <= 32639, split into two
//     signed bytes v = 256 h + l (l in [-128, 127]); the planes h and l sit in shared memory, with the sum of v over
//     every 16-column chunk and 2^e per block;
//   * a lane reads 16 weight bytes of a row (one 128-bit load; a warp reads 512 contiguous bytes of the row), and
//     eight dp4a (four per plane) give sum q h and sum q l exactly in int32;
//   * V = 256 sum q h + sum q l = sum q v exactly, and the chunk's contribution is s 2^e (V - z X), X the chunk's
//     sum of v: one fp32 multiply-add per 16 weights.
// A warp carries four rows at once, so the activation planes are read once per four weight loads.
//
// One persistent launch runs a whole list of linears.  Rows are never split: the rows of all entries of a phase (a
// run of entries that do not wait for each other) are dealt out in contiguous, byte-balanced ranges, one per CTA, so
// nothing is exchanged between CTAs.  An entry with QIL_DEP_PREVIOUS starts a new phase: every CTA counts itself in
// at the end of a phase and waits (bounded) until all have.  Every wait has a limit; when it runs out
// QIL_ERR_TIMEOUT is recorded in the status word and the CTA leaves.
#include <algorithm>
#include <atomic>
#include <mutex>

#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kRows = 4;          // rows a warp carries at once
constexpr int kMaxEntries = 256;
constexpr int kMaxM = 4;
constexpr size_t kSmemLimit = 232448;
constexpr unsigned long long kDefaultWaitNs = 2000000000ull;

struct W8Entry {  // 64 bytes
    const uint16_t* x;
    const uint8_t* w;
    const __half* s;
    const __half* z;
    __nv_bfloat16* y;
    int N, K, M;
    int chunks_per_group;  // group_size / 16
    int flags;             // bit 0: starts a phase that waits for all earlier phases
    int pad;
    unsigned long long base;   // bytes of the phase before this entry
    unsigned long long total;  // bytes of the phase
};

struct W8Params {
    W8Entry e[kMaxEntries];
    int count;
    int k_max;                 // largest K of the list (sizes the activation planes)
    unsigned long long wait_ns;
    int* status;
    unsigned int* arrived;     // CTAs that have finished phase 0, 1, ... (one counter, counts up)
};

__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {  // unsigned bytes of a x signed bytes of b
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ unsigned long long now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Activation planes of one entry in shared memory, for token t: h[K], l[K] (signed bytes), xc[K/16] (int: sum of v
// over the chunk), pe[K/128] (float 2^e).
struct Planes {
    unsigned char* h;
    unsigned char* l;
    int* xc;
    float* pe;
    int kmax;
    __device__ Planes(unsigned char* smem, int kmax_) : kmax(kmax_) {
        h = smem;
        l = h + (size_t)kMaxM * kmax;
        xc = reinterpret_cast<int*>(l + (size_t)kMaxM * kmax);
        pe = reinterpret_cast<float*>(xc + (size_t)kMaxM * (kmax / 16));
    }
};

// bf16 rows -> block fixed point planes; a warp converts one 128-column block of one token per pass
__device__ void stage_x(const W8Entry& E, const Planes& P) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = E.K >> 7;
    for (int task = warp; task < E.M * KB; task += kWarps) {
        const int t = task / KB, b = task - t * KB;
        const uint2 raw = __ldcg(reinterpret_cast<const uint2*>(E.x + (size_t)t * E.K + (size_t)b * 128 + lane * 4));
        const uint32_t u[2] = {raw.x, raw.y};
        uint32_t amax = 0;  // bf16 magnitudes order like unsigned integers
#pragma unroll
        for (int j = 0; j < 2; ++j) amax = max(amax, max((u[j] << 16) & 0x7FFFFFFFu, u[j] & 0x7FFF0000u));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        // 2^e = smallest power of two with max|x| / 2^e <= 32639 (exponent field F -> F - 127 - 14, one more when the
        // mantissa exceeds 32639/16384); zero, subnormal or non-finite blocks use 2^0
        int ef = (int)(amax >> 23);
        if (ef < 1 || ef >= 255) ef = 127 + 14;
        int e = ef - 127 - 14 + (((amax & 0x7FFFFFu) > 0x7EFE00u) ? 1 : 0);
        if (e < -126) e = -126;
        const float inv = __uint_as_float((uint32_t)(127 - e) << 23);  // 2^-e
        int v[4];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            v[2 * j] = __float2int_rn(__uint_as_float(u[j] << 16) * inv);
            v[2 * j + 1] = __float2int_rn(__uint_as_float(u[j] & 0xFFFF0000u) * inv);
        }
        uint32_t hw = 0, lw = 0;
        int sum = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int hi = (v[j] + 128) >> 8, lo = v[j] - (hi << 8);  // lo in [-128, 127]
            hw |= ((uint32_t)hi & 0xFFu) << (8 * j);
            lw |= ((uint32_t)lo & 0xFFu) << (8 * j);
            sum += v[j];
        }
        const size_t off = (size_t)t * P.kmax + (size_t)b * 128 + lane * 4;
        *reinterpret_cast<uint32_t*>(P.h + off) = hw;
        *reinterpret_cast<uint32_t*>(P.l + off) = lw;
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        if ((lane & 3) == 0) P.xc[(size_t)t * (P.kmax / 16) + b * 8 + (lane >> 2)] = sum;
        if (lane == 0) P.pe[(size_t)t * (P.kmax / 128) + b] = __uint_as_float((uint32_t)(127 + e) << 23);
    }
}

template <int kM>
__global__ void __launch_bounds__(kThreads, 1) w8a16_stream_kernel(const __grid_constant__ W8Params p) {
    extern __shared__ __align__(16) unsigned char smem[];
    const Planes P(smem, p.k_max);
    int2* rows = reinterpret_cast<int2*>(P.pe + (size_t)kMaxM * (p.k_max / 128));  // [count] {first row, end row} of this CTA
    __shared__ int dead;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const unsigned long long C = gridDim.x, c = blockIdx.x;

    if (tid == 0) dead = 0;
    for (int i = tid; i < p.count; i += kThreads) {
        // rows whose first byte lies in this CTA's byte range of the phase
        const W8Entry& E = p.e[i];
        const unsigned long long lo = c * E.total / C, hi = (c + 1) * E.total / C;
        const unsigned long long bytes = (unsigned long long)E.N * E.K, K = (unsigned long long)E.K;
        const unsigned long long a = lo > E.base ? lo - E.base : 0ull;
        const unsigned long long b = hi > E.base ? (hi - E.base < bytes ? hi - E.base : bytes) : 0ull;
        const int r0 = (int)((a + K - 1) / K), r1 = (int)((b + K - 1) / K);
        rows[i] = make_int2(r0 < E.N ? r0 : E.N, r1 < E.N ? r1 : E.N);
    }
    __syncthreads();

    unsigned int phases_done = 0;
    for (int ei = 0; ei < p.count; ++ei) {
        const W8Entry& E = p.e[ei];
        if (ei > 0 && (E.flags & 1)) {
            // end of a phase: count this CTA in (its outputs are written), then wait for all CTAs
            __syncthreads();
            if (tid == 0) {
                __threadfence();
                atomicAdd(p.arrived, 1u);
                ++phases_done;
                const unsigned int need = (E.flags & 2) ? 0xFFFFFFFFu : (unsigned int)C * phases_done;
                const unsigned long long t0 = now_ns();
                unsigned int spins = 0;
                while (*reinterpret_cast<volatile unsigned int*>(p.arrived) < need) {
                    if (++spins > 4) __nanosleep(64);
                    if ((spins & 15u) == 0u && now_ns() - t0 > p.wait_ns) {
                        atomicOr(p.status, (int)QIL_ERR_TIMEOUT);
                        dead = 1;
                        break;
                    }
                }
                __threadfence();
            }
            __syncthreads();
            if (dead) break;
        }
        const int2 rr = rows[ei];
        if (rr.x >= rr.y) continue;
        __syncthreads();  // every warp is done with the previous entry's planes
        stage_x(E, P);
        __syncthreads();

        const int K = E.K, chunks = K >> 4, cpg = E.chunks_per_group, ng = chunks / cpg;
        const int cpg_shift = (cpg & (cpg - 1)) == 0 ? __ffs(cpg) - 1 : -1;  // groups of a power of two: no division
        for (int r0 = rr.x + kRows * warp; r0 < rr.y; r0 += kRows * kWarps) {
            float fin[kRows][kM];
#pragma unroll
            for (int r = 0; r < kRows; ++r)
#pragma unroll
                for (int t = 0; t < kM; ++t) fin[r][t] = 0.f;
            const uint8_t* wrow[kRows];
            int nrow[kRows];
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                nrow[r] = min(r0 + r, rr.y - 1);  // (rows past the range repeat the last one; they are not written)
                wrow[r] = E.w + (size_t)nrow[r] * K;
            }
            uint4 cur[kRows], nxt[kRows];
#pragma unroll
            for (int r = 0; r < kRows; ++r) cur[r] = lane < chunks ? ld_stream_u4(wrow[r] + 16 * lane) : make_uint4(0, 0, 0, 0);
            for (int j = lane; j < chunks; j += 32) {
                const int jn = j + 32;
#pragma unroll
                for (int r = 0; r < kRows; ++r) nxt[r] = jn < chunks ? ld_stream_u4(wrow[r] + 16 * (size_t)jn) : make_uint4(0, 0, 0, 0);
                const int g = cpg_shift >= 0 ? (j >> cpg_shift) : j / cpg;
                float s[kRows];
                int z[kRows];
#pragma unroll
                for (int r = 0; r < kRows; ++r) {
                    s[r] = __half2float(__ldg(E.s + (size_t)nrow[r] * ng + g));
                    z[r] = __half2int_rn(__ldg(E.z + (size_t)nrow[r] * ng + g));
                }
#pragma unroll
                for (int t = 0; t < kM; ++t) {
                    if (t < E.M) {
                        const uint4 xh = *reinterpret_cast<const uint4*>(P.h + (size_t)t * P.kmax + 16 * (size_t)j);
                        const uint4 xl = *reinterpret_cast<const uint4*>(P.l + (size_t)t * P.kmax + 16 * (size_t)j);
                        const int X = P.xc[(size_t)t * (P.kmax / 16) + j];
                        const float pe = P.pe[(size_t)t * (P.kmax / 128) + (j >> 3)];
#pragma unroll
                        for (int r = 0; r < kRows; ++r) {
                            int ah = dp4a_us(cur[r].x, xh.x, 0), al = dp4a_us(cur[r].x, xl.x, 0);
                            ah = dp4a_us(cur[r].y, xh.y, ah); al = dp4a_us(cur[r].y, xl.y, al);
                            ah = dp4a_us(cur[r].z, xh.z, ah); al = dp4a_us(cur[r].z, xl.z, al);
                            ah = dp4a_us(cur[r].w, xh.w, ah); al = dp4a_us(cur[r].w, xl.w, al);
                            const int v = ah * 256 + al - z[r] * X;  // |.| < 2^31: 16 x 255 x 32767 x 2
                            fin[r][t] = fmaf((float)v, s[r] * pe, fin[r][t]);
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < kRows; ++r) cur[r] = nxt[r];
            }
#pragma unroll
            for (int r = 0; r < kRows; ++r)
#pragma unroll
                for (int t = 0; t < kM; ++t) fin[r][t] = warp_sum(fin[r][t]);
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < kRows; ++r)
                    if (r0 + r < rr.y) {
#pragma unroll
                        for (int t = 0; t < kM; ++t)
                            if (t < E.M) E.y[(size_t)t * E.N + r0 + r] = __float2bfloat16_rn(fin[r][t]);
                    }
            }
        }
    }
}

// Any shape (K % 16 == 0, any group size dividing K): a warp per output feature, fp32 multiply-adds.
__global__ void __launch_bounds__(256) w8a16_general_kernel(const uint16_t* __restrict__ x, const uint8_t* __restrict__ w,
                                                            const __half* __restrict__ s, const __half* __restrict__ z,
                                                            __nv_bfloat16* __restrict__ y, int M, int N, int K, int G) {
    const int lane = threadIdx.x & 31;
    const int ng = K / G;
    const long long total = (long long)M * N, warps = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long o = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); o < total; o += warps) {
        const int m = (int)(o / N), n = (int)(o % N);
        float acc = 0.f;
        for (int k = lane; k < K; k += 32) {
            const int g = k / G;
            const float wv = ((float)w[(size_t)n * K + k] - __half2float(z[(size_t)n * ng + g])) * __half2float(s[(size_t)n * ng + g]);
            acc = fmaf(bf16_bits_to_f32(x[(size_t)m * K + k]), wv, acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) y[(size_t)m * N + n] = __float2bfloat16_rn(acc);
    }
}

size_t stream_smem(int k_max, int count) {
    return (size_t)kMaxM * k_max * 2 + (size_t)kMaxM * (k_max / 16) * 4 + (size_t)kMaxM * (k_max / 128) * 4 + (size_t)count * 8 + 16;
}

std::atomic<unsigned long long> g_wait_ns{kDefaultWaitNs};

template <int kM>
cudaError_t launch_stream(const W8Params& p, int C, size_t smem, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(w8a16_stream_kernel<kM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // the CTAs wait for each other between phases: all of them must be resident (cooperative launch)
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
    return cudaLaunchKernelEx(&cfg, w8a16_stream_kernel<kM>, p);
}

}  // namespace

void w8a16_set_wait_limit(unsigned long long ns) { g_wait_ns.store(ns ? ns : kDefaultWaitNs); }

bool w8a16_stream_supported(int M, int N, int K, int G) {
    if (M < 1 || M > kMaxM || N < 1 || K % 128 != 0 || G % 128 != 0 || K % G != 0) return false;
    return stream_smem(K, kMaxEntries) <= kSmemLimit;
}

size_t w8a16_workspace() { return 256; }

qil_status launch_w8a16_general(const void* x, const uint8_t* w, const void* s, const void* z, void* y, int M, int N, int K,
                                int G, cudaStream_t st) {
    long long blocks = ((long long)M * N + 7) / 8;
    const long long cap = (long long)num_sms() * 16;
    if (blocks > cap) blocks = cap;
    w8a16_general_kernel<<<(int)blocks, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), w, reinterpret_cast<const __half*>(s),
                                                      reinterpret_cast<const __half*>(z), reinterpret_cast<__nv_bfloat16*>(y), M,
                                                      N, K, G);
    return launch_status();
}

// Every entry must satisfy w8a16_stream_supported(); scales and zeros are [N][K / group_size] fp16.
qil_status launch_w8a16_stream(const qil_linear_desc* entries, int count, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (ws == nullptr || ws_bytes < w8a16_workspace()) return QIL_ERR_WORKSPACE;
    static W8Params p;  // 16 KiB: kept off the caller's stack; guarded by the mutex below
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    const int C = num_sms();
    for (int first = 0; first < count; first += kMaxEntries) {
        const int n = count - first < kMaxEntries ? count - first : kMaxEntries;
        int max_m = 1, k_max = 128;
        bool any_dep = false;
        for (int i = 0; i < n; ++i) {
            const qil_linear_desc& d = entries[first + i];
            W8Entry& e = p.e[i];
            e.x = reinterpret_cast<const uint16_t*>(d.x);
            e.w = reinterpret_cast<const uint8_t*>(d.qweight);
            e.s = reinterpret_cast<const __half*>(d.scales);
            e.z = reinterpret_cast<const __half*>(d.zeros);
            e.y = reinterpret_cast<__nv_bfloat16*>(d.y);
            e.N = d.N; e.K = d.K; e.M = d.M;
            e.chunks_per_group = d.group_size / 16;
            e.flags = 0;
            if (i > 0 && (d.flags & (QIL_DEP_PREVIOUS | QIL_DEP_NEVER))) e.flags = 1 | ((d.flags & QIL_DEP_NEVER) ? 2 : 0);
            e.pad = 0;
            any_dep |= e.flags != 0;
            max_m = std::max(max_m, d.M);
            k_max = std::max(k_max, d.K);
        }
        for (int i = 0; i < n;) {  // phases: byte offsets of their entries
            int j = i + 1;
            while (j < n && !p.e[j].flags) ++j;
            unsigned long long total = 0;
            for (int k = i; k < j; ++k) {
                p.e[k].base = total;
                total += (unsigned long long)p.e[k].N * p.e[k].K;
            }
            for (int k = i; k < j; ++k) p.e[k].total = total;
            i = j;
        }
        p.count = n;
        p.k_max = k_max;
        p.wait_ns = g_wait_ns.load();
        p.status = reinterpret_cast<int*>(ws);
        p.arrived = reinterpret_cast<unsigned int*>(ws) + 1;
        if (any_dep && cudaMemsetAsync(p.arrived, 0, 4, st) != cudaSuccess) {
            (void)cudaGetLastError();
            return QIL_ERR_CUDA;
        }
        const size_t smem = stream_smem(k_max, n);
        if (smem > kSmemLimit) return QIL_ERR_UNSUPPORTED;
        const cudaError_t err = max_m <= 1 ? launch_stream<1>(p, C, smem, st)
                                : max_m <= 2 ? launch_stream<2>(p, C, smem, st)
                                             : launch_stream<4>(p, C, smem, st);
        if (err != cudaSuccess) {
            (void)cudaGetLastError();
            return err == cudaErrorCooperativeLaunchTooLarge ? QIL_ERR_UNSUPPORTED : QIL_ERR_CUDA;
        }
    }
    return QIL_OK;
}

}  // namespace qil
