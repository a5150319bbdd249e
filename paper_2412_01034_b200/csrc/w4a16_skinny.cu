// Weight-only 4-bit linear for few activation rows (decode, M <= 64 per slab):
// the memory-bound stage of the paper's OpenVLA deployment (Sec. 5.4, App. A.4.2).
//
// Every packed weight is read from HBM exactly once.  A warp owns a tile of
// 16 output features x 128 input features (1 KiB of packed codes):
//   * two 128-bit loads per lane fetch the tile (rows g and g+8 of the tile,
//     words 4t..4t+3, with g = lane/4, t = lane%4);
//   * each 32-bit word (8 codes) becomes four bf16x2 registers holding 128+q via
//     (w >> 4i) & 0x000F000F | 0x43004300 - the pairs are (k0,k4) (k1,k5) (k2,k6)
//     (k3,k7);
//   * the registers are A fragments of mma.sync m16n8k16 (bf16 in, fp32 out); the
//     activations are staged in shared memory in the same pair order, so the
//     permutation of k cancels in the sum;
//   * per 128-column block the warp holds sum_k (128+q) x in fp32 and folds scale
//     and zero once per block:  y += s * (acc - (128 + z) * X),  X = sum_k x over
//     the block (computed once per CTA while staging x).
// Lanes therefore only unpack (7 integer ops per 8 weights); the multiply-adds for
// up to 8 activation rows cost one tensor instruction per 256 weights.
//
// Work split: grid = (row tiles, K slices).  The 8 warps of a CTA take the
// 128-column blocks of the CTA's K slice round-robin, then combine in shared
// memory in a fixed order.  With more than one K slice the CTAs leave fp32
// partial tiles in the workspace; the last CTA to arrive (bounded by nothing: it
// is decided by an atomic counter, no CTA ever waits for another) adds them in
// slice order, so the result does not depend on arrival order.
#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kCounterBytes = 16384;  // arrival counters at the start of the workspace (4096 row tiles max)
constexpr int kRowPadBytes = 16;      // shared-memory row skew that keeps the 128-bit reads conflict-free

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// bf16x2 {128 + nibble i, 128 + nibble i+4} of a packed word
__device__ __forceinline__ uint32_t nib_pair(uint32_t w, int i) {
    return ((w >> (4 * i)) & 0x000F000Fu) | 0x43004300u;
}

struct SkinnyParams {
    const uint16_t* x;
    const uint32_t* qw;
    const __half* scales;
    const __half* zeros;
    __nv_bfloat16* y;
    int M, N, K;
    int blocks_per_group;  // group_size / 128
    int layout;
    int kblocks;           // K / 128
    int slices;            // gridDim.y
    int chunk_blocks;      // 128-column blocks of x staged per pass
    int rows_staged;       // min(M, 8*MT)
    int m0;                // first activation row of this slab
    int* counters;
    float* partials;
};

template <int MT>
__global__ void __launch_bounds__(kThreads) w4a16_skinny_kernel(const SkinnyParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int rt = blockIdx.x, slice = blockIdx.y;
    const int n0 = rt * 16;
    const int words = p.K >> 3;
    const int ng = p.kblocks / p.blocks_per_group;

    // K slice of this CTA
    const int per = p.kblocks / p.slices, rem = p.kblocks % p.slices;
    const int kb_begin = slice * per + min(slice, rem);
    const int kb_end = kb_begin + per + (slice < rem ? 1 : 0);

    const int row_bytes = p.chunk_blocks * 256 + kRowPadBytes;
    unsigned char* xs = smem;                                                    // [rows_staged][row_bytes]
    float* xsum = reinterpret_cast<float*>(smem + (size_t)p.rows_staged * row_bytes);  // [8*MT][chunk_blocks]
    float* red = xsum + 8 * MT * p.chunk_blocks;                                 // [kWarps][4*MT][32]

    float fin[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int c = 0; c < 4; ++c) fin[mt][c] = 0.f;

    const bool row_a_ok = (n0 + g) < p.N, row_b_ok = (n0 + g + 8) < p.N;
    const int rows_in_slab = min(p.M - p.m0, 8 * MT);

    for (int cb = kb_begin; cb < kb_end; cb += p.chunk_blocks) {
        const int nblk = min(p.chunk_blocks, kb_end - cb);
        __syncthreads();  // previous pass is done with xs / xsum
        // ---- stage x[m0 .. m0+rows)[cb*128 .. (cb+nblk)*128) permuted, and the block sums ----
        for (int i = tid; i < 8 * MT * p.chunk_blocks; i += kThreads) xsum[i] = 0.f;
        __syncthreads();
        const int items = rows_in_slab * nblk * 16;  // one item = 8 consecutive k of one row
        for (int it = tid; it < ((items + 31) & ~31); it += kThreads) {  // whole warps stay in the loop
            float s = 0.f;
            int r = 0, b8 = 0;
            if (it < items) {
                r = it / (nblk * 16);
                b8 = it % (nblk * 16);
                const uint4 v = *reinterpret_cast<const uint4*>(p.x + (size_t)(p.m0 + r) * p.K +
                                                                (size_t)cb * 128 + (size_t)b8 * 8);
                uint4 o;
                o.x = __byte_perm(v.x, v.z, 0x5410);  // (x0, x4)
                o.y = __byte_perm(v.x, v.z, 0x7632);  // (x1, x5)
                o.z = __byte_perm(v.y, v.w, 0x5410);  // (x2, x6)
                o.w = __byte_perm(v.y, v.w, 0x7632);  // (x3, x7)
                *reinterpret_cast<uint4*>(xs + (size_t)r * row_bytes + (size_t)b8 * 16) = o;
                const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    s += __uint_as_float(u[j] << 16) + __uint_as_float(u[j] & 0xFFFF0000u);
            }
            // 16 consecutive items form one 128-column block of one row
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if ((lane & 15) == 0 && it < items) xsum[r * p.chunk_blocks + (b8 >> 4)] = s;
        }
        __syncthreads();

        // ---- this warp's blocks of the chunk ----
        for (int kl = warp; kl < nblk; kl += kWarps) {
            const int kb = cb + kl;
            uint4 wa = make_uint4(0, 0, 0, 0), wb = make_uint4(0, 0, 0, 0);
            if (p.layout == QIL_LAYOUT_TILE16) {
                const uint32_t* tile = p.qw + ((size_t)rt * p.kblocks + kb) * 256;
                wa = ld_stream_u4(tile + lane * 4);
                wb = ld_stream_u4(tile + 128 + lane * 4);
            } else {
                if (row_a_ok) wa = ld_stream_u4(p.qw + (size_t)(n0 + g) * words + kb * 16 + t * 4);
                if (row_b_ok) wb = ld_stream_u4(p.qw + (size_t)(n0 + g + 8) * words + kb * 16 + t * 4);
            }
            const int gi = kb / p.blocks_per_group;
            float sa = 0.f, sb = 0.f, za = 0.f, zb = 0.f;
            if (row_a_ok) {
                sa = __half2float(p.scales[(size_t)(n0 + g) * ng + gi]);
                za = 128.f + __half2float(p.zeros[(size_t)(n0 + g) * ng + gi]);
            }
            if (row_b_ok) {
                sb = __half2float(p.scales[(size_t)(n0 + g + 8) * ng + gi]);
                zb = 128.f + __half2float(p.zeros[(size_t)(n0 + g + 8) * ng + gi]);
            }
            float acc[MT][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[mt][c] = 0.f;

            const uint32_t was[4] = {wa.x, wa.y, wa.z, wa.w};
            const uint32_t wbs[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t a0 = nib_pair(was[j], 0), a1 = nib_pair(wbs[j], 0);
                const uint32_t a2 = nib_pair(was[j], 1), a3 = nib_pair(wbs[j], 1);
                const uint32_t a4 = nib_pair(was[j], 2), a5 = nib_pair(wbs[j], 2);
                const uint32_t a6 = nib_pair(was[j], 3), a7 = nib_pair(wbs[j], 3);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const int tok = mt * 8 + g;
                    uint4 b = make_uint4(0, 0, 0, 0);
                    if (tok < rows_in_slab)
                        b = *reinterpret_cast<const uint4*>(xs + (size_t)tok * row_bytes +
                                                            (size_t)(kl * 16 + t * 4 + j) * 16);
                    mma_bf16_16816(acc[mt], a0, a1, a2, a3, b.x, b.y);
                    mma_bf16_16816(acc[mt], a4, a5, a6, a7, b.z, b.w);
                }
            }
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const float x0 = xsum[(mt * 8 + 2 * t) * p.chunk_blocks + kl];
                const float x1 = xsum[(mt * 8 + 2 * t + 1) * p.chunk_blocks + kl];
                fin[mt][0] = fmaf(sa, fmaf(-za, x0, acc[mt][0]), fin[mt][0]);
                fin[mt][1] = fmaf(sa, fmaf(-za, x1, acc[mt][1]), fin[mt][1]);
                fin[mt][2] = fmaf(sb, fmaf(-zb, x0, acc[mt][2]), fin[mt][2]);
                fin[mt][3] = fmaf(sb, fmaf(-zb, x1, acc[mt][3]), fin[mt][3]);
            }
        }
    }

    // ---- combine the 8 warps in a fixed order ----
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int c = 0; c < 4; ++c) red[(warp * 4 * MT + mt * 4 + c) * 32 + lane] = fin[mt][c];
    __syncthreads();

    __shared__ int is_last;
    const int elems = 4 * MT * 32;
    float* my_partial = p.partials ? p.partials + ((size_t)slice * gridDim.x + rt) * elems : nullptr;
    for (int e = tid; e < elems; e += kThreads) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += red[w * elems + e];
        if (p.slices == 1) {
            const int ln = e & 31, c = (e >> 5) & 3, mt = e >> 7;
            const int row = n0 + (ln >> 2) + ((c & 2) ? 8 : 0);
            const int tok = mt * 8 + 2 * (ln & 3) + (c & 1);
            if (row < p.N && tok < rows_in_slab) p.y[(size_t)(p.m0 + tok) * p.N + row] = __float2bfloat16_rn(s);
        } else {
            my_partial[e] = s;
        }
    }
    if (p.slices == 1) return;

    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(&p.counters[rt], 1);
        is_last = (prev == p.slices - 1);
        if (is_last) p.counters[rt] = 0;  // leave the workspace ready for the next call
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int e = tid; e < elems; e += kThreads) {
        float s = 0.f;
        for (int sl = 0; sl < p.slices; ++sl) s += __ldcg(p.partials + ((size_t)sl * gridDim.x + rt) * elems + e);
        const int ln = e & 31, c = (e >> 5) & 3, mt = e >> 7;
        const int row = n0 + (ln >> 2) + ((c & 2) ? 8 : 0);
        const int tok = mt * 8 + 2 * (ln & 3) + (c & 1);
        if (row < p.N && tok < rows_in_slab) p.y[(size_t)(p.m0 + tok) * p.N + row] = __float2bfloat16_rn(s);
    }
}

struct SkinnyPlan {
    int mt;            // 8-row activation tiles per slab (1, 2, 4, 8)
    int slices;        // K slices
    int chunk_blocks;  // staged 128-column blocks per pass
    int rows_staged;
    size_t smem;
};

SkinnyPlan make_plan(int M, int N, int K) {
    SkinnyPlan pl;
    const int slab = M < 64 ? M : 64;
    pl.mt = slab <= 8 ? 1 : slab <= 16 ? 2 : slab <= 32 ? 4 : 8;
    pl.rows_staged = slab;
    const int kblocks = K / 128;
    const int row_tiles = (N + 15) / 16;
    // enough CTAs for about four per SM, but never slices shorter than one block per warp
    int slices = (4 * num_sms() + row_tiles - 1) / row_tiles;
    int max_slices = kblocks / kWarps;
    if (max_slices < 1) max_slices = 1;
    if (slices > max_slices) slices = max_slices;
    if (slices < 1) slices = 1;
    pl.slices = slices;
    const int slice_blocks = (kblocks + slices - 1) / slices;
    const size_t budget = (slab <= 16 ? 96 : 200) * 1024;
    const size_t fixed = (size_t)kWarps * 4 * pl.mt * 32 * 4;
    int cb = slice_blocks;
    while (cb > 1 && (size_t)slab * (cb * 256 + kRowPadBytes) + (size_t)8 * pl.mt * cb * 4 + fixed > budget) --cb;
    pl.chunk_blocks = cb;
    pl.smem = (size_t)slab * (cb * 256 + kRowPadBytes) + (size_t)8 * pl.mt * cb * 4 + fixed;
    return pl;
}

}  // namespace

bool w4a16_skinny_supported(int M, int N, int K, int G, qil_layout layout) {
    (void)M;
    if (K % 128 != 0 || G % 128 != 0) return false;
    if (layout == QIL_LAYOUT_TILE16 && N % 16 != 0) return false;
    if ((N + 15) / 16 > kCounterBytes / 4) return false;
    return true;
}

size_t w4a16_skinny_counter_bytes() { return kCounterBytes; }

size_t w4a16_skinny_workspace(int M, int N, int K, int G) {
    (void)G;
    const SkinnyPlan pl = make_plan(M, N, K);
    if (pl.slices == 1) return 0;
    const size_t row_tiles = (N + 15) / 16;
    return (size_t)kCounterBytes + (size_t)pl.slices * row_tiles * 4 * pl.mt * 32 * sizeof(float);
}

qil_status launch_w4a16_skinny(const void* x, const uint32_t* qw, const void* scales, const void* zeros,
                               void* y, int M, int N, int K, int G, qil_layout layout, void* ws,
                               size_t ws_bytes, cudaStream_t st) {
    const SkinnyPlan pl = make_plan(M, N, K);
    if (pl.slices > 1 && (ws == nullptr || ws_bytes < w4a16_skinny_workspace(M, N, K, G))) return QIL_ERR_WORKSPACE;
    SkinnyParams p;
    p.x = reinterpret_cast<const uint16_t*>(x);
    p.qw = qw;
    p.scales = reinterpret_cast<const __half*>(scales);
    p.zeros = reinterpret_cast<const __half*>(zeros);
    p.y = reinterpret_cast<__nv_bfloat16*>(y);
    p.M = M; p.N = N; p.K = K;
    p.blocks_per_group = G / 128;
    p.layout = (int)layout;
    p.kblocks = K / 128;
    p.slices = pl.slices;
    p.chunk_blocks = pl.chunk_blocks;
    p.rows_staged = pl.rows_staged;
    p.counters = pl.slices > 1 ? reinterpret_cast<int*>(ws) : nullptr;
    p.partials = pl.slices > 1 ? reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + kCounterBytes) : nullptr;
    const dim3 grid((N + 15) / 16, pl.slices);
    for (int m0 = 0; m0 < M; m0 += 64) {
        p.m0 = m0;
        cudaError_t e = cudaSuccess;
#define QIL_LAUNCH(MT)                                                                                          \
    do {                                                                                                        \
        e = cudaFuncSetAttribute(w4a16_skinny_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,          \
                                 (int)pl.smem);                                                                 \
        if (e == cudaSuccess) w4a16_skinny_kernel<MT><<<grid, kThreads, pl.smem, st>>>(p);                      \
    } while (0)
        switch (pl.mt) {
            case 1: QIL_LAUNCH(1); break;
            case 2: QIL_LAUNCH(2); break;
            case 4: QIL_LAUNCH(4); break;
            default: QIL_LAUNCH(8); break;
        }
#undef QIL_LAUNCH
        if (e != cudaSuccess) return QIL_ERR_CUDA;
        const qil_status s = launch_status();
        if (s != QIL_OK) return s;
    }
    return QIL_OK;
}

}  // namespace qil
