// Round-to-nearest 4-bit quantisers and the nibble packer (paper Sec. 2.1).
//
// The fp32 operation order is the one documented in qil.h; every result equals that of an
// IEEE division (__fdiv_rn) followed by rintf (ties to even), so the codes are reproducible
// bit for bit.  No step is contracted into a fused multiply-add.  The activation quantiser
// has one fast path: it multiplies by a reciprocal and keeps that result only when it is
// provably the same integer (the product is far enough from a rounding boundary), and falls
// back to the exact division otherwise (rint_div below).
#include "qil_common.cuh"

namespace qil {

namespace {

template <typename T>
__device__ __forceinline__ float load_f32(const T* p, size_t i);
template <>
__device__ __forceinline__ float load_f32<float>(const float* p, size_t i) { return p[i]; }
template <>
__device__ __forceinline__ float load_f32<__nv_bfloat16>(const __nv_bfloat16* p, size_t i) {
    return __bfloat162float(p[i]);
}
template <>
__device__ __forceinline__ float load_f32<__half>(const __half* p, size_t i) { return __half2float(p[i]); }

__device__ __forceinline__ float clampf(float v, float lo, float hi) { return fminf(fmaxf(v, lo), hi); }

// fp16 scale with the two special cases: 0 -> 1, inf -> flag.
__device__ __forceinline__ float round_scale_f16(float s32, __half* out, int* status) {
    __half h = __float2half_rn(s32);
    unsigned short bits = __half_as_ushort(h) & 0x7FFFu;
    if (bits == 0x7C00u && status) atomicOr(status, (int)QIL_ERR_RANGE);
    if (bits == 0) h = __ushort_as_half(0x3C00u);
    *out = h;
    return __half2float(h);
}

// One warp per (row, group).  Asymmetric uint4 with integer zero point.
template <typename T>
__global__ void __launch_bounds__(256) quantize_asym_kernel(const T* __restrict__ w, int N, int K, int G,
                                                            uint8_t* __restrict__ codes,
                                                            __half* __restrict__ scales,
                                                            __half* __restrict__ zeros, int* status, float top) {
    // top = 15 (4-bit) or 255 (8-bit): the highest level of the grid
    const int lane = threadIdx.x & 31;
    const int ng = K / G;
    const long long total = (long long)N * ng;
    const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long grp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); grp < total; grp += warps) {
        const size_t base = (size_t)(grp / ng) * K + (size_t)(grp % ng) * G;
        float lo = 0.0f, hi = 0.0f;
        for (int k = lane; k < G; k += 32) {
            float v = load_f32<T>(w, base + k);
            lo = fminf(lo, v);
            hi = fmaxf(hi, v);
        }
        lo = warp_min(lo);
        hi = warp_max(hi);
        const float r = __fsub_rn(hi, lo);
        const float s32 = __fdiv_rn(r, top);
        __half s16;
        const float s = round_scale_f16(s32, &s16, lane == 0 ? status : nullptr);
        const float z = clampf(rintf(__fdiv_rn(-lo, s)), 0.0f, top);
        for (int k = lane; k < G; k += 32) {
            float v = load_f32<T>(w, base + k);
            float q = clampf(__fadd_rn(rintf(__fdiv_rn(v, s)), z), 0.0f, top);
            codes[base + k] = (uint8_t)(int)q;
        }
        if (lane == 0) {
            scales[grp] = s16;
            zeros[grp] = __int2half_rn((int)z);
        }
    }
}

// One warp per (row, group).  Symmetric: divisor qmax = 7 (4-bit) or 127 (8-bit), clamp to [-qmax - 1, qmax].
template <typename T, bool kScaleF16>
__global__ void __launch_bounds__(256) quantize_sym_kernel(const T* __restrict__ v, int R, int K, int G,
                                                           int8_t* __restrict__ codes, void* __restrict__ scales,
                                                           int* status, float qmax) {
    const int lane = threadIdx.x & 31;
    const int ng = K / G;
    const long long total = (long long)R * ng;
    const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long grp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); grp < total; grp += warps) {
        const size_t base = (size_t)(grp / ng) * K + (size_t)(grp % ng) * G;
        float a = 0.0f;
        for (int k = lane; k < G; k += 32) a = fmaxf(a, fabsf(load_f32<T>(v, base + k)));
        a = warp_max(a);
        float s = __fdiv_rn(a, qmax);
        if (a == 0.0f) s = 1.0f;
        if (kScaleF16) {
            __half s16;
            s = round_scale_f16(s, &s16, lane == 0 ? status : nullptr);
            if (lane == 0) reinterpret_cast<__half*>(scales)[grp] = s16;
        } else if (lane == 0) {
            reinterpret_cast<float*>(scales)[grp] = s;
        }
        for (int k = lane; k < G; k += 32) {
            float q = clampf(rintf(__fdiv_rn(load_f32<T>(v, base + k), s)), -qmax - 1.0f, qmax);
            codes[base + k] = (int8_t)(int)q;
        }
    }
}

// rint(f / s) with the IEEE division of the specification, without paying for a division per element: the product
// with the reciprocal is within a few ulp of the quotient, so unless it lies that close to a rounding boundary
// (k + 0.5) it rounds to the same integer; the rare close calls (and anything not finite) take the true division.
__device__ __forceinline__ float rint_div(float f, float s, float inv_s) {
    const float r = f * inv_s;
    const float dist = fabsf(fabsf(r - rintf(r)) - 0.5f);  // distance of r from the nearest k + 0.5
    if (dist > 1e-4f * fmaxf(fabsf(r), 1.0f) && fabsf(r) < 1e6f) return rintf(r);
    return rintf(__fdiv_rn(f, s));
}

// Per-token symmetric int4 of bf16 activations, fused with packing.  One warp per row.
// Each lane owns whole 32-bit output words (8 consecutive k).
// Rows of at most 256 kPer elements: a warp keeps its row in registers between the maximum and the rounding, and all
// of the row's loads are in flight at once (same arithmetic as the general kernel below, hence the same codes).
template <int kPer>
__global__ void __launch_bounds__(256) quantize_act_cached_kernel(const __nv_bfloat16* __restrict__ x, int M, int K,
                                                                  bool use_static, float static_scale,
                                                                  uint32_t* __restrict__ qx, float* __restrict__ scales) {
    const int lane = threadIdx.x & 31;
    const int words = K >> 3;
    const int warps = gridDim.x * (blockDim.x >> 5);
    for (int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); m < M; m += warps) {
        const uint4* row = reinterpret_cast<const uint4*>(x + (size_t)m * K);
        uint4 buf[kPer];
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const int i = lane + 32 * j;
            buf[j] = i < words ? __ldg(row + i) : make_uint4(0, 0, 0, 0);
        }
        float s;
        if (use_static) {
            s = static_scale;
        } else {
            float a = 0.0f;
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                const uint32_t u[4] = {buf[j].x, buf[j].y, buf[j].z, buf[j].w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    a = fmaxf(a, fabsf(__uint_as_float(u[c] << 16)));
                    a = fmaxf(a, fabsf(__uint_as_float(u[c] & 0xFFFF0000u)));
                }
            }
            a = warp_max(a);
            s = __fdiv_rn(a, 7.0f);
            if (a == 0.0f) s = 1.0f;
        }
        if (lane == 0) scales[m] = s;
        const float inv_s = __frcp_rn(s);
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const int i = lane + 32 * j;
            if (i >= words) continue;
            const uint32_t u[4] = {buf[j].x, buf[j].y, buf[j].z, buf[j].w};
            uint32_t word = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float f0 = __uint_as_float(u[c] << 16);
                const float f1 = __uint_as_float(u[c] & 0xFFFF0000u);
                const int q0 = (int)clampf(rint_div(f0, s, inv_s), -8.0f, 7.0f);
                const int q1 = (int)clampf(rint_div(f1, s, inv_s), -8.0f, 7.0f);
                word |= (uint32_t)(q0 & 0xF) << (8 * c);
                word |= (uint32_t)(q1 & 0xF) << (8 * c + 4);
            }
            qx[(size_t)m * words + i] = word;
        }
    }
}

__global__ void __launch_bounds__(256) quantize_act_kernel(const __nv_bfloat16* __restrict__ x, int M, int K,
                                                           bool use_static, float static_scale,
                                                           uint32_t* __restrict__ qx, float* __restrict__ scales) {
    const int lane = threadIdx.x & 31;
    const int words = K >> 3;
    const int warps = gridDim.x * (blockDim.x >> 5);
    for (int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); m < M; m += warps) {
        const uint4* row = reinterpret_cast<const uint4*>(x + (size_t)m * K);
        float s;
        if (use_static) {
            s = static_scale;
        } else {
            float a = 0.0f;
            for (int i = lane; i < words; i += 32) {
                uint4 v = row[i];
                const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    a = fmaxf(a, fabsf(__uint_as_float(u[j] << 16)));
                    a = fmaxf(a, fabsf(__uint_as_float(u[j] & 0xFFFF0000u)));
                }
            }
            a = warp_max(a);
            s = __fdiv_rn(a, 7.0f);
            if (a == 0.0f) s = 1.0f;
        }
        if (lane == 0) scales[m] = s;
        const float inv_s = __frcp_rn(s);
        for (int i = lane; i < words; i += 32) {
            uint4 v = row[i];
            const uint32_t u[4] = {v.x, v.y, v.z, v.w};
            uint32_t word = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float f0 = __uint_as_float(u[j] << 16);
                float f1 = __uint_as_float(u[j] & 0xFFFF0000u);
                int q0 = (int)clampf(rint_div(f0, s, inv_s), -8.0f, 7.0f);
                int q1 = (int)clampf(rint_div(f1, s, inv_s), -8.0f, 7.0f);
                word |= (uint32_t)(q0 & 0xF) << (8 * j);
                word |= (uint32_t)(q1 & 0xF) << (8 * j + 4);
            }
            qx[(size_t)m * words + i] = word;
        }
    }
}

__device__ __forceinline__ size_t packed_index(int n, int i, int words, qil_layout layout) {
    if (layout == QIL_LAYOUT_TILE16)
        return ((size_t)(n >> 4) * (words >> 4) + (i >> 4)) * 256 + (size_t)(n & 15) * 16 + (i & 15);
    return (size_t)n * words + i;
}

__global__ void __launch_bounds__(256) pack_kernel(const uint8_t* __restrict__ codes, int N, int K,
                                                   qil_layout layout, uint32_t* __restrict__ packed) {
    const int words = K >> 3;
    const long long total = (long long)N * words;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const int n = (int)(t / words), i = (int)(t % words);
        const uint2 c = *reinterpret_cast<const uint2*>(codes + (size_t)n * K + (size_t)i * 8);
        uint32_t word = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            word |= ((c.x >> (8 * j)) & 0xFu) << (4 * j);
            word |= ((c.y >> (8 * j)) & 0xFu) << (4 * (j + 4));
        }
        packed[packed_index(n, i, words, layout)] = word;
    }
}

__global__ void __launch_bounds__(256) unpack_kernel(const uint32_t* __restrict__ packed, int N, int K,
                                                     qil_layout layout, int is_signed,
                                                     uint8_t* __restrict__ codes) {
    const int words = K >> 3;
    const long long total = (long long)N * words;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const int n = (int)(t / words), i = (int)(t % words);
        const uint32_t word = packed[packed_index(n, i, words, layout)];
        uint2 c = make_uint2(0u, 0u);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t nib = (word >> (4 * j)) & 0xFu;
            if (is_signed && nib >= 8u) nib |= 0xF0u;
            if (j < 4) c.x |= nib << (8 * j);
            else c.y |= nib << (8 * (j - 4));
        }
        *reinterpret_cast<uint2*>(codes + (size_t)n * K + (size_t)i * 8) = c;
    }
}

// Per-token symmetric int8 of bf16 activations (divisor 127), one code per byte.  One warp per row; the same
// division rule as the 4-bit quantiser (rint_div).
__global__ void __launch_bounds__(256) quantize_act_a8_kernel(const __nv_bfloat16* __restrict__ x, int M, int K,
                                                              bool use_static, float static_scale,
                                                              int8_t* __restrict__ qx, float* __restrict__ scales) {
    const int lane = threadIdx.x & 31;
    const int words = K >> 3;  // 8 elements = one 16-byte load, one 8-byte store
    const int warps = gridDim.x * (blockDim.x >> 5);
    for (int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); m < M; m += warps) {
        const uint4* row = reinterpret_cast<const uint4*>(x + (size_t)m * K);
        float s;
        if (use_static) {
            s = static_scale;
        } else {
            uint32_t amax = 0;  // bf16 magnitudes order like unsigned integers
            for (int i = lane; i < words; i += 32) {
                const uint4 v = __ldg(row + i);
                const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) amax = max(amax, max((u[j] << 16) & 0x7FFFFFFFu, u[j] & 0x7FFF0000u));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            const float a = __uint_as_float(amax);
            s = __fdiv_rn(a, 127.0f);
            if (a == 0.0f) s = 1.0f;
        }
        const float inv_s = __frcp_rn(s);
        for (int i = lane; i < words; i += 32) {
            const uint4 v = __ldg(row + i);
            const uint32_t u[4] = {v.x, v.y, v.z, v.w};
            uint32_t out[2] = {0u, 0u};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int q0 = (int)clampf(rint_div(__uint_as_float(u[j] << 16), s, inv_s), -128.0f, 127.0f);
                const int q1 = (int)clampf(rint_div(__uint_as_float(u[j] & 0xFFFF0000u), s, inv_s), -128.0f, 127.0f);
                out[j >> 1] |= (((uint32_t)q0 & 0xFFu) | (((uint32_t)q1 & 0xFFu) << 8)) << (16 * (j & 1));
            }
            *reinterpret_cast<uint2*>(qx + (size_t)m * K + (size_t)i * 8) = make_uint2(out[0], out[1]);
        }
        if (lane == 0) scales[m] = s;
    }
}

inline int grid_for(long long work_items, int per_block) {
    long long blocks = (work_items + per_block - 1) / per_block;
    long long cap = (long long)num_sms() * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

}  // namespace

qil_status launch_quantize_rtn(const void* w, qil_dtype w_dtype, int N, int K, int G, int symmetric, int bits,
                               uint8_t* codes, void* scales, qil_dtype scale_dtype, void* zeros,
                               int* dev_status, cudaStream_t st) {
    const float top = bits == 8 ? 255.0f : 15.0f, qmax = bits == 8 ? 127.0f : 7.0f;
    const long long groups = (long long)N * (K / G);
    const int grid = grid_for(groups, 8);
#define QIL_ASYM(T)                                                                                  \
    quantize_asym_kernel<T><<<grid, 256, 0, st>>>(reinterpret_cast<const T*>(w), N, K, G, codes,     \
                                                  reinterpret_cast<__half*>(scales),                 \
                                                  reinterpret_cast<__half*>(zeros), dev_status, top)
#define QIL_SYM(T, F16)                                                                              \
    quantize_sym_kernel<T, F16><<<grid, 256, 0, st>>>(reinterpret_cast<const T*>(w), N, K, G,        \
                                                      reinterpret_cast<int8_t*>(codes), scales, dev_status, qmax)
    if (!symmetric) {
        if (w_dtype == QIL_F32) QIL_ASYM(float);
        else if (w_dtype == QIL_BF16) QIL_ASYM(__nv_bfloat16);
        else QIL_ASYM(__half);
    } else {
        const bool f16 = scale_dtype == QIL_F16;
        if (w_dtype == QIL_F32) { if (f16) QIL_SYM(float, true); else QIL_SYM(float, false); }
        else if (w_dtype == QIL_BF16) { if (f16) QIL_SYM(__nv_bfloat16, true); else QIL_SYM(__nv_bfloat16, false); }
        else { if (f16) QIL_SYM(__half, true); else QIL_SYM(__half, false); }
    }
#undef QIL_ASYM
#undef QIL_SYM
    return launch_status();
}

qil_status launch_pack_w4(const uint8_t* codes, int N, int K, qil_layout layout, uint32_t* packed, cudaStream_t st) {
    const long long words = (long long)N * (K / 8);
    pack_kernel<<<grid_for(words, 256), 256, 0, st>>>(codes, N, K, layout, packed);
    return launch_status();
}

qil_status launch_unpack_w4(const uint32_t* packed, int N, int K, qil_layout layout, int is_signed,
                            uint8_t* codes, cudaStream_t st) {
    const long long words = (long long)N * (K / 8);
    unpack_kernel<<<grid_for(words, 256), 256, 0, st>>>(packed, N, K, layout, is_signed, codes);
    return launch_status();
}

qil_status launch_quantize_act_a4(const void* x, int M, int K, bool use_static, float static_scale,
                                  uint32_t* qx, float* scales, cudaStream_t st) {
    const int words = K >> 3;
#define QIL_ACT_CACHED(P)                                                                                           \
    if (words <= 32 * (P)) {                                                                                        \
        quantize_act_cached_kernel<P><<<grid_for(M, 8), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(x), M, \
                                                                      K, use_static, static_scale, qx, scales);      \
        return launch_status();                                                                                     \
    }
    QIL_ACT_CACHED(3)
    QIL_ACT_CACHED(5)
    QIL_ACT_CACHED(9)
    QIL_ACT_CACHED(18)
#undef QIL_ACT_CACHED
    quantize_act_kernel<<<grid_for(M, 8), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(x), M, K,
                                                        use_static, static_scale, qx, scales);
    return launch_status();
}

qil_status launch_quantize_act_a8(const void* x, int M, int K, bool use_static, float static_scale, int8_t* qx,
                                  float* scales, cudaStream_t st) {
    quantize_act_a8_kernel<<<grid_for(M, 8), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(x), M, K, use_static,
                                                           static_scale, qx, scales);
    return launch_status();
}

}  // namespace qil
