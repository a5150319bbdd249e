/*
 * Plain-C oracle of the quantised linear layer (test infrastructure only; the
 * product library never links or calls this file).
 *
 * It restates, with explicit loops, the same specification as the NumPy oracle:
 * the round-to-nearest uniform quantiser the paper names in Sec. 2.1, applied
 * group-wise to weights (4-bit weight-only linears of the OpenVLA decode path,
 * Sec. 5.4 / App. A.4.2) and row-wise to weights and activations of the W4A4
 * path (Sec. 5.1, App. A.1.2), followed by the dequantise-then-matmul in fp64
 * and the integer matmul in int64.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC.
 * Every fp32 step is a single IEEE operation (no fused multiply-add, no
 * reciprocal), rounding is round-half-to-even (rintf under the default mode).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- 16-bit float formats, by their published bit layouts ---- */

static float qo_bf16_to_f32(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* binary16 -> binary32, exact */
static float qo_f16_to_f32(uint16_t h) {
    uint32_t sign = ((uint32_t)h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1Fu;
    uint32_t man = h & 0x3FFu;
    uint32_t u;
    if (exp == 0) {
        if (man == 0) {
            u = sign;
        } else { /* subnormal: value = man * 2^-24 */
            float f = (float)man * 5.9604644775390625e-08f;
            memcpy(&u, &f, 4);
            u |= sign;
        }
    } else if (exp == 31) {
        u = sign | 0x7F800000u | (man << 13);
    } else {
        u = sign | ((exp + 112u) << 23) | (man << 13);
    }
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* binary32 -> binary16, round-to-nearest-even, with subnormals and overflow to inf */
static uint16_t qo_f32_to_f16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t absu = u & 0x7FFFFFFFu;
    if (absu >= 0x7F800000u) { /* inf / nan */
        return (uint16_t)(sign | 0x7C00u | ((absu > 0x7F800000u) ? 0x200u : 0u));
    }
    int32_t e = (int32_t)(absu >> 23) - 127; /* unbiased */
    uint32_t m = (absu & 0x7FFFFFu) | 0x800000u; /* 24-bit significand */
    if (absu < 0x00800000u) return sign;      /* fp32 subnormal: far below half's smallest */
    if (e > 15) return (uint16_t)(sign | 0x7C00u);
    int shift;
    uint32_t base;
    if (e >= -14) { /* normal half: keep 11 significant bits */
        shift = 13;
        base = ((uint32_t)(e + 15)) << 10;
        m &= 0x7FFFFFu; /* drop the hidden bit; it is implied by the exponent */
    } else {       /* subnormal half: value = q * 2^-24, q = m * 2^(e-23+24) */
        shift = 13 + (-14 - e);
        base = 0;
        if (shift > 24) return sign; /* below half of the smallest subnormal */
    }
    uint32_t q = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (q & 1u))) q += 1u;
    /* a carry out of the mantissa correctly bumps the exponent (and reaches inf at the top) */
    return (uint16_t)(sign | (uint16_t)(base + q));
}

static float qo_clampf(float v, float lo, float hi) { return v < lo ? lo : (v > hi ? hi : v); }

/* ---- asymmetric uint4 group quantiser ---- */
/* returns 0, or 1 when a scale overflows fp16 */
int qo_quantize_rtn_w4_asym(const float* w, int N, int K, int G,
                            uint8_t* codes, uint16_t* scales, uint16_t* zeros) {
    int ng = K / G;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < ng; ++g) {
            const float* p = w + (size_t)n * K + (size_t)g * G;
            float lo = 0.0f, hi = 0.0f;
            for (int k = 0; k < G; ++k) {
                if (p[k] < lo) lo = p[k];
                if (p[k] > hi) hi = p[k];
            }
            float r = hi - lo;
            float s32 = r / 15.0f;
            uint16_t s16 = qo_f32_to_f16(s32);
            if ((s16 & 0x7FFFu) == 0x7C00u) bad |= 1;
            if ((s16 & 0x7FFFu) == 0) s16 = 0x3C00u; /* 1.0 */
            float s = qo_f16_to_f32(s16);
            float z = qo_clampf(rintf(-lo / s), 0.0f, 15.0f);
            for (int k = 0; k < G; ++k) {
                float q = qo_clampf(rintf(p[k] / s) + z, 0.0f, 15.0f);
                codes[(size_t)n * K + (size_t)g * G + k] = (uint8_t)q;
            }
            scales[(size_t)n * ng + g] = s16;
            zeros[(size_t)n * ng + g] = qo_f32_to_f16((float)(int)z); /* integer, never -0 */
        }
    }
    return bad;
}

/* ---- symmetric int4 quantiser ---- */
/* scales: float* when scale_f16 == 0, uint16_t* (fp16 bits) otherwise */
int qo_quantize_sym4(const float* v, int R, int K, int G, int scale_f16,
                     const float* static_scale, int8_t* codes, void* scales) {
    int ng = K / G;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int r = 0; r < R; ++r) {
        for (int g = 0; g < ng; ++g) {
            const float* p = v + (size_t)r * K + (size_t)g * G;
            float s;
            if (static_scale) {
                s = *static_scale;
            } else {
                float a = 0.0f;
                for (int k = 0; k < G; ++k) {
                    float t = fabsf(p[k]);
                    if (t > a) a = t;
                }
                s = a / 7.0f;
                if (a == 0.0f) s = 1.0f;
            }
            if (scale_f16) {
                uint16_t s16 = qo_f32_to_f16(s);
                if ((s16 & 0x7FFFu) == 0x7C00u) bad |= 1;
                if ((s16 & 0x7FFFu) == 0) s16 = 0x3C00u;
                s = qo_f16_to_f32(s16);
                ((uint16_t*)scales)[(size_t)r * ng + g] = s16;
            } else {
                ((float*)scales)[(size_t)r * ng + g] = s;
            }
            for (int k = 0; k < G; ++k) {
                float q = qo_clampf(rintf(p[k] / s), -8.0f, 7.0f);
                codes[(size_t)r * K + (size_t)g * G + k] = (int8_t)q;
            }
        }
    }
    return bad;
}

/* ---- the same two quantisers on a grid of 2^bits levels (bits = 4 or 8): the 8-bit deployment
 * points of the paper (INT8 weight-only OpenVLA, W8A8 CILRS; Sec. 5.4) ---- */
int qo_quantize_rtn_asym(const float* w, int N, int K, int G, int bits,
                         uint8_t* codes, uint16_t* scales, uint16_t* zeros) {
    int ng = K / G;
    int bad = 0;
    const float top = (float)((1 << bits) - 1);
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < ng; ++g) {
            const float* p = w + (size_t)n * K + (size_t)g * G;
            float lo = 0.0f, hi = 0.0f;
            for (int k = 0; k < G; ++k) {
                if (p[k] < lo) lo = p[k];
                if (p[k] > hi) hi = p[k];
            }
            float r = hi - lo;
            float s32 = r / top;
            uint16_t s16 = qo_f32_to_f16(s32);
            if ((s16 & 0x7FFFu) == 0x7C00u) bad |= 1;
            if ((s16 & 0x7FFFu) == 0) s16 = 0x3C00u;
            float s = qo_f16_to_f32(s16);
            float z = qo_clampf(rintf(-lo / s), 0.0f, top);
            for (int k = 0; k < G; ++k) {
                float q = qo_clampf(rintf(p[k] / s) + z, 0.0f, top);
                codes[(size_t)n * K + (size_t)g * G + k] = (uint8_t)q;
            }
            scales[(size_t)n * ng + g] = s16;
            zeros[(size_t)n * ng + g] = qo_f32_to_f16((float)(int)z);
        }
    }
    return bad;
}

void qo_quantize_sym(const float* v, int R, int K, int G, int bits, const float* static_scale,
                     int8_t* codes, float* scales) {
    int ng = K / G;
    const float qmax = (float)((1 << (bits - 1)) - 1), qmin = -(float)(1 << (bits - 1));
#pragma omp parallel for schedule(static)
    for (int r = 0; r < R; ++r) {
        for (int g = 0; g < ng; ++g) {
            const float* p = v + (size_t)r * K + (size_t)g * G;
            float s;
            if (static_scale) {
                s = *static_scale;
            } else {
                float a = 0.0f;
                for (int k = 0; k < G; ++k) {
                    float t = fabsf(p[k]);
                    if (t > a) a = t;
                }
                s = a / qmax;
                if (a == 0.0f) s = 1.0f;
            }
            scales[(size_t)r * ng + g] = s;
            for (int k = 0; k < G; ++k) {
                float q = qo_clampf(rintf(p[k] / s), qmin, qmax);
                codes[(size_t)r * K + (size_t)g * G + k] = (int8_t)q;
            }
        }
    }
}

/* ---- packing: element k of a row -> word k/8, bits [4(k%8), 4(k%8)+3] ---- */
void qo_pack_w4(const uint8_t* codes, int R, int K, uint32_t* packed) {
    int W = K / 8;
    for (int r = 0; r < R; ++r)
        for (int i = 0; i < W; ++i) {
            uint32_t word = 0;
            for (int j = 0; j < 8; ++j)
                word |= ((uint32_t)(codes[(size_t)r * K + 8 * i + j] & 0xF)) << (4 * j);
            packed[(size_t)r * W + i] = word;
        }
}

void qo_unpack_w4(const uint32_t* packed, int R, int K, int is_signed, uint8_t* codes) {
    int W = K / 8;
    for (int r = 0; r < R; ++r)
        for (int i = 0; i < W; ++i)
            for (int j = 0; j < 8; ++j) {
                int v = (int)((packed[(size_t)r * W + i] >> (4 * j)) & 0xFu);
                if (is_signed && v >= 8) v -= 16;
                codes[(size_t)r * K + 8 * i + j] = (uint8_t)(int8_t)v;
            }
}

/* 16-row x 128-column tiles, tiles of one row-tile consecutive, rows inside a tile consecutive */
void qo_to_tile16(const uint32_t* canon, int N, int K, uint32_t* out) {
    int W = K / 8, kt = W / 16;
    for (int n = 0; n < N; ++n)
        for (int i = 0; i < W; ++i)
            out[((size_t)(n / 16) * kt + i / 16) * 256 + (size_t)(n % 16) * 16 + i % 16] =
                canon[(size_t)n * W + i];
}

/* ---- W4A16: y = x . dequant(W)^T in fp64, natural k order ---- */
void qo_linear_w4a16(const uint16_t* x_bf16, const uint8_t* codes, const uint16_t* scales,
                     const uint16_t* zeros, int M, int N, int K, int G, double* y) {
    int ng = K / G;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                double s = (double)qo_f16_to_f32(scales[(size_t)n * ng + k / G]);
                double z = (double)qo_f16_to_f32(zeros[(size_t)n * ng + k / G]);
                double q = (double)codes[(size_t)n * K + k];
                double xv = (double)qo_bf16_to_f32(x_bf16[(size_t)m * K + k]);
                acc += xv * ((q - z) * s);
            }
            y[(size_t)m * N + n] = acc;
        }
    }
}

/* ---- W4A4: int64 accumulate, fp64 rescale ---- */
void qo_linear_w4a4(const int8_t* qx, const float* sx, const int8_t* qw, const float* sw,
                    int M, int N, int K, int64_t* acc_out, double* y) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            int64_t acc = 0;
            for (int k = 0; k < K; ++k)
                acc += (int64_t)qx[(size_t)m * K + k] * (int64_t)qw[(size_t)n * K + k];
            if (acc_out) acc_out[(size_t)m * N + n] = acc;
            if (y) y[(size_t)m * N + n] = (double)acc * (double)sx[m] * (double)sw[n];
        }
    }
}

/* ---- W4A4 linear followed by the next layer's static-scale int4 quantiser, on the fp32 output ---- */
void qo_linear_w4a4_requant(const int8_t* qx, const float* sx, const int8_t* qw, const float* sw,
                            int M, int N, int K, float out_scale, int relu, int8_t* q_out) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            int64_t acc = 0;
            for (int k = 0; k < K; ++k)
                acc += (int64_t)qx[(size_t)m * K + k] * (int64_t)qw[(size_t)n * K + k];
            float scale = sx[m] * sw[n];
            float y = (float)acc * scale;
            if (relu && y < 0.0f) y = 0.0f;
            float q = qo_clampf(rintf(y / out_scale), -8.0f, 7.0f);
            q_out[(size_t)m * N + n] = (int8_t)q;
        }
    }
}

int qo_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
