// Shared device/host helpers of the qil kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qil.h"

#define QIL_NUM_SMS_FALLBACK 148

namespace qil {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline qil_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? QIL_OK : QIL_ERR_CUDA;
}

// Number of SMs of the current device (cached per device ordinal).
int num_sms();

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) {
    return __uint_as_float(static_cast<uint32_t>(b) << 16);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Streaming 128-bit load that does not allocate in L1 (weights are read exactly once).
__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Internal launchers (one per translation unit).
qil_status launch_quantize_rtn(const void* w, qil_dtype w_dtype, int N, int K, int G, int symmetric, int bits,
                               uint8_t* codes, void* scales, qil_dtype scale_dtype, void* zeros,
                               int* dev_status, cudaStream_t st);
qil_status launch_pack_w4(const uint8_t* codes, int N, int K, qil_layout layout, uint32_t* packed, cudaStream_t st);
qil_status launch_unpack_w4(const uint32_t* packed, int N, int K, qil_layout layout, int is_signed,
                            uint8_t* codes, cudaStream_t st);
qil_status launch_quantize_act_a4(const void* x, int M, int K, bool use_static, float static_scale,
                                  uint32_t* qx, float* scales, cudaStream_t st);

qil_status launch_quantize_act_a8(const void* x, int M, int K, bool use_static, float static_scale, int8_t* qx,
                                  float* scales, cudaStream_t st);

bool w8a16_stream_supported(int M, int N, int K, int G);
size_t w8a16_workspace();
void w8a16_set_wait_limit(unsigned long long ns);
qil_status launch_w8a16_general(const void* x, const uint8_t* w, const void* s, const void* z, void* y, int M, int N, int K,
                                int G, cudaStream_t st);
qil_status launch_w8a16_stream(const qil_linear_desc* entries, int count, void* ws, size_t ws_bytes, cudaStream_t st);

qil_status launch_w4a16_general(const void* x, const uint32_t* qw, const void* scales, const void* zeros,
                                void* y, int M, int N, int K, int G, cudaStream_t st);
bool w4a16_skinny_supported(int M, int N, int K, int G, qil_layout layout);
size_t w4a16_skinny_workspace(int M, int N, int K, int G);
size_t w4a16_skinny_counter_bytes();  // leading part of that workspace that must be zero before a launch
qil_status launch_w4a16_skinny(const void* x, const uint32_t* qw, const void* scales, const void* zeros,
                               void* y, int M, int N, int K, int G, qil_layout layout, void* ws,
                               size_t ws_bytes, cudaStream_t st);

bool w4a16_prefill_supported(int M, int N, int K, int G, qil_layout layout);
size_t w4a16_prefill_workspace(int M, int N, int K, int G);  // tile counters + the fp32 parts of tiles that CTAs share
qil_status launch_w4a16_prefill(const void* x, const void* qw, const void* scales, const void* zeros, void* y, int M, int N,
                                int K, int G, int bits, int* status, void* scratch, size_t scratch_bytes, cudaStream_t st, int swiglu = 0);
// low-rank side path y += scale * (x . A^T) . B^T, rank <= 32 (lora_side.cu)
size_t lora_side_workspace(int M);
bool lora_side_supported(int M, int N, int K, int r);
qil_status launch_lora_side_add(const void* x, const void* a, const void* b, void* y, int M, int N, int K, int r, float scale,
                                void* ws, cudaStream_t st);
// y[m][i] = silu(t[m][2 i]) * t[m][2 i + 1] for a linear's output t[M][N] (the shapes the GEMM above does not take)
qil_status launch_swiglu_rows(const void* t, void* y, int M, int N, cudaStream_t st);

bool w4a16_tc_supported(int M, int N, int K, int G);
size_t w4a16_tc_weight_bytes(int N, int K);
size_t w4a16_tc_workspace();
qil_status launch_pack_stream128_w4(const uint8_t* codes, const void* scales, const void* zeros, int N, int K, int G,
                                    void* out, cudaStream_t st);
qil_status launch_w4a16_tc(const qil_linear_desc* entries, int count, void* ws, size_t ws_bytes, cudaStream_t st);
void w4a16_tc_set_wait_limit(unsigned long long ns);  // 0 restores the default

size_t w4a4_workspace(int M, int N, int K);
qil_status launch_w4a4(const void* qx, const float* sx, const void* qw, const float* sw, void* y, int32_t* acc_out, int M,
                       int N, int K, int bits, void* ws, size_t ws_bytes, cudaStream_t st, uint32_t* qy = nullptr,
                       float out_scale = 1.f, int relu = 0, int conv_C = 0, int conv_H = 0, int conv_W = 0, float x_scale = 1.f);

bool igemm_list_supported(const qil_igemm_desc* d, int count);
qil_status launch_igemm_list(const qil_igemm_desc* d, int count, void* ws, size_t ws_bytes, cudaStream_t st);

qil_status launch_ref_gemv_bf16(const void* x, const void* w, void* y, int N, int K, cudaStream_t st);
qil_status launch_probe_mma(bool i8, int iters, int commit_every, double* ops_out, int* status, cudaStream_t st);
qil_status launch_probe_hbm_read(const void* buf, size_t bytes, unsigned int* sink, cudaStream_t st);

}  // namespace qil
