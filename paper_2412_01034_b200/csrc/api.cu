// C ABI of the library: argument validation on the host, then one launcher each.
#include <atomic>

#include "qil_common.cuh"

namespace qil {

int num_sms() {
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cached[kMaxDevices];
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_NUM_SMS_FALLBACK;  // (no device: only sizes are asked for)
    }
    const bool slot = dev >= 0 && dev < kMaxDevices;
    if (slot) {
        const int v = cached[dev].load(std::memory_order_relaxed);
        if (v > 0) return v;
    }
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
        (void)cudaGetLastError();
        return QIL_NUM_SMS_FALLBACK;  // not cached: a later call may succeed
    }
    if (slot) cached[dev].store(sms, std::memory_order_relaxed);
    return sms;
}

// The workspace of qil_linear_w4a16 has two parts that never overlap: the streaming list kernel's header and
// hand-over slots first, the split-K scratch of the skinny kernel after them.
size_t w4a16_skinny_ws_offset() { return (w4a16_tc_workspace() + 255) & ~(size_t)255; }

}  // namespace qil

using namespace qil;

namespace {
inline cudaStream_t S(qil_stream_t s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool dtype_ok(int d) { return d == QIL_F32 || d == QIL_BF16 || d == QIL_F16; }
inline bool layout_ok(int l) { return l == QIL_LAYOUT_CANONICAL || l == QIL_LAYOUT_TILE16 || l == QIL_LAYOUT_STREAM128; }
inline bool pack_layout_ok(int l) { return l == QIL_LAYOUT_CANONICAL || l == QIL_LAYOUT_TILE16; }
}  // namespace

extern "C" {

const char* qil_status_string(qil_status s) {
    switch (s) {
        case QIL_OK: return "ok";
        case QIL_ERR_NULL: return "null pointer";
        case QIL_ERR_SHAPE: return "bad shape";
        case QIL_ERR_ALIGN: return "pointer not 16-byte aligned";
        case QIL_ERR_UNSUPPORTED: return "unsupported argument";
        case QIL_ERR_WORKSPACE: return "workspace missing or too small";
        case QIL_ERR_CUDA: return "CUDA error";
        case QIL_ERR_TIMEOUT: return "device-side wait timed out";
        case QIL_ERR_RANGE: return "scale does not fit fp16";
    }
    return "unknown status";
}

int qil_version(void) { return 100; }

qil_status qil_set_wait_limit_ns(unsigned long long ns) {
    w4a16_tc_set_wait_limit(ns);
    w8a16_set_wait_limit(ns);
    return QIL_OK;
}

qil_status qil_device_status(const int* dev_status, int* out, qil_stream_t stream) {
    if (!dev_status || !out) return QIL_ERR_NULL;
    if (cudaMemcpyAsync(out, dev_status, sizeof(int), cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess ||
        cudaStreamSynchronize(S(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    return QIL_OK;
}

qil_status qil_quantize_rtn_w4(const void* w, qil_dtype w_dtype, int N, int K, int group_size, int symmetric,
                               uint8_t* codes, void* scales, qil_dtype scale_dtype, void* zeros,
                               int* dev_status, qil_stream_t stream) {
    if (!w || !codes || !scales) return QIL_ERR_NULL;
    if (!symmetric && !zeros) return QIL_ERR_NULL;
    if (N <= 0 || K <= 0 || group_size <= 0 || K % group_size != 0) return QIL_ERR_SHAPE;
    if (!dtype_ok(w_dtype) || !dtype_ok(scale_dtype)) return QIL_ERR_UNSUPPORTED;
    if (!symmetric && scale_dtype != QIL_F16) return QIL_ERR_UNSUPPORTED;
    if (symmetric && scale_dtype == QIL_BF16) return QIL_ERR_UNSUPPORTED;
    if (!aligned16(w) || !aligned16(codes) || !aligned16(scales) || (zeros && !aligned16(zeros))) return QIL_ERR_ALIGN;
    return launch_quantize_rtn(w, w_dtype, N, K, group_size, symmetric, 4, codes, scales, scale_dtype, zeros,
                               dev_status, S(stream));
}

qil_status qil_quantize_rtn_w8(const void* w, qil_dtype w_dtype, int N, int K, int group_size, int symmetric,
                               uint8_t* codes, void* scales, qil_dtype scale_dtype, void* zeros,
                               int* dev_status, qil_stream_t stream) {
    if (!w || !codes || !scales) return QIL_ERR_NULL;
    if (!symmetric && !zeros) return QIL_ERR_NULL;
    if (N <= 0 || K <= 0 || group_size <= 0 || K % group_size != 0) return QIL_ERR_SHAPE;
    if (!dtype_ok(w_dtype) || !dtype_ok(scale_dtype)) return QIL_ERR_UNSUPPORTED;
    if (!symmetric && scale_dtype != QIL_F16) return QIL_ERR_UNSUPPORTED;
    if (symmetric && scale_dtype == QIL_BF16) return QIL_ERR_UNSUPPORTED;
    if (!aligned16(w) || !aligned16(codes) || !aligned16(scales) || (zeros && !aligned16(zeros))) return QIL_ERR_ALIGN;
    return launch_quantize_rtn(w, w_dtype, N, K, group_size, symmetric, 8, codes, scales, scale_dtype, zeros,
                               dev_status, S(stream));
}

static qil_status check_pack(const void* a, const void* b, int N, int K, qil_layout layout) {
    if (!a || !b) return QIL_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 8 != 0) return QIL_ERR_SHAPE;
    if (!pack_layout_ok(layout)) return QIL_ERR_UNSUPPORTED;
    if (layout == QIL_LAYOUT_TILE16 && (N % 16 != 0 || K % 128 != 0)) return QIL_ERR_SHAPE;
    if (!aligned16(a) || !aligned16(b)) return QIL_ERR_ALIGN;
    return QIL_OK;
}

size_t qil_stream128_w4_bytes(int N, int K) {
    if (N <= 0 || K <= 0 || K % 128 != 0) return 0;
    return w4a16_tc_weight_bytes(N, K);
}

qil_status qil_pack_stream128_w4(const uint8_t* codes, const void* scales, const void* zeros, int N, int K,
                                 int group_size, void* out, qil_stream_t stream) {
    if (!codes || !scales || !zeros || !out) return QIL_ERR_NULL;
    if (N <= 0 || K <= 0 || group_size <= 0 || K % 128 != 0 || group_size % 128 != 0 || K % group_size != 0)
        return QIL_ERR_SHAPE;
    if (!aligned16(codes) || !aligned16(scales) || !aligned16(zeros) || !aligned16(out)) return QIL_ERR_ALIGN;
    return launch_pack_stream128_w4(codes, scales, zeros, N, K, group_size, out, S(stream));
}

qil_status qil_pack_w4(const uint8_t* codes, int N, int K, qil_layout layout, uint32_t* packed, qil_stream_t stream) {
    const qil_status s = check_pack(codes, packed, N, K, layout);
    if (s != QIL_OK) return s;
    return launch_pack_w4(codes, N, K, layout, packed, S(stream));
}

qil_status qil_unpack_w4(const uint32_t* packed, int N, int K, qil_layout layout, int is_signed, uint8_t* codes,
                         qil_stream_t stream) {
    const qil_status s = check_pack(packed, codes, N, K, layout);
    if (s != QIL_OK) return s;
    return launch_unpack_w4(packed, N, K, layout, is_signed, codes, S(stream));
}

static qil_status check_w4a16(const void* x, const void* qw, const void* sc, const void* z, const void* y, int M,
                              int N, int K, int G, qil_layout layout) {
    const bool stream_layout = layout == QIL_LAYOUT_STREAM128;
    if (!x || !qw || !y || (!stream_layout && (!sc || !z))) return QIL_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || G <= 0 || K % 8 != 0 || K % G != 0) return QIL_ERR_SHAPE;
    if (!layout_ok(layout)) return QIL_ERR_UNSUPPORTED;
    if (layout == QIL_LAYOUT_TILE16 && (N % 16 != 0 || K % 128 != 0)) return QIL_ERR_SHAPE;
    if (layout == QIL_LAYOUT_STREAM128 && K % 128 != 0) return QIL_ERR_SHAPE;
    if (stream_layout && G % 128 != 0) return QIL_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(qw) || !aligned16(y)) return QIL_ERR_ALIGN;
    if (!stream_layout && (!aligned16(sc) || !aligned16(z))) return QIL_ERR_ALIGN;
    if (layout == QIL_LAYOUT_STREAM128 && !w4a16_tc_supported(M, N, K, G)) return QIL_ERR_UNSUPPORTED;
    return QIL_OK;
}

size_t qil_linear_w4a16_workspace_size(int M, int N, int K, int group_size) {
    if (M <= 0 || N <= 0 || K <= 0 || group_size <= 0) return 0;
    if (K % 128 != 0 || group_size % 128 != 0) return 0;
    size_t scratch = w4a16_skinny_workspace(M, N, K, group_size);
    if (w4a16_prefill_supported(M, N, K, group_size, QIL_LAYOUT_CANONICAL)) {
        const size_t pf = w4a16_prefill_workspace(M, N, K, group_size);
        if (pf > scratch) scratch = pf;
    }
    return w4a16_skinny_ws_offset() + scratch;  // serves every layout
}

qil_status qil_linear_w4a16(const void* x, const uint32_t* qweight, const void* scales, const void* zeros, void* y,
                            int M, int N, int K, int group_size, qil_layout layout, void* workspace,
                            size_t workspace_bytes, qil_stream_t stream) {
    const qil_status s = check_w4a16(x, qweight, scales, zeros, y, M, N, K, group_size, layout);
    if (s != QIL_OK) return s;
    if (workspace && !aligned16(workspace)) return QIL_ERR_ALIGN;
    if (layout == QIL_LAYOUT_STREAM128) {
        qil_linear_desc d;
        d.x = x; d.qweight = qweight; d.scales = nullptr; d.zeros = nullptr; d.y = y;
        d.M = M; d.N = N; d.K = K; d.group_size = group_size; d.layout = layout; d.flags = 0;
        return launch_w4a16_tc(&d, 1, workspace, workspace_bytes, S(stream));
    }
    if (w4a16_prefill_supported(M, N, K, group_size, layout)) {
        const size_t off = w4a16_skinny_ws_offset();
        const bool have = workspace != nullptr && workspace_bytes > off;
        return launch_w4a16_prefill(x, qweight, scales, zeros, y, M, N, K, group_size, 4,
                                    workspace_bytes >= sizeof(int) ? static_cast<int*>(workspace) : nullptr,
                                    have ? static_cast<char*>(workspace) + off : nullptr, have ? workspace_bytes - off : 0,
                                    S(stream));
    }
    if (w4a16_skinny_supported(M, N, K, group_size, layout)) {
        const size_t off = w4a16_skinny_ws_offset();
        const bool have = workspace != nullptr && workspace_bytes > off;
        return launch_w4a16_skinny(x, qweight, scales, zeros, y, M, N, K, group_size, layout,
                                   have ? static_cast<char*>(workspace) + off : nullptr, have ? workspace_bytes - off : 0,
                                   S(stream));
    }
    if (layout != QIL_LAYOUT_CANONICAL) return QIL_ERR_UNSUPPORTED;
    return launch_w4a16_general(x, qweight, scales, zeros, y, M, N, K, group_size, S(stream));
}

// Bytes of the plain linear's workspace, rounded so that the bf16 scratch of the unfused path can follow it.
static size_t swiglu_tmp_offset(int M, int N, int K, int group_size) {
    return (qil_linear_w4a16_workspace_size(M, N, K, group_size) + 255) / 256 * 256;
}

size_t qil_linear_w4a16_swiglu_workspace_size(int M, int N, int K, int group_size) {
    if (M <= 0 || N <= 0 || K <= 0 || group_size <= 0) return 0;
    size_t bytes = swiglu_tmp_offset(M, N, K, group_size);
    if (!w4a16_prefill_supported(M, N, K, group_size, QIL_LAYOUT_CANONICAL)) bytes += (size_t)M * N * 2;
    return bytes;
}

qil_status qil_linear_w4a16_swiglu(const void* x, const uint32_t* qweight, const void* scales, const void* zeros, void* y,
                                   int M, int N, int K, int group_size, void* workspace, size_t workspace_bytes,
                                   qil_stream_t stream) {
    const qil_status s = check_w4a16(x, qweight, scales, zeros, y, M, N, K, group_size, QIL_LAYOUT_CANONICAL);
    if (s != QIL_OK) return s;
    if (N % 2 != 0) return QIL_ERR_SHAPE;
    if (workspace && !aligned16(workspace)) return QIL_ERR_ALIGN;
    if (w4a16_prefill_supported(M, N, K, group_size, QIL_LAYOUT_CANONICAL)) {
        const size_t off = w4a16_skinny_ws_offset();
        const bool have = workspace != nullptr && workspace_bytes > off;
        return launch_w4a16_prefill(x, qweight, scales, zeros, y, M, N, K, group_size, 4,
                                    workspace_bytes >= sizeof(int) ? static_cast<int*>(workspace) : nullptr,
                                    have ? static_cast<char*>(workspace) + off : nullptr, have ? workspace_bytes - off : 0,
                                    S(stream), 1);
    }
    const size_t off = swiglu_tmp_offset(M, N, K, group_size);
    if (!workspace || workspace_bytes < off + (size_t)M * N * 2) return QIL_ERR_WORKSPACE;
    void* tmp = static_cast<char*>(workspace) + off;
    const qil_status s2 = qil_linear_w4a16(x, qweight, scales, zeros, tmp, M, N, K, group_size, QIL_LAYOUT_CANONICAL, workspace, off, stream);
    if (s2 != QIL_OK) return s2;
    return launch_swiglu_rows(tmp, y, M, N, S(stream));
}

size_t qil_lora_side_workspace_size(int M) { return M > 0 ? lora_side_workspace(M) : 0; }

qil_status qil_lora_side_add(const void* x, const void* a, const void* b, void* y, int M, int N, int K, int rank, float scale,
                             void* workspace, size_t workspace_bytes, qil_stream_t stream) {
    if (!x || !a || !b || !y) return QIL_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || rank <= 0 || K % 2 != 0) return QIL_ERR_SHAPE;
    if (!lora_side_supported(M, N, K, rank)) return QIL_ERR_UNSUPPORTED;   // rank > 32
    if (reinterpret_cast<uintptr_t>(x) % 4 || reinterpret_cast<uintptr_t>(a) % 4 || reinterpret_cast<uintptr_t>(b) % 2 ||
        reinterpret_cast<uintptr_t>(y) % 2)
        return QIL_ERR_ALIGN;
    if (!workspace || workspace_bytes < lora_side_workspace(M)) return QIL_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) % 4) return QIL_ERR_ALIGN;
    return launch_lora_side_add(x, a, b, y, M, N, K, rank, scale, workspace, S(stream));
}

qil_status qil_linear_w4a16_batch(const qil_linear_desc* descs, int count, void* workspace, size_t workspace_bytes,
                                  qil_stream_t stream) {
    if (!descs) return QIL_ERR_NULL;
    if (count <= 0) return QIL_ERR_SHAPE;
    if (workspace && !aligned16(workspace)) return QIL_ERR_ALIGN;
    // validate the whole list before the first launch
    bool all_tc = true;
    for (int i = 0; i < count; ++i) {
        const qil_linear_desc& d = descs[i];
        if ((d.flags & ~(QIL_DEP_PREVIOUS | QIL_DEP_NEVER)) != 0) return QIL_ERR_UNSUPPORTED;
        const qil_status s = check_w4a16(d.x, d.qweight, d.scales, d.zeros, d.y, d.M, d.N, d.K, d.group_size,
                                         (qil_layout)d.layout);
        if (s != QIL_OK) return s;
        if (d.layout == QIL_LAYOUT_STREAM128) {
            if (!workspace || workspace_bytes < w4a16_tc_workspace()) return QIL_ERR_WORKSPACE;
            continue;
        }
        all_tc = false;
        const bool skinny = w4a16_skinny_supported(d.M, d.N, d.K, d.group_size, (qil_layout)d.layout);
        if (!skinny && d.layout != QIL_LAYOUT_CANONICAL) return QIL_ERR_UNSUPPORTED;
        if (skinny) {
            const size_t need = w4a16_skinny_workspace(d.M, d.N, d.K, d.group_size);
            if (need > 0 && (!workspace || workspace_bytes < w4a16_skinny_ws_offset() + need)) return QIL_ERR_WORKSPACE;
        }
    }
    if (all_tc) return launch_w4a16_tc(descs, count, workspace, workspace_bytes, S(stream));
    for (int i = 0; i < count; ++i) {
        const qil_linear_desc& d = descs[i];
        const qil_status s = qil_linear_w4a16(d.x, d.qweight, d.scales, d.zeros, d.y, d.M, d.N, d.K, d.group_size,
                                              (qil_layout)d.layout, workspace, workspace_bytes, stream);
        if (s != QIL_OK) return s;
    }
    return QIL_OK;
}

qil_status qil_linear_w4a16_batch_host(const qil_linear_desc* descs, int count, const void* x_host, void* x_stage,
                                       size_t x_bytes, void* y_host, const void* y_stage, size_t y_bytes,
                                       void* workspace, size_t workspace_bytes, qil_stream_t stream) {
    if (!x_host || !x_stage || !y_host || !y_stage) return QIL_ERR_NULL;
    if (x_bytes == 0 || y_bytes == 0) return QIL_ERR_SHAPE;
    if (cudaMemcpyAsync(x_stage, x_host, x_bytes, cudaMemcpyHostToDevice, S(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    const qil_status s = qil_linear_w4a16_batch(descs, count, workspace, workspace_bytes, stream);
    if (s != QIL_OK) return s;
    if (cudaMemcpyAsync(y_host, y_stage, y_bytes, cudaMemcpyDeviceToHost, S(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    return QIL_OK;
}

static qil_status check_w8a16(const void* x, const void* qw, const void* sc, const void* z, const void* y, int M, int N,
                              int K, int G) {
    if (!x || !qw || !y || !sc || !z) return QIL_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || G <= 0 || K % 16 != 0 || K % G != 0) return QIL_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(qw) || !aligned16(y) || !aligned16(sc) || !aligned16(z)) return QIL_ERR_ALIGN;
    return QIL_OK;
}

size_t qil_linear_w8a16_workspace_size(int M, int N, int K, int group_size) {
    if (M <= 0 || N <= 0 || K <= 0 || group_size <= 0) return 0;
    size_t scratch = 0;
    if (w4a16_prefill_supported(M, N, K, group_size, QIL_LAYOUT_CANONICAL)) scratch = w4a16_prefill_workspace(M, N, K, group_size);
    return w8a16_workspace() + scratch;
}

// One linear: the streaming kernel in slabs of four activation rows where the shape allows it, the general kernel
// otherwise.
static qil_status w8a16_one(const qil_linear_desc& d, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    if (w4a16_prefill_supported(d.M, d.N, d.K, d.group_size, QIL_LAYOUT_CANONICAL)) {  // M > 8: the tensor-core GEMM
        const size_t off = w8a16_workspace();
        const bool have = workspace_bytes > off;
        return launch_w4a16_prefill(d.x, d.qweight, d.scales, d.zeros, d.y, d.M, d.N, d.K, d.group_size, 8,
                                    static_cast<int*>(workspace), have ? static_cast<char*>(workspace) + off : nullptr,
                                    have ? workspace_bytes - off : 0, st);
    }
    if (!w8a16_stream_supported(1, d.N, d.K, d.group_size))
        return launch_w8a16_general(d.x, reinterpret_cast<const uint8_t*>(d.qweight), d.scales, d.zeros, d.y, d.M, d.N, d.K,
                                    d.group_size, st);
    for (int m0 = 0; m0 < d.M; m0 += 4) {
        qil_linear_desc s = d;
        s.x = static_cast<const char*>(d.x) + (size_t)m0 * d.K * 2;
        s.y = static_cast<char*>(d.y) + (size_t)m0 * d.N * 2;
        s.M = d.M - m0 < 4 ? d.M - m0 : 4;
        s.flags = 0;
        const qil_status r = launch_w8a16_stream(&s, 1, workspace, workspace_bytes, st);
        if (r != QIL_OK) return r;
    }
    return QIL_OK;
}

qil_status qil_linear_w8a16(const void* x, const uint8_t* qweight, const void* scales, const void* zeros, void* y, int M,
                            int N, int K, int group_size, void* workspace, size_t workspace_bytes, qil_stream_t stream) {
    const qil_status s = check_w8a16(x, qweight, scales, zeros, y, M, N, K, group_size);
    if (s != QIL_OK) return s;
    if (!workspace || workspace_bytes < w8a16_workspace()) return QIL_ERR_WORKSPACE;
    if (!aligned16(workspace)) return QIL_ERR_ALIGN;
    qil_linear_desc d;
    d.x = x; d.qweight = reinterpret_cast<const uint32_t*>(qweight); d.scales = scales; d.zeros = zeros; d.y = y;
    d.M = M; d.N = N; d.K = K; d.group_size = group_size; d.layout = QIL_LAYOUT_CANONICAL; d.flags = 0;
    return w8a16_one(d, workspace, workspace_bytes, S(stream));
}

qil_status qil_linear_w8a16_batch(const qil_linear_desc* descs, int count, void* workspace, size_t workspace_bytes,
                                  qil_stream_t stream) {
    if (!descs) return QIL_ERR_NULL;
    if (count <= 0) return QIL_ERR_SHAPE;
    if (!workspace || workspace_bytes < w8a16_workspace()) return QIL_ERR_WORKSPACE;
    if (!aligned16(workspace)) return QIL_ERR_ALIGN;
    bool all_stream = true;
    for (int i = 0; i < count; ++i) {
        const qil_linear_desc& d = descs[i];
        if ((d.flags & ~(QIL_DEP_PREVIOUS | QIL_DEP_NEVER)) != 0 || d.layout != QIL_LAYOUT_CANONICAL) return QIL_ERR_UNSUPPORTED;
        const qil_status s = check_w8a16(d.x, d.qweight, d.scales, d.zeros, d.y, d.M, d.N, d.K, d.group_size);
        if (s != QIL_OK) return s;
        all_stream = all_stream && w8a16_stream_supported(d.M, d.N, d.K, d.group_size);
    }
    if (all_stream) return launch_w8a16_stream(descs, count, workspace, workspace_bytes, S(stream));
    for (int i = 0; i < count; ++i) {  // stream order keeps every dependency
        const qil_status s = w8a16_one(descs[i], workspace, workspace_bytes, S(stream));
        if (s != QIL_OK) return s;
    }
    return QIL_OK;
}

qil_status qil_quantize_act_a8(const void* x, int M, int K, const float* static_scale, int8_t* qx, float* scales,
                               qil_stream_t stream) {
    if (!x || !qx || !scales) return QIL_ERR_NULL;
    if (M <= 0 || K <= 0 || K % 8 != 0) return QIL_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(qx) || !aligned16(scales)) return QIL_ERR_ALIGN;
    if (static_scale && !(*static_scale > 0.0f)) return QIL_ERR_UNSUPPORTED;
    return launch_quantize_act_a8(x, M, K, static_scale != nullptr, static_scale ? *static_scale : 0.0f, qx, scales,
                                  S(stream));
}

qil_status qil_quantize_act_a4(const void* x, int M, int K, const float* static_scale, uint32_t* qx, float* scales,
                               qil_stream_t stream) {
    if (!x || !qx || !scales) return QIL_ERR_NULL;
    if (M <= 0 || K <= 0 || K % 8 != 0) return QIL_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(qx) || !aligned16(scales)) return QIL_ERR_ALIGN;
    if (static_scale && !(*static_scale > 0.0f)) return QIL_ERR_UNSUPPORTED;
    return launch_quantize_act_a4(x, M, K, static_scale != nullptr, static_scale ? *static_scale : 0.0f, qx, scales,
                                  S(stream));
}

size_t qil_linear_w4a4_workspace_size(int M, int N, int K) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    return w4a4_workspace(M, N, K);
}

qil_status qil_linear_w4a4(const uint32_t* qx, const float* sx, const uint32_t* qw, const float* sw, void* y,
                           int32_t* acc_out, int M, int N, int K, void* workspace, size_t workspace_bytes,
                           qil_stream_t stream) {
    if (!qx || !sx || !qw || !sw || !y) return QIL_ERR_NULL;
    // (the kernel accumulates 256 x the true sum: 256 * 64 * K must stay below 2^31)
    if (M <= 0 || N <= 0 || K <= 0 || K % 32 != 0 || K >= 131072) return QIL_ERR_SHAPE;
    if (!aligned16(qx) || !aligned16(sx) || !aligned16(qw) || !aligned16(sw) || !aligned16(y) ||
        (acc_out && !aligned16(acc_out)) || (workspace && !aligned16(workspace)))
        return QIL_ERR_ALIGN;
    if (w4a4_workspace(M, N, K) > 0 && (!workspace || workspace_bytes < w4a4_workspace(M, N, K)))
        return QIL_ERR_WORKSPACE;
    return launch_w4a4(qx, sx, qw, sw, y, acc_out, M, N, K, 4, workspace, workspace_bytes, S(stream));
}

qil_status qil_linear_w4a4_requant(const uint32_t* qx, const float* sx, const uint32_t* qw, const float* sw, uint32_t* qy,
                                   float out_scale, int relu, int M, int N, int K, void* workspace,
                                   size_t workspace_bytes, qil_stream_t stream) {
    if (!qx || !sx || !qw || !sw || !qy) return QIL_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || K % 32 != 0 || K >= 131072 || N % 8 != 0) return QIL_ERR_SHAPE;
    if (!(out_scale > 0.0f)) return QIL_ERR_UNSUPPORTED;
    if (!aligned16(qx) || !aligned16(sx) || !aligned16(qw) || !aligned16(sw) || !aligned16(qy) ||
        (workspace && !aligned16(workspace)))
        return QIL_ERR_ALIGN;
    if (!workspace || workspace_bytes < w4a4_workspace(M, N, K)) return QIL_ERR_WORKSPACE;
    return launch_w4a4(qx, sx, qw, sw, qy /*unused as y*/, nullptr, M, N, K, 4, workspace, workspace_bytes, S(stream), qy,
                       out_scale, relu ? 1 : 0);
}

qil_status qil_conv3x3_w4a4(const uint32_t* qx, float x_scale, const uint32_t* qw, const float* sw, void* y, int32_t* acc_out,
                            uint32_t* qy, float out_scale, int relu, int B, int H, int W, int C, int Cout, void* workspace,
                            size_t workspace_bytes, qil_stream_t stream) {
    if (!qx || !qw || !sw || (!y && !qy) || (y && qy)) return QIL_ERR_NULL;
    if (B <= 0 || H <= 0 || W <= 0 || C <= 0 || Cout <= 0 || C % 32 != 0 || 9 * C >= 131072) return QIL_ERR_SHAPE;
    if ((long long)B * H * W > 0x7FFFFFFFll) return QIL_ERR_SHAPE;
    if (qy && (Cout % 8 != 0 || acc_out)) return QIL_ERR_SHAPE;
    if (qy && !(out_scale > 0.0f)) return QIL_ERR_UNSUPPORTED;
    if (!aligned16(qx) || !aligned16(qw) || !aligned16(sw) || (y && !aligned16(y)) || (qy && !aligned16(qy)) ||
        (acc_out && !aligned16(acc_out)) || (workspace && !aligned16(workspace)))
        return QIL_ERR_ALIGN;
    const int M = B * H * W, K = 9 * C;
    if (!workspace || workspace_bytes < w4a4_workspace(M, Cout, K)) return QIL_ERR_WORKSPACE;
    return launch_w4a4(qx, nullptr, qw, sw, y ? y : static_cast<void*>(qy), acc_out, M, Cout, K, 4, workspace, workspace_bytes, S(stream),
                       qy, qy ? out_scale : 1.f, relu ? 1 : 0, C, H, W, x_scale);
}

qil_status qil_linear_w8a8(const int8_t* qx, const float* sx, const int8_t* qw, const float* sw, void* y,
                           int32_t* acc_out, int M, int N, int K, void* workspace, size_t workspace_bytes,
                           qil_stream_t stream) {
    if (!qx || !sx || !qw || !sw || !y) return QIL_ERR_NULL;
    // (|acc| <= 2^14 K must stay below 2^31)
    if (M <= 0 || N <= 0 || K <= 0 || K % 16 != 0 || K >= 131072) return QIL_ERR_SHAPE;
    if (!aligned16(qx) || !aligned16(sx) || !aligned16(qw) || !aligned16(sw) || !aligned16(y) ||
        (acc_out && !aligned16(acc_out)) || (workspace && !aligned16(workspace)))
        return QIL_ERR_ALIGN;
    if (!workspace || workspace_bytes < w4a4_workspace(M, N, K)) return QIL_ERR_WORKSPACE;
    return launch_w4a4(qx, sx, qw, sw, y, acc_out, M, N, K, 8, workspace, workspace_bytes, S(stream));
}

qil_status qil_linear_int_batch(const qil_igemm_desc* descs, int count, void* workspace, size_t workspace_bytes,
                                qil_stream_t stream) {
    if (!descs) return QIL_ERR_NULL;
    if (count <= 0) return QIL_ERR_SHAPE;
    if (!workspace || workspace_bytes < 16) return QIL_ERR_WORKSPACE;
    if (!aligned16(workspace)) return QIL_ERR_ALIGN;
    for (int i = 0; i < count; ++i) {
        const qil_igemm_desc& d = descs[i];
        if (!d.qx || !d.sx || !d.qw || !d.sw || !d.y) return QIL_ERR_NULL;
        if (d.bits != 4 && d.bits != 8) return QIL_ERR_UNSUPPORTED;
        if (d.M <= 0 || d.N <= 0 || d.K <= 0 || d.K % (d.bits == 4 ? 32 : 16) != 0 || d.K >= 131072) return QIL_ERR_SHAPE;
        if (!aligned16(d.qx) || !aligned16(d.sx) || !aligned16(d.qw) || !aligned16(d.sw) || !aligned16(d.y) ||
            (d.acc_out && !aligned16(d.acc_out)))
            return QIL_ERR_ALIGN;
    }
    if (igemm_list_supported(descs, count)) return launch_igemm_list(descs, count, workspace, workspace_bytes, S(stream));
    for (int i = 0; i < count; ++i) {
        const qil_igemm_desc& d = descs[i];
        const qil_status s = launch_w4a4(d.qx, d.sx, d.qw, d.sw, d.y, d.acc_out, d.M, d.N, d.K, d.bits, workspace,
                                         workspace_bytes, S(stream));
        if (s != QIL_OK) return s;
    }
    return QIL_OK;
}

qil_status qil_ref_gemv_bf16(const void* x, const void* w, void* y, int N, int K, qil_stream_t stream) {
    if (!x || !w || !y) return QIL_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 8 != 0) return QIL_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y)) return QIL_ERR_ALIGN;
    return launch_ref_gemv_bf16(x, w, y, N, K, S(stream));
}

qil_status qil_probe_mma_i8(int iters, int commit_every, double* ops_out, int* dev_status, qil_stream_t stream) {
    if (iters <= 0 || iters > (1 << 24) || commit_every <= 0) return QIL_ERR_SHAPE;
    return launch_probe_mma(true, iters, commit_every, ops_out, dev_status, S(stream));
}

qil_status qil_probe_mma_bf16(int iters, int commit_every, double* ops_out, int* dev_status, qil_stream_t stream) {
    if (iters <= 0 || iters > (1 << 24) || commit_every <= 0) return QIL_ERR_SHAPE;
    return launch_probe_mma(false, iters, commit_every, ops_out, dev_status, S(stream));
}

qil_status qil_probe_hbm_read(const void* buf, size_t bytes, unsigned int* sink, qil_stream_t stream) {
    if (!buf || !sink) return QIL_ERR_NULL;
    if (bytes < 16) return QIL_ERR_SHAPE;
    if (!aligned16(buf)) return QIL_ERR_ALIGN;
    return launch_probe_hbm_read(buf, bytes, sink, S(stream));
}

}  // extern "C"
