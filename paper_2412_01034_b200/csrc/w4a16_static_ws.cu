// qil_linear_w4a16_static_ws: the weight-only 4-bit linear for callers that cannot
// allocate device memory (see qil.h).  The split-K scratch of the decode kernel lives
// in a fixed array inside the library image instead of a caller-supplied workspace.
#include <mutex>

#include "qil_common.cuh"

namespace {

// Scratch shared by every call on a device: arrival counters followed by fp32 partial
// tiles.  Each GPU that loads the library carries this array until the process exits.
static __device__ __align__(256) unsigned char g_static_ws[QIL_STATIC_WS_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_ws_ptr[kMaxDevices] = {};  // device address of g_static_ws, per device ordinal

// The array's name is only a handle on the host; kernels need its device address, which
// differs per device and must be looked up with that device current.
qil_status static_ws_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_ws_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_ws) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return QIL_ERR_CUDA;
        }
        g_ws_ptr[dev] = ptr;
    }
    *out = g_ws_ptr[dev];
    return QIL_OK;
}

}  // namespace

extern "C" size_t qil_linear_w4a16_static_ws_need(int M, int N, int K, int group_size) {
    if (M <= 0 || N <= 0 || K <= 0 || group_size <= 0 || K % 128 != 0 || group_size % 128 != 0) return 0;
    return qil::w4a16_skinny_workspace(M, N, K, group_size);
}

extern "C" qil_status qil_linear_w4a16_static_ws(const void* x, const uint32_t* qweight, const void* scales,
                                                 const void* zeros, void* y, int M, int N, int K, int group_size,
                                                 qil_layout layout, qil_stream_t stream) {
    using namespace qil;
    if (!x || !qweight || !scales || !zeros || !y) return QIL_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || group_size <= 0 || K % 8 != 0 || K % group_size != 0) return QIL_ERR_SHAPE;
    if (layout != QIL_LAYOUT_CANONICAL && layout != QIL_LAYOUT_TILE16) return QIL_ERR_UNSUPPORTED;
    if (layout == QIL_LAYOUT_TILE16 && (N % 16 != 0 || K % 128 != 0)) return QIL_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(qweight) || !aligned16(scales) || !aligned16(zeros) || !aligned16(y))
        return QIL_ERR_ALIGN;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (!w4a16_skinny_supported(M, N, K, group_size, layout)) {
        // shapes outside the tensor-core decode kernel use the general kernel, which needs no scratch
        if (layout != QIL_LAYOUT_CANONICAL) return QIL_ERR_UNSUPPORTED;
        return launch_w4a16_general(x, qweight, scales, zeros, y, M, N, K, group_size, st);
    }
    const size_t need = w4a16_skinny_workspace(M, N, K, group_size);
    if (need > (size_t)QIL_STATIC_WS_BYTES) return QIL_ERR_WORKSPACE;  // beyond the built-in scratch
    void* ws = nullptr;
    if (need > 0) {
        const qil_status s = static_ws_address(&ws);
        if (s != QIL_OK) return s;
        // the array keeps whatever the previous call (or an interrupted one) left: the arrival
        // counters must start at zero, the partial tiles are fully rewritten before they are read
        if (cudaMemsetAsync(ws, 0, w4a16_skinny_counter_bytes(), st) != cudaSuccess) {
            (void)cudaGetLastError();
            return QIL_ERR_CUDA;
        }
    }
    return launch_w4a16_skinny(x, qweight, scales, zeros, y, M, N, K, group_size, layout, ws, need, st);
}
