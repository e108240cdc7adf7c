// Expert FFN entry point for callers that cannot allocate device memory.
//
// Some hosts of this library run under rules that forbid cudaMalloc at the point where the
// layer is called: a serving loop that pre-allocates everything at start-up and treats any
// later allocation as a bug, a plug-in that is handed input and output buffers by a
// framework and owns no allocator of its own, code running while a CUDA graph is being
// captured or inside a memory pool it must not grow.  monde_moe_ffn_fwd needs a caller-
// provided workspace (hidden activations, dependency counters, split-K partial tiles);
// this variant brings its own: a fixed array in the library's device image.
//
// The array exists once per GPU that loads the library, from load until the process exits,
// and is shared by every call on that GPU.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kStaticWsBytes = MONDE_STATIC_WS_BYTES;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress;
// it is not a device address and must never be passed to a kernel or a memset.
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

using monde::kMaxDevices;
std::mutex g_mutex;
void* g_ws_ptr[kMaxDevices] = {};

// Device address of the array on the current device, looked up once per device.
int static_ws_ptr(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MONDE_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_ws_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || p == nullptr) {
            cudaGetLastError();      // do not leave the failure behind for an unrelated later call to find
            return MONDE_ERR_CUDA;
        }
        g_ws_ptr[dev] = p;
    }
    *out = g_ws_ptr[dev];
    return MONDE_OK;
}

}  // namespace

extern "C" int monde_moe_ffn_fwd_static_ws(const monde_problem* p, const void* x_perm,
                                           const void* W1, const void* b1, const void* W2, const void* b2,
                                           const int32_t* counts, const int32_t* offsets, const uint8_t* cls,
                                           const int32_t* hot_ids, const int32_t* cold_ids,
                                           const int32_t* n_hot_cold, void* y_perm, void* stream) {
    int st = monde::check_problem(p);
    if (st != MONDE_OK) return st;
    if (p->T == 0) return MONDE_OK;
    const monde::WsLayout L = monde::ws_layout(*p);
    if (L.total > kStaticWsBytes) return MONDE_ERR_WORKSPACE;   // needs more scratch than the built-in array holds
    // every check that can reject the call comes before the shared array is touched
    if ((st = monde::check_ffn_fwd_args(x_perm, W1, b1, W2, b2, counts, offsets, cls, hot_ids, cold_ids, n_hot_cold,
                                        y_perm)) != MONDE_OK)
        return st;
    void* ws = nullptr;
    if ((st = static_ws_ptr(&ws)) != MONDE_OK) return st;
    // The array keeps whatever the previous call left.  Everything the kernels expect to find
    // at zero lives in the header (status, tickets, dependency counters, split-K counters):
    // clear it, in stream order, before the launch.  The hidden activations and partial tiles
    // are fully rewritten before they are read.
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, monde::WsLayout::kHidden, s) != cudaSuccess) return MONDE_ERR_CUDA;
    return monde_moe_ffn_fwd(p, x_perm, W1, b1, W2, b2, counts, offsets, cls, hot_ids, cold_ids, n_hot_cold, y_perm,
                             ws, kStaticWsBytes, stream);
}

extern "C" int monde_poll_static_ws_status(void* stream, int32_t* site) {
    void* ws = nullptr;
    const int st = static_ws_ptr(&ws);
    if (st != MONDE_OK) return st;
    return monde_poll_device_status(ws, stream, site);   // copies two words out, clears the header if it reports: no allocation
}
