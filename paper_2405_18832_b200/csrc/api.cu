// extern "C" entry points: argument checks, workspace carving, launches.
#include <atomic>
#include <mutex>

#include "../../include/monde_diagnostics.h"
#include "common.cuh"

namespace monde {

int check_problem(const monde_problem* p) {
    if (p == nullptr) return MONDE_ERR_INVALID_ARG;
    if (p->T < 0 || p->d_model <= 0 || p->d_ff <= 0 || p->E <= 0 || p->top_k <= 0) return MONDE_ERR_INVALID_ARG;
    if (p->top_k > p->E) return MONDE_ERR_INVALID_ARG;
    if (p->dtype != MONDE_F32 && p->dtype != MONDE_BF16) return MONDE_ERR_UNSUPPORTED;
    if (p->act != MONDE_ACT_RELU && p->act != MONDE_ACT_GELU_ERF) return MONDE_ERR_UNSUPPORTED;
    if (p->E > kMaxExperts || p->top_k > kMaxTopK) return MONDE_ERR_UNSUPPORTED;
    const int mult = p->dtype == MONDE_BF16 ? 64 : 4;
    if (p->d_model % mult != 0 || p->d_ff % mult != 0) return MONDE_ERR_UNSUPPORTED;
    if (static_cast<int64_t>(p->T) * p->top_k > kMaxAssignments) return MONDE_ERR_UNSUPPORTED;
    return MONDE_OK;
}

static std::atomic<long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---- per-device set-up bookkeeping ----------------------------------------------------------
namespace {
std::mutex g_dev_mutex;
// 0: not run on that device yet; 1: ran and succeeded; otherwise 2 + the cudaError_t it returned
int g_setup[kMaxDevices][kSetupKeys] = {};
int g_sms[kMaxDevices] = {};
}  // namespace

cudaError_t per_device_once(int key, cudaError_t (*fn)()) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices || key < 0 || key >= kSetupKeys) return cudaErrorInvalidValue;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    int& state = g_setup[dev][key];
    if (state == 0) {
        e = fn();
        state = e == cudaSuccess ? 1 : 2 + static_cast<int>(e);
    }
    return state == 1 ? cudaSuccess : static_cast<cudaError_t>(state - 2);
}

int current_sm_count() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (g_sms[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        g_sms[dev] = v;
    }
    return g_sms[dev];
}

// ---- diagnostic switches --------------------------------------------------------------------
namespace {
constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;   // 2 s
std::atomic<unsigned long long*> g_trace{nullptr};
std::atomic<int> g_trace_slots{0};
std::atomic<int> g_ffn_pair{-1};
std::atomic<unsigned long long> g_wait_limit_ns{kDefaultWaitLimitNs};
std::atomic<int> g_hold_hidden_ready{0};
}  // namespace

#ifdef MONDE_DIAGNOSTICS
namespace {
__device__ DiagRecord g_diag_record;      // host code may only take its address through cudaGetSymbolAddress
DiagRecord* g_diag_ptr[kMaxDevices] = {};
}  // namespace
DiagRecord* diag_record_ptr() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (g_diag_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_diag_record) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        g_diag_ptr[dev] = static_cast<DiagRecord*>(p);
    }
    return g_diag_ptr[dev];
}
#else
DiagRecord* diag_record_ptr() { return nullptr; }
#endif

DiagState diag_state() {
    DiagState d;
    d.trace = g_trace.load(std::memory_order_relaxed);
    d.trace_slots = g_trace_slots.load(std::memory_order_relaxed);
    d.ffn_pair = g_ffn_pair.load(std::memory_order_relaxed);
    d.wait_limit_ns = g_wait_limit_ns.load(std::memory_order_relaxed);
    d.hold_hidden_ready = g_hold_hidden_ready.load(std::memory_order_relaxed);
    return d;
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_arch() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MONDE_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return MONDE_ERR_CUDA;
    return major == 10 ? MONDE_OK : MONDE_ERR_ARCH;
}

int check_ws(const monde_problem& p, const void* ws, size_t ws_bytes) {
    if (ws == nullptr || !aligned16(ws)) return MONDE_ERR_INVALID_ARG;
    if (ws_bytes < ws_layout(p).total) return MONDE_ERR_WORKSPACE;
    return MONDE_OK;
}

}  // namespace

int check_ffn_fwd_args(const void* x_perm, const void* W1, const void* b1, const void* W2, const void* b2,
                       const int32_t* counts, const int32_t* offsets, const uint8_t* cls, const int32_t* hot_ids,
                       const int32_t* cold_ids, const int32_t* n_hot_cold, const void* y_perm) {
    if (!x_perm || !W1 || !W2 || !counts || !offsets || !cls || !hot_ids || !cold_ids || !n_hot_cold || !y_perm)
        return MONDE_ERR_INVALID_ARG;
    if (!aligned16(x_perm) || !aligned16(W1) || !aligned16(W2) || !aligned16(y_perm) || !aligned16(b1) ||
        !aligned16(b2))
        return MONDE_ERR_INVALID_ARG;
    return check_arch();
}

}  // namespace monde

using namespace monde;

extern "C" {

size_t monde_workspace_bytes(const monde_problem* p) {
    if (check_problem(p) != MONDE_OK) return 0;
    return ws_layout(*p).total;
}

const char* monde_status_string(int status) {
    switch (status) {
        case MONDE_OK: return "ok";
        case MONDE_ERR_INVALID_ARG: return "invalid argument";
        case MONDE_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case MONDE_ERR_WORKSPACE: return "workspace too small";
        case MONDE_ERR_ARCH: return "device is not compute capability 10.x";
        case MONDE_ERR_CUDA: return "CUDA call failed";
        case MONDE_ERR_TIMEOUT: return "device-side wait timed out";
        case MONDE_ERR_BOUNDS: return "index out of range (diagnostics build)";
        default: return "unknown status";
    }
}

int monde_route(const monde_problem* p, const void* x, const void* Wg, const float* bg,
                int32_t* topk_idx, float* topk_w, int32_t* counts, int32_t* offsets,
                uint8_t* cls, int32_t* hot_ids, int32_t* cold_ids, int32_t* n_hot_cold,
                float* probs, void* ws, size_t ws_bytes, void* stream) {
    int st = check_problem(p);
    if (st != MONDE_OK) return st;
    if (!Wg || !counts || !offsets || !cls || !hot_ids || !cold_ids || !n_hot_cold) return MONDE_ERR_INVALID_ARG;
    if (p->T > 0 && (!x || !topk_idx || !topk_w)) return MONDE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(Wg)) return MONDE_ERR_INVALID_ARG;
    if ((st = check_ws(*p, ws, ws_bytes)) != MONDE_OK) return st;
    if ((st = check_arch()) != MONDE_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return launch_route(*p, x, Wg, bg, topk_idx, topk_w, probs, counts, offsets, cls, hot_ids, cold_ids, n_hot_cold,
                        ws, s);
}

int monde_classify_top_h(const monde_problem* p, const int32_t* counts, double alpha, double bw_hot_feed,
                         double bw_cold_feed, uint8_t* cls, int32_t* hot_ids, int32_t* cold_ids,
                         int32_t* n_hot_cold, void* stream) {
    int st = check_problem(p);
    if (st != MONDE_OK) return st;
    if (!counts || !cls || !hot_ids || !cold_ids || !n_hot_cold) return MONDE_ERR_INVALID_ARG;
    if (!(alpha >= 0.0) || !(bw_hot_feed > 0.0) || !(bw_cold_feed > 0.0)) return MONDE_ERR_INVALID_ARG;
    if ((st = check_arch()) != MONDE_OK) return st;
    const double share = alpha * bw_hot_feed / (bw_cold_feed + bw_hot_feed);
    return launch_classify_top_h(*p, share, counts, cls, hot_ids, cold_ids, n_hot_cold,
                                 static_cast<cudaStream_t>(stream));
}

int monde_permute(const monde_problem* p, const void* x, const int32_t* topk_idx,
                  const int32_t* offsets, int32_t* perm, int32_t* inv_perm, void* x_perm,
                  void* ws, size_t ws_bytes, void* stream) {
    int st = check_problem(p);
    if (st != MONDE_OK) return st;
    if (p->T == 0) return MONDE_OK;
    if (!x || !topk_idx || !offsets || !perm || !inv_perm || !x_perm) return MONDE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(x_perm)) return MONDE_ERR_INVALID_ARG;
    if ((st = check_ws(*p, ws, ws_bytes)) != MONDE_OK) return st;
    if ((st = check_arch()) != MONDE_OK) return st;
    return launch_permute(*p, x, topk_idx, offsets, perm, inv_perm, x_perm, ws, static_cast<cudaStream_t>(stream));
}

int monde_moe_ffn_fwd(const monde_problem* p, const void* x_perm,
                      const void* W1, const void* b1, const void* W2, const void* b2,
                      const int32_t* counts, const int32_t* offsets, const uint8_t* cls,
                      const int32_t* hot_ids, const int32_t* cold_ids, const int32_t* n_hot_cold,
                      void* y_perm, void* ws, size_t ws_bytes, void* stream) {
    int st = check_problem(p);
    if (st != MONDE_OK) return st;
    if (p->T == 0) return MONDE_OK;
    if ((st = check_ffn_fwd_args(x_perm, W1, b1, W2, b2, counts, offsets, cls, hot_ids, cold_ids, n_hot_cold,
                                 y_perm)) != MONDE_OK)
        return st;
    if ((st = check_ws(*p, ws, ws_bytes)) != MONDE_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    void* h = static_cast<char*>(ws) + WsLayout::kHidden;
    if (p->dtype == MONDE_F32) {
        // Same kernel for both classes; the class lists still select the experts.
        const int32_t* lists[2] = {hot_ids, cold_ids};
        for (int c = 0; c < 2; ++c) {
            st = launch_linear_simt(p->dtype, p->act, p->E, p->d_model, p->d_ff, x_perm, W1, b1, offsets,
                                    lists[c], n_hot_cold + c, h, s);
            if (st != MONDE_OK) return st;
            st = launch_linear_simt(p->dtype, -1, p->E, p->d_ff, p->d_model, h, W2, b2, offsets, lists[c],
                                    n_hot_cold + c, y_perm, s);
            if (st != MONDE_OK) return st;
        }
        return MONDE_OK;
    }
    // (the tensor-core kernel rebuilds the class lists from cls, counts and offsets in one pass)
    return launch_ffn_bf16(*p, x_perm, W1, b1, W2, b2, counts, offsets, cls, y_perm, ws, s);
}

int monde_moe_ffn_combine_fwd(const monde_problem* p, const void* x_perm,
                              const void* W1, const void* b1, const void* W2, const void* b2,
                              const int32_t* counts, const int32_t* offsets, const uint8_t* cls,
                              const int32_t* perm, const float* topk_w, void* out,
                              void* ws, size_t ws_bytes, void* stream) {
    int st = check_problem(p);
    if (st != MONDE_OK) return st;
    if (p->dtype != MONDE_BF16) return MONDE_ERR_UNSUPPORTED;
    if (p->T == 0) return MONDE_OK;
    if (!x_perm || !W1 || !W2 || !counts || !offsets || !cls || !perm || !topk_w || !out) return MONDE_ERR_INVALID_ARG;
    if (!aligned16(x_perm) || !aligned16(W1) || !aligned16(W2) || !aligned16(out) || !aligned16(b1) || !aligned16(b2))
        return MONDE_ERR_INVALID_ARG;
    if ((st = check_ws(*p, ws, ws_bytes)) != MONDE_OK) return st;
    if ((st = check_arch()) != MONDE_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (p->top_k == 1)      // one term per token: the last store applies the gate weight and writes `out`
        return launch_ffn_bf16(*p, x_perm, W1, b1, W2, b2, counts, offsets, cls, nullptr, ws, s, perm, topk_w, out);
    // Several terms per token: the last store puts every expert output row at its assignment id, i.e. the
    // top_k rows of a token side by side (a staging buffer in the workspace), and the combine kernel adds
    // them in slot order without looking anything up: same arithmetic as monde_combine, same bytes.
    void* stage = static_cast<char*>(ws) + ws_layout(*p).stage_off;
    st = launch_ffn_bf16(*p, x_perm, W1, b1, W2, b2, counts, offsets, cls, nullptr, ws, s, perm, nullptr, stage);
    if (st != MONDE_OK) return st;
    return launch_combine(*p, stage, nullptr, topk_w, out, s);
}

int monde_combine(const monde_problem* p, const void* y_perm, const int32_t* inv_perm,
                  const float* topk_w, void* out, void* stream) {
    int st = check_problem(p);
    if (st != MONDE_OK) return st;
    if (p->T == 0) return MONDE_OK;
    if (!y_perm || !inv_perm || !topk_w || !out) return MONDE_ERR_INVALID_ARG;
    if (!aligned16(y_perm) || !aligned16(out)) return MONDE_ERR_INVALID_ARG;
    if ((st = check_arch()) != MONDE_OK) return st;
    return launch_combine(*p, y_perm, inv_perm, topk_w, out, static_cast<cudaStream_t>(stream));
}

long long monde_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int monde_poll_device_status(void* ws, void* stream, int32_t* site) {
    if (ws == nullptr) return MONDE_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t word[2] = {0, 0};
    if (cudaMemcpyAsync(word, static_cast<char*>(ws) + WsLayout::kStatus, sizeof word, cudaMemcpyDeviceToHost, s) !=
        cudaSuccess)
        return MONDE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return MONDE_ERR_CUDA;
    if (site != nullptr) *site = word[1];
    if (word[0] != 0) {   // a kernel gave up: its counters may be mid-way, so clear the whole header
        if (cudaMemsetAsync(ws, 0, WsLayout::kHidden, s) != cudaSuccess)
            return MONDE_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return MONDE_ERR_CUDA;
    }
    return word[0];
}

// ---- include/monde_diagnostics.h --------------------------------------------------------------
int monde_diag_bounds_violations(int32_t* first_site, long long* first_value) {
#ifdef MONDE_DIAGNOSTICS
    DiagRecord* dev = diag_record_ptr();
    if (dev == nullptr) return -2;
    DiagRecord rec;
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(&rec, dev, sizeof rec, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemset(dev, 0, sizeof rec) != cudaSuccess)
        return -2;
    if (first_site != nullptr) *first_site = rec.site;
    if (first_value != nullptr) *first_value = rec.value;
    return rec.count;
#else
    (void)first_site;
    (void)first_value;
    return -1;      // not a diagnostics build
#endif
}

void monde_diag_set_ffn_cta_pairs(int mode) { g_ffn_pair.store(mode < 0 ? -1 : (mode != 0), std::memory_order_relaxed); }

void monde_diag_set_trace(void* device_buf, int slots) {
    g_trace_slots.store(device_buf != nullptr && slots > 0 ? slots : 0, std::memory_order_relaxed);
    g_trace.store(slots > 0 ? static_cast<unsigned long long*>(device_buf) : nullptr, std::memory_order_relaxed);
}

void monde_diag_set_wait_limit_ns(unsigned long long ns) {
    g_wait_limit_ns.store(ns == 0 ? kDefaultWaitLimitNs : ns, std::memory_order_relaxed);
}

void monde_diag_set_hold_hidden_ready(int on) { g_hold_hidden_ready.store(on != 0, std::memory_order_relaxed); }

int monde_diag_device_setups(int device) {
    if (device < 0 || device >= kMaxDevices) return -1;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    int n = 0;
    for (int k = 0; k < kSetupKeys; ++k) n += g_setup[device][k] != 0;
    return n;
}

}  // extern "C"
