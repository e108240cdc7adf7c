// Shared declarations of the CUDA library: problem checks, workspace layout,
// element load/convert helpers, launch prototypes.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/monde.h"

namespace monde {

constexpr int kMaxExperts = 256;
constexpr int kMaxTopK = 8;

// Workspace carving.  Offsets in bytes from the workspace base.
struct WsLayout {
    static constexpr size_t kStatus = 0;        // int32 status, int32 site
    static constexpr size_t kRouteTicket = 512; // int32: router CTAs finished; then one int32 per 16-token tile of the split router
    static constexpr size_t kCounters = 1024;   // int32 counters used by the FFN kernels
    static constexpr size_t kCountersBytes = 15 * 1024;
    static constexpr size_t kTiles = 16 * 1024; // work lists built on the device
    static constexpr size_t kTilesBytes = 112 * 1024;
    static constexpr size_t kPartDone = 128 * 1024;   // int32 per cold second-layer tile: partial tiles finished
    static constexpr size_t kPartDoneBytes = 128 * 1024;
    static constexpr size_t kHidden = 256 * 1024;  // h [A, d_ff] in the problem dtype
    size_t hidden_bytes;
    int n_split;            // K-splits of a cold second-layer unit
    size_t part_done_off;   // = kPartDone: inside the header, so it is zero whatever problem used the buffer before
    size_t part_done_bytes;
    size_t partials_off;    // fp32 partial tiles of the K-split cold second-layer units
    size_t partials_bytes;
    size_t logits_off;         // fp32 [T][kMaxExperts]: gate logits of small batches, between the two phases of the split router
    size_t stage_off;          // [T][top_k][d_model] in the problem dtype: expert outputs in token order (fused combine, top_k > 1)
    size_t total;
};
constexpr int kSplitRouteMaxTokens = 256;   // batches up to this size take the split router (experts dealt over CTAs)
// The header (first kHidden bytes) holds everything that must be zero between calls: the
// status word, the CTA ticket (kCounters), one int32 per token tile that counts finished
// first-layer units (kTiles) and one per cold second-layer tile that counts finished partial
// tiles (kPartDone).  Its layout does not depend on the problem, so problems of different shapes
// may take turns on one workspace.  A <= kMaxAssignments keeps the token-tile counters inside
// it; problems with more cold second-layer tiles than kPartDone holds run without the K-split.
constexpr int64_t kMaxAssignments = 1 << 20;
static_assert(4 * (kMaxAssignments / 64 + 2 * 256 + 64) <= 112 * 1024, "token-tile counters overflow the header");

inline size_t elem_bytes(int dtype) { return dtype == MONDE_BF16 ? 2 : 4; }

// Token-tile width of the cold class: a cold expert has at most hot_threshold-1 rows.
inline int cold_token_tile(const monde_problem& p) {
    const long long t = (static_cast<long long>(p.hot_threshold) - 1 + 15) / 16 * 16;
    return static_cast<int>(t < 16 ? 16 : (t > 64 ? 64 : t));
}

inline WsLayout ws_layout(const monde_problem& p) {
    WsLayout l;
    size_t A = static_cast<size_t>(p.T) * p.top_k;
    l.hidden_bytes = (A * p.d_ff * elem_bytes(p.dtype) + 1023) / 1024 * 1024;
    // Cold second-layer units are split along K when d_ff is a multiple of d_model's size and
    // the partial tiles fit a bounded scratch (otherwise no split).
    const size_t ct = cold_token_tile(p);
    const size_t nt2 = (static_cast<size_t>(p.d_model) + 127) / 128;
    const size_t cold_tiles = (A / ct + p.E) * (nt2 + 1);    // upper bound on cold second-layer tiles (units cover pairs)
    int split = p.d_ff / p.d_model;
    split = split < 1 ? 1 : (split > 4 ? 4 : split);
    const int kb2 = p.d_ff / 64;                              // every sub-unit must own at least one K block
    while (split > 1 && (split - 1) * ((kb2 + split - 1) / split) >= kb2) --split;
    size_t part = cold_tiles * (split - 1) * ct * 128 * 4;
    if (part > (size_t(1) << 30) || cold_tiles * 4 > WsLayout::kPartDoneBytes) { split = 1; part = 0; }
    l.n_split = split;
    l.part_done_off = WsLayout::kPartDone;
    l.part_done_bytes = split > 1 ? (cold_tiles * 4 + 1023) / 1024 * 1024 : 0;
    l.partials_off = WsLayout::kHidden + l.hidden_bytes;
    l.partials_bytes = part;
    auto round256 = [](size_t v) { return (v + 255) / 256 * 256; };
    l.logits_off = round256(l.partials_off + l.partials_bytes);
    const size_t logits_bytes = p.T <= kSplitRouteMaxTokens ? static_cast<size_t>(p.T) * kMaxExperts * 4 : 0;
    l.stage_off = round256(l.logits_off + logits_bytes);
    const size_t stage_bytes = (p.top_k > 1 && p.dtype == MONDE_BF16) ? A * p.d_model * elem_bytes(p.dtype) : 0;
    l.total = l.stage_off + stage_bytes + 1024;
    return l;
}

// MONDE_OK when the problem is inside the stated limits.
int check_problem(const monde_problem* p);
// Pointer, alignment and architecture checks of monde_moe_ffn_fwd (everything but the workspace).
int check_ffn_fwd_args(const void* x_perm, const void* W1, const void* b1, const void* W2, const void* b2,
                       const int32_t* counts, const int32_t* offsets, const uint8_t* cls, const int32_t* hot_ids,
                       const int32_t* cold_ids, const int32_t* n_hot_cold, const void* y_perm);

// ---- element helpers --------------------------------------------------------
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}

// 16-byte vector of elements, unpacked to floats.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void load(const float* p, float (&o)[4]) {
        float4 v = *reinterpret_cast<const float4*>(p);
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
    __device__ static __forceinline__ void store(float* p, const float (&o)[4]) {
        *reinterpret_cast<float4*>(p) = make_float4(o[0], o[1], o[2], o[3]);
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&o)[8]) {
        uint4 v = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            o[2 * i] = __uint_as_float(w[i] << 16);
            o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static __forceinline__ void store(__nv_bfloat16* p, const float (&o)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(o[2 * i], o[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act == MONDE_ACT_RELU) return fmaxf(v, 0.0f);
    return 0.5f * v * (1.0f + erff(v * 0.70710678118654752440f));
}

// ---- launch prototypes (each returns a monde_status) -------------------------
// Gate + softmax + top-k; the router CTA that finishes last also runs the histogram,
// classification and scan.  `ticket` is an int32 in the workspace header (zero between calls).
int launch_route(const monde_problem& p, const void* x, const void* Wg, const float* bg,
                 int32_t* topk_idx, float* topk_w, float* probs, int32_t* counts, int32_t* offsets, uint8_t* cls,
                 int32_t* hot_ids, int32_t* cold_ids, int32_t* n_hot_cold, void* ws, cudaStream_t s);
int launch_classify_top_h(const monde_problem& p, double share, const int32_t* counts, uint8_t* cls,
                          int32_t* hot_ids, int32_t* cold_ids, int32_t* n_hot_cold, cudaStream_t s);
// Large batches use a dead part of the workspace (the hidden-activation region) for per-expert prefix counts.
int launch_permute(const monde_problem& p, const void* x, const int32_t* topk_idx, const int32_t* offsets,
                   int32_t* perm, int32_t* inv_perm, void* x_perm, const void* ws, cudaStream_t s);
int launch_combine(const monde_problem& p, const void* y_perm, const int32_t* inv_perm,
                   const float* topk_w, void* out, cudaStream_t s);

// Out[r, n] = act?(bias[e, n] + sum_k In[r, k] * W[e, n, k]) for the rows of the experts in
// `ids[0 .. *n_ids)`; plain CUDA-core kernel (fp32 problems; debugging aid for bf16).
int launch_linear_simt(int dtype, int act_or_neg1, int E, int K, int N, const void* in, const void* W,
                       const void* bias, const int32_t* offsets, const int32_t* ids, const int32_t* n_ids,
                       void* out, cudaStream_t s);

// bf16 problems: hot experts on the tcgen05 grouped GEMM, cold experts on the
// weight-streaming kernel.
int launch_ffn_bf16(const monde_problem& p, const void* x_perm, const void* W1, const void* b1,
                    const void* W2, const void* b2, const int32_t* counts, const int32_t* offsets,
                    const uint8_t* cls, void* y_perm, void* ws, cudaStream_t s,
                    const int32_t* fuse_perm = nullptr, const float* fuse_w = nullptr, void* fuse_out = nullptr);

// Process-wide count of kernels this library has launched (diagnostic).
void count_launches(int n);

// ---- range checks of the diagnostics build ---------------------------------------------------
// Built with -DMONDE_DIAGNOSTICS the kernels check every index they take from memory before they use
// it as an address (expert ids, positions of the permutation, the rows and features of an FFN work
// unit), count violations in a record inside the library's device image, keep the first one (site and
// value) and skip the access.  The ordinary build compiles the checks away.  This stands in for a
// memory checker on machines where none may be run.
struct DiagRecord {
    int32_t count;      // violations since the record was last read
    int32_t site;       // of the first one: 1 permute expert id, 2 permute position, 3 combine position,
    long long value;    //                   4 FFN unit rows, 5 FFN unit features; and the offending value
};
DiagRecord* diag_record_ptr();    // device address of the record on the current device; null in the ordinary build
#ifdef MONDE_DIAGNOSTICS
__device__ __forceinline__ bool diag_in_range(bool ok, DiagRecord* rec, int site, long long value) {
    if (!ok && rec != nullptr && atomicAdd(&rec->count, 1) == 0) {
        rec->site = site;
        rec->value = value;
    }
    return ok;
}
#define MONDE_IN_RANGE(cond, rec, site, value) diag_in_range((cond), (rec), (site), static_cast<long long>(value))
#else
#define MONDE_IN_RANGE(cond, rec, site, value) true
#endif

// ---- per-device set-up ---------------------------------------------------------------------
// Function attributes (the opt-in to more than 48 KB of dynamic shared memory) and the SM count
// belong to a device, not to the process: a process that drives several GPUs must set them up on
// each.  `per_device_once(key, fn)` runs `fn` once for the current device and the given key and
// returns its (cached) result on every later call; keys are small integers owned by the callers.
constexpr int kMaxDevices = 64;
enum SetupKey { kSetupFfn = 0, kSetupRoute1, kSetupRoute2, kSetupRoute4, kSetupRoute8, kSetupKeys };
cudaError_t per_device_once(int key, cudaError_t (*fn)());
int current_sm_count();        // multiprocessors of the current device (cached per device)

// ---- diagnostic switches (include/monde_diagnostics.h) ---------------------------------------
// Process-wide, read at launch time; defaults leave the product path unchanged.
struct DiagState {
    unsigned long long* trace;      // per-unit device timeline of the expert FFN (null = off)
    int trace_slots;
    int ffn_pair;                   // -1 default, 0 single CTAs, 1 CTA pairs
    unsigned long long wait_limit_ns;   // bound of every device-side wait
    int hold_hidden_ready;          // 1: first-layer units do not publish their rows (a dependency wait then runs out)
};
DiagState diag_state();

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? MONDE_OK : MONDE_ERR_CUDA; }

// Programmatic dependent launch.  Every kernel of the library is launched with the
// programmatic-stream-serialization attribute, calls pdl_launch_dependents() early (the next
// kernel in the stream may then be scheduled and run its set-up), and calls pdl_wait() before
// it reads anything another kernel may have produced and before it writes anything to global
// memory.  pdl_wait() returns once the preceding kernel in the stream has completed and its
// writes are visible; since that kernel waited the same way, everything earlier is complete too.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// The same, with the grid grouped into thread-block clusters of `cluster_x` consecutive CTAs.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, unsigned cluster_x,
                                      cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
inline int launched(int n = 1) {
    count_launches(n);
    return cuda_status(cudaGetLastError());
}

}  // namespace monde
