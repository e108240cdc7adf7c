/* monde.h -- C ABI of the B200 (sm_100a) MoE FFN layer forward with a load-aware
 * hot/cold expert split (MoNDE, arXiv 2405.18832).
 *
 * The layer (paper Section 2.1, Fig. 1): a gating network scores every token
 * against E experts, each token goes to its top-k experts, every expert is an
 * FFN of two linear layers with one activation between, and expert outputs are
 * combined back in token order.  Experts that receive many tokens are "hot",
 * experts that receive few are "cold" and memory-bound (Section 2.2); the paper
 * sends the two classes to different hardware (Section 3.3).  On one GPU the
 * split selects between two kernel classes that both read weights from HBM:
 * a tensor-core grouped GEMM tiled for many tokens (hot) and a weight-streaming
 * kernel tiled for few tokens (cold).  The arithmetic result does not depend on
 * the class.
 *
 * Conventions for every call
 *  - All tensor pointers are DEVICE pointers owned by the caller.  The library
 *    allocates and frees no device memory.  Between calls it keeps nothing that a result
 *    depends on: only which devices have had their one-time kernel set-up, and a small
 *    cache of TMA descriptors keyed by address and shape (both under a mutex).  The
 *    switches of monde_diagnostics.h are process-wide state and off by default.
 *  - Tensors are row-major with the last index contiguous; base pointers are
 *    16-byte aligned (cudaMalloc-style 256-byte alignment recommended).
 *  - `stream` is a cudaStream_t cast to void* (NULL = the legacy default stream).
 *    Calls enqueue work and return; none synchronises or reads results back
 *    (except monde_poll_device_status, which exists to do exactly that).
 *  - Return value: a monde_status.  Argument errors are detected on the host
 *    before anything is launched.  Errors found on the device (a bounded wait
 *    that ran out) are recorded in a status word inside the workspace and
 *    reported by monde_poll_device_status.
 *  - T == 0 is valid: MONDE_OK, nothing launched.
 *  - Notation (paper Table 1): T = B*S tokens, d_model, d_ff, E experts;
 *    A = T*top_k assignments; an assignment id is a = t*top_k + j.
 *  - Limits: 1 <= top_k <= min(E, 8); E <= 256; T*top_k <= 2^20; bf16 path needs d_model and d_ff
 *    to be multiples of 64; fp32 path needs multiples of 4.
 */
#ifndef MONDE_H_
#define MONDE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MONDE_OK = 0,
    MONDE_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, top_k > E, misaligned pointer */
    MONDE_ERR_UNSUPPORTED = 2,  /* shape or dtype outside the stated limits */
    MONDE_ERR_WORKSPACE = 3,    /* ws_bytes smaller than monde_workspace_bytes() */
    MONDE_ERR_ARCH = 4,         /* current device is not compute capability 10.x */
    MONDE_ERR_CUDA = 5,         /* a CUDA runtime / driver call failed */
    MONDE_ERR_TIMEOUT = 6,      /* a bounded device-side wait gave up */
    MONDE_ERR_BOUNDS = 7        /* diagnostics build only: an index read from memory was out of range */
} monde_status;

typedef enum { MONDE_F32 = 0, MONDE_BF16 = 1 } monde_dtype;
typedef enum { MONDE_ACT_RELU = 0, MONDE_ACT_GELU_ERF = 1 } monde_act;

typedef struct {
    int32_t T;              /* tokens (B*S) */
    int32_t d_model;        /* embedding dimension */
    int32_t d_ff;           /* intra-FFN dimension */
    int32_t E;              /* experts */
    int32_t top_k;          /* experts per token */
    int32_t hot_threshold;  /* an expert with count >= hot_threshold is hot */
    int32_t renormalize;    /* 0: weight = softmax prob; 1: divided by the sum over the k selected */
    int32_t dtype;          /* monde_dtype of x, Wg, W1, b1, W2, b2, x_perm, y_perm, out */
    int32_t act;            /* monde_act */
} monde_problem;

/* Bytes of caller-provided device scratch that monde_route / monde_permute /
 * monde_moe_ffn_fwd need for this problem.  One buffer serves all three calls of a
 * layer; calls that share a buffer must be ordered on one stream.  The caller
 * zero-fills it ONCE after allocating it (it holds the sticky status word and
 * counters that every call leaves at zero again); its contents need not be
 * preserved otherwise.  Problems of different shapes may take turns on one buffer that
 * is large enough for each of them; calls that run at the same time (different streams)
 * need a buffer each.  Returns 0 for an invalid problem. */
size_t monde_workspace_bytes(const monde_problem* p);

const char* monde_status_string(int status);

/* Gate, softmax, top-k, histogram, hot/cold classification, scan.
 * Paper: Section 2.1 (gating function, token x expert score map, top-k routing);
 * Section 2.2 (hot / cold experts by token count); Section 3.3, Eq. 5 (an expert is
 * activated when it has at least one token).
 *   logits[t,e] = bg[e] + sum_i x[t,i]*Wg[e,i]   (fp32 accumulate, kept in fp32)
 *   probs[t,:]  = softmax(logits[t,:]) over all E
 *   topk_idx[t,0..k-1]: the k largest logits, best first, exact ties to the smaller id
 *   topk_w[t,j] = probs[t,idx]               (renormalize = 0)
 *               = probs[t,idx] / sum_j' probs[t,idx_j']   (renormalize = 1)
 *   counts[e]   = number of assignments to e;  offsets = exclusive scan, offsets[E] = A
 *   cls[e]      = 0 (no token), 1 (cold: 1 <= count < hot_threshold), 2 (hot)
 *   hot_ids / cold_ids: ascending expert ids of each class; n_hot_cold = {n_hot, n_cold}
 * in : x [T,d_model], Wg [E,d_model] (dtype); bg [E] fp32 or NULL
 * out: topk_idx [T,k] int32; topk_w [T,k] fp32; counts [E] int32; offsets [E+1] int32;
 *      cls [E] uint8; hot_ids [E], cold_ids [E] int32 (entries past n are left as is);
 *      n_hot_cold [2] int32; probs [T,E] fp32 or NULL.
 */
int monde_route(const monde_problem* p, const void* x, const void* Wg, const float* bg,
                int32_t* topk_idx, float* topk_w, int32_t* counts, int32_t* offsets,
                uint8_t* cls, int32_t* hot_ids, int32_t* cold_ids, int32_t* n_hot_cold,
                float* probs, void* ws, size_t ws_bytes, void* stream);

/* Hot / cold lists by the paper's own placement rule instead of a count threshold; run it after
 * monde_route to overwrite cls / hot_ids / cold_ids / n_hot_cold (counts, offsets and the
 * permutation do not depend on the classes).
 * Paper: Section 3.3, Eq. 3-6.  The H experts with the most tokens go to the engine whose cost is
 * fetching their weights (bandwidth BW_a; the GPU behind PCIe in the paper, the hot class here),
 * the rest to the engine that streams them in place (bandwidth BW_b; the near-data device in the
 * paper, the cold class here), with
 *     H = alpha * BW_a / (BW_b + BW_a) * Expert_Activ                                  (Eq. 6)
 * Expert_Activ = experts with at least one token (Eq. 5).  H is rounded down and clamped to
 * [0, Expert_Activ]; "most compute-intensive" = most tokens; equal counts: the smaller id is hotter;
 * experts without tokens stay class 0.  alpha is the paper's tuning factor (its auto-tuner tries
 * H, H+1, H+2 on recent batches and keeps the fastest).
 * in : counts [E] (device); alpha >= 0, bw_hot_feed (BW_a) > 0, bw_cold_feed (BW_b) > 0 (any common unit)
 * out: cls [E], hot_ids [E], cold_ids [E], n_hot_cold [2] as in monde_route
 */
int monde_classify_top_h(const monde_problem* p, const int32_t* counts, double alpha, double bw_hot_feed,
                         double bw_cold_feed, uint8_t* cls, int32_t* hot_ids, int32_t* cold_ids,
                         int32_t* n_hot_cold, void* stream);

/* Stable permutation of assignments into expert-contiguous order and row gather.
 * Paper: Section 2.1 (tokens routed to experts, later re-organised into the original
 * order); Section 4.1 (drop-less, padding-less routing: no capacity, no padded slot).
 *   pos(a) = offsets[e_a] + #{a' < a : e_a' = e_a};  perm[pos] = a;  inv_perm[a] = pos
 *   x_perm[pos,:] = x[a / top_k,:]
 * in : x [T,d_model]; topk_idx [T,k]; offsets [E+1]
 * out: perm [A], inv_perm [A] int32; x_perm [A,d_model] (dtype)
 */
int monde_permute(const monde_problem* p, const void* x, const int32_t* topk_idx,
                  const int32_t* offsets, int32_t* perm, int32_t* inv_perm, void* x_perm,
                  void* ws, size_t ws_bytes, void* stream);

/* Expert FFN on the expert-contiguous rows; hot experts on the tensor-core grouped
 * GEMM, cold experts on the weight-streaming kernel, same arithmetic for both.
 * Paper: Section 2.1 (an expert is two linear layers with an activation between);
 * Section 3.1 (C = A x B with A the routed tokens, B the expert parameters);
 * Section 3.4 (gemm and gemm+relu kernels; ReLU or GeLU); Section 3.3 (hot / cold
 * assignment to the hardware that suits each).
 *   for e with counts[e] > 0, rows r in [offsets[e], offsets[e+1]):
 *     h[r,:]      = act(x_perm[r,:] * W1[e]^T + b1[e])     (fp32 accumulate, stored in dtype)
 *     y_perm[r,:] = h[r,:] * W2[e]^T + b2[e]               (fp32 accumulate, stored in dtype)
 * Reads counts / offsets / classes from device memory; nothing comes back to the host.  cls, hot_ids,
 * cold_ids and n_hot_cold must describe the same classification (as monde_route and
 * monde_classify_top_h write them): a kernel may use either form.
 * in : x_perm [A,d_model]; W1 [E,d_ff,d_model]; b1 [E,d_ff] or NULL; W2 [E,d_model,d_ff];
 *      b2 [E,d_model] or NULL (all dtype); counts, offsets, cls, hot_ids, cold_ids,
 *      n_hot_cold as written by monde_route
 * out: y_perm [A,d_model] (dtype)
 */
int monde_moe_ffn_fwd(const monde_problem* p, const void* x_perm,
                      const void* W1, const void* b1, const void* W2, const void* b2,
                      const int32_t* counts, const int32_t* offsets, const uint8_t* cls,
                      const int32_t* hot_ids, const int32_t* cold_ids, const int32_t* n_hot_cold,
                      void* y_perm, void* ws, size_t ws_bytes, void* stream);

/* Gate-weighted combine back to token order (paper Section 2.1: expert outputs are
 * combined and re-organised into the original order of the input tokens).
 *   out[t,:] = sum_{j=0..k-1} topk_w[t,j] * y_perm[inv_perm[t*k+j],:]   (fp32, j ascending,
 *   rounded once to dtype)
 * in : y_perm [A,d_model] (dtype); inv_perm [A] int32; topk_w [T,k] fp32
 * out: out [T,d_model] (dtype)
 */
int monde_combine(const monde_problem* p, const void* y_perm, const int32_t* inv_perm,
                  const float* topk_w, void* out, void* stream);

/* Expert FFN and combine in one call, without a caller-side y_perm (bf16 problems).
 * Paper: Section 2.1 (expert outputs are weighted by the gate and re-organised into the original
 * token order); Section 3.4 (kernels fuse what follows a GEMM into it, as gemm+relu does).
 *   top_k == 1 (one expert per token: the sum over experts has a single term, so no order of
 *   additions is lost): the FFN's last store applies the gate weight and writes `out` directly,
 *     for rows r of expert e, t = perm[r]:
 *     out[t,:] = topk_w[t] * round_dtype(h[r,:] * W2[e]^T + b2[e])      (rounded once more to dtype)
 *   top_k > 1: the FFN's last store puts every output row at its assignment id perm[r] = t*top_k + j,
 *   so the top_k rows of a token lie side by side in a staging buffer inside the workspace, and the
 *   combine kernel then adds them in slot order (j ascending, fp32, one rounding) with no index
 *   look-up.
 * Either way `out` holds bit for bit what monde_moe_ffn_fwd followed by monde_combine writes.
 * Returns MONDE_ERR_UNSUPPORTED unless dtype is bf16.
 * in : as monde_moe_ffn_fwd (the class lists are not needed), perm [A] as written by
 *      monde_permute, topk_w [T,top_k] fp32
 * out: out [T,d_model] (dtype)
 */
int monde_moe_ffn_combine_fwd(const monde_problem* p, const void* x_perm,
                              const void* W1, const void* b1, const void* W2, const void* b2,
                              const int32_t* counts, const int32_t* offsets, const uint8_t* cls,
                              const int32_t* perm, const float* topk_w, void* out,
                              void* ws, size_t ws_bytes, void* stream);

/* Synchronises `stream`, then returns and clears the sticky device-side status word
 * kept in `ws` (MONDE_OK, or MONDE_ERR_TIMEOUT if a bounded wait inside a kernel gave
 * up; the outputs of that call are then undefined).  `site` (nullable, host pointer)
 * receives an implementation-defined code saying which wait gave up. */
int monde_poll_device_status(void* ws, void* stream, int32_t* site);

/* monde_moe_ffn_fwd for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, same arithmetic, same outputs.)
 *
 * Who needs it: a serving loop that allocates everything at start-up and forbids cudaMalloc
 * afterwards, a plug-in that is handed its input and output buffers and owns no allocator,
 * code that runs where growing a memory pool is not allowed.  Such a caller has nowhere to
 * get the workspace that monde_moe_ffn_fwd asks for, so this entry point uses a fixed
 * scratch array of MONDE_STATIC_WS_BYTES that is part of the library's device image.  The
 * call itself allocates and frees nothing.
 *
 *  - Arguments are those of monde_moe_ffn_fwd without ws / ws_bytes; inputs and outputs are
 *    still the caller's device buffers.
 *  - Limit: monde_workspace_bytes(p) must not exceed MONDE_STATIC_WS_BYTES; otherwise the call
 *    returns MONDE_ERR_WORKSPACE and launches nothing.  (Decode-sized batches fit: E=128,
 *    d_model=1024, d_ff=4096, T=32 needs about 26 MB; a 4096-token batch does not.)
 *  - Every GPU that loads the library holds the array from load until the process exits.
 *  - The first call on a device looks up the array's device address (once per device, with
 *    that device current).  Make that first call before any stream capture begins.
 *  - All calls on a GPU share the one array, and it keeps the previous call's contents; the
 *    entry point clears the parts that must start at zero (in stream order) before it
 *    launches.  Two calls that overlap on the GPU - different streams, or the same stream
 *    from two threads without ordering - race on the array and give undefined results:
 *    order them, or use monde_moe_ffn_fwd with separate workspaces.
 *  - Errors found on the device (a bounded wait that ran out) are recorded in the array's
 *    header.  The next call clears the header again, so a caller that wants to know must ask
 *    before it: monde_poll_static_ws_status.
 */
#define MONDE_STATIC_WS_BYTES (32u << 20)
int monde_moe_ffn_fwd_static_ws(const monde_problem* p, const void* x_perm,
                                const void* W1, const void* b1, const void* W2, const void* b2,
                                const int32_t* counts, const int32_t* offsets, const uint8_t* cls,
                                const int32_t* hot_ids, const int32_t* cold_ids, const int32_t* n_hot_cold,
                                void* y_perm, void* stream);

/* monde_poll_device_status for the built-in scratch array of monde_moe_ffn_fwd_static_ws (the
 * paper has no counterpart): synchronises `stream`, then returns and clears the status word that
 * the kernels of the last static-workspace call on the current device left in the array
 * (MONDE_OK, or MONDE_ERR_TIMEOUT with `site` as above; y_perm of that call is then undefined).
 * Allocates nothing.  Call it after the call it is asked about and before the next
 * static-workspace call on that GPU, which clears the word. */
int monde_poll_static_ws_status(void* stream, int32_t* site);

/* Diagnostic: number of kernels this library has launched in this process so far. */
long long monde_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* MONDE_H_ */
