// Stable counting-sort permutation of assignments into expert-contiguous order, fused
// with the row gather.  Deterministic: positions follow from counts alone, never from
// the order in which threads run.
// Paper: Section 2.1 (routing to experts); Section 4.1 (drop-less, padding-less).
#include "common.cuh"

namespace monde {

namespace {

constexpr int kChunk = 16;           // assignments per CTA, ranked by half a warp
constexpr int kThreads = 128;        // four warps, four rows each
constexpr int kRowsPerWarp = kChunk / (kThreads / 32);

// CTA c owns assignments [c*kChunk, (c+1)*kChunk).  The number of earlier assignments to
// each expert is recounted from topk_idx (at most A integers, L2-resident), which keeps
// the kernel single-pass and free of inter-CTA ordering.  Small chunks give many CTAs and
// every warp keeps the loads of its four rows in flight together, which is what matters
// for a decode-sized batch where the whole gather is a few dozen rows.
// Large batches: the recount of earlier assignments would grow quadratically, so it is cut at
// super-chunk boundaries.  `super_before` [n_super][E] holds, per expert, the number of assignments in
// all earlier super-chunks (two small kernels below build it); a CTA then recounts only from the start
// of its own super-chunk.  Null for small batches: recount from assignment 0.
constexpr int kSuper = 2048;         // assignments per super-chunk
constexpr int kTwoLevelFrom = 8192;  // batches with more assignments take the two-level path

__global__ void __launch_bounds__(256) super_histogram_kernel(int A, int E, const int32_t* __restrict__ topk_idx,
                                                              int32_t* __restrict__ super_before, DiagRecord* diag) {
    __shared__ int hist[kMaxExperts];
    pdl_launch_dependents();
    for (int e = threadIdx.x; e < kMaxExperts; e += blockDim.x) hist[e] = 0;
    __syncthreads();
    pdl_wait();
    const int first = blockIdx.x * kSuper;
    for (int a = first + threadIdx.x; a < min(A, first + kSuper); a += blockDim.x) {
        const int e = topk_idx[a];
        if (MONDE_IN_RANGE(e >= 0 && e < E, diag, 1, e)) atomicAdd(&hist[e], 1);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) super_before[static_cast<size_t>(blockIdx.x) * E + e] = hist[e];
}

// In place: counts per super-chunk -> exclusive prefix over super-chunks, one thread per expert.
__global__ void __launch_bounds__(256) super_scan_kernel(int n_super, int E, int32_t* __restrict__ super_before) {
    pdl_launch_dependents();
    pdl_wait();
    const int e = threadIdx.x;
    if (e >= E) return;
    int running = 0;
    for (int s = 0; s < n_super; ++s) {
        const int c = super_before[static_cast<size_t>(s) * E + e];
        super_before[static_cast<size_t>(s) * E + e] = running;
        running += c;
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads) permute_gather_kernel(
        int A, int E, int k, int d, const T* __restrict__ x, const int32_t* __restrict__ topk_idx,
        const int32_t* __restrict__ offsets, const int32_t* __restrict__ super_before,
        int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm, T* __restrict__ x_perm, DiagRecord* diag) {
    __shared__ int before[kMaxExperts];   // assignments to e in earlier chunks
    __shared__ int row_pos[kChunk];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int first = blockIdx.x * kChunk;
    pdl_launch_dependents();
    for (int e = tid; e < kMaxExperts; e += kThreads) before[e] = 0;
    __syncthreads();
    pdl_wait();
    // The rows this warp will copy are known before their positions are: their first vectors are
    // requested now, so that trip to memory overlaps the recount and the rank computation.
    constexpr int V = Vec16<T>::N;
    constexpr int kIter = 3;                         // vectors per lane and row in flight
    const int vec_per_row = d / V;
    const uint4* src[kRowsPerWarp];
    uint4 v[kIter][kRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r) {
        const int a = first + warp * kRowsPerWarp + r;
        src[r] = a < A ? reinterpret_cast<const uint4*>(x + static_cast<int64_t>(a / k) * d) : nullptr;
    }
#pragma unroll
    for (int it = 0; it < kIter; ++it)
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r)
            if (src[r] != nullptr && lane + 32 * it < vec_per_row) v[it][r] = src[r][lane + 32 * it];
    const int recount_from = super_before != nullptr ? (first / kSuper) * kSuper : 0;
    if (super_before != nullptr)
        for (int e = tid; e < E; e += kThreads) before[e] = super_before[static_cast<size_t>(first / kSuper) * E + e];
    __syncthreads();
    // Recount: the loads are batched (four 16-byte loads per thread in flight, 2048 assignments per
    // trip to L2) because the last chunks look back over thousands of assignments and a load per
    // loop iteration made them the critical path of the whole call.
    if ((reinterpret_cast<uintptr_t>(topk_idx) & 15) == 0) {
        const int4* src4 = reinterpret_cast<const int4*>(topk_idx + recount_from);   // both multiples of 16
        const int n4 = (first - recount_from) >> 2;
        for (int i = tid; i < n4; i += 4 * kThreads) {
            int4 v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int q = i + j * kThreads;
                v[j] = q < n4 ? __ldg(src4 + q) : make_int4(-1, -1, -1, -1);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (v[j].x < 0) continue;
                const int ev[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (MONDE_IN_RANGE(ev[i] >= 0 && ev[i] < E, diag, 1, ev[i])) atomicAdd(&before[ev[i]], 1);
            }
        }
    } else {
        for (int a = recount_from + tid; a < first; a += kThreads) {
            const int e = topk_idx[a];
            if (MONDE_IN_RANGE(e >= 0 && e < E, diag, 1, e)) atomicAdd(&before[e], 1);
        }
    }
    __syncthreads();
    if (warp == 0) {
        const int a = first + lane;
        int e = (lane < kChunk && a < A) ? topk_idx[a] : -1;
        if (e >= 0 && !MONDE_IN_RANGE(e < E, diag, 1, e)) e = -1;
        const unsigned same = __match_any_sync(0xffffffffu, e);
        int pos = -1;
        if (e >= 0) {
            pos = offsets[e] + before[e] + __popc(same & ((1u << lane) - 1u));
            if (MONDE_IN_RANGE(pos >= 0 && pos < A, diag, 2, pos)) {
                perm[pos] = a;
                inv_perm[a] = pos;
            } else {
                pos = -1;
            }
        }
        if (lane < kChunk) row_pos[lane] = pos;
    }
    __syncthreads();
    // Row gather with 16-byte accesses; the warp's rows advance together, kIter vectors per lane and
    // row requested before any is stored (one trip to memory per batch, not per vector).
    uint4* dst[kRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r) {
        const int p = row_pos[warp * kRowsPerWarp + r];
        dst[r] = p >= 0 ? reinterpret_cast<uint4*>(x_perm + static_cast<int64_t>(p) * d) : nullptr;
    }
    for (int i0 = lane; i0 < vec_per_row; i0 += 32 * kIter) {
        if (i0 != lane) {      // the first batch is already in registers
#pragma unroll
            for (int it = 0; it < kIter; ++it)
#pragma unroll
                for (int r = 0; r < kRowsPerWarp; ++r)
                    if (dst[r] != nullptr && i0 + 32 * it < vec_per_row) v[it][r] = src[r][i0 + 32 * it];
        }
#pragma unroll
        for (int it = 0; it < kIter; ++it)
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r)
                if (dst[r] != nullptr && i0 + 32 * it < vec_per_row) dst[r][i0 + 32 * it] = v[it][r];
    }
}

// out[t,:] = sum_j w[t,j] * y_perm[inv_perm[t*k+j],:]; one thread per 16-byte vector.
template <typename T>
__global__ void __launch_bounds__(256) combine_kernel(
        int T_tokens, int d, int k, const T* __restrict__ y_perm, const int32_t* __restrict__ inv_perm,
        const float* __restrict__ topk_w, T* __restrict__ out, DiagRecord* diag) {
    constexpr int V = Vec16<T>::N;
    const int vec_per_row = d / V;
    const int64_t g = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    if (g >= static_cast<int64_t>(T_tokens) * vec_per_row) return;
    const int64_t t = g / vec_per_row;
    const int c = static_cast<int>(g % vec_per_row) * V;
    float acc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = 0.0f;
    for (int j = 0; j < k; ++j) {
        const int pos = inv_perm != nullptr ? inv_perm[t * k + j] : static_cast<int>(t * k + j);   // null: rows already in token order
        const float w = topk_w[t * k + j];
        if (!MONDE_IN_RANGE(pos >= 0 && pos < T_tokens * k, diag, 3, pos)) continue;
        float y[V];
        Vec16<T>::load(y_perm + static_cast<int64_t>(pos) * d + c, y);
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = fmaf(w, y[v], acc[v]);
    }
    Vec16<T>::store(out + t * d + c, acc);
}

}  // namespace

int launch_permute(const monde_problem& p, const void* x, const int32_t* topk_idx, const int32_t* offsets,
                   int32_t* perm, int32_t* inv_perm, void* x_perm, const void* ws, cudaStream_t s) {
    // scratch for the two-level recount: ceil(A / 2048) * E int32 in the hidden-activation region, which is dead
    // during this call (the expert FFN rewrites it before reading it)
    int32_t* scratch = reinterpret_cast<int32_t*>(static_cast<char*>(const_cast<void*>(ws)) + WsLayout::kHidden);
    const int A = p.T * p.top_k;
    const int grid = (A + kChunk - 1) / kChunk;
    int32_t* super_before = nullptr;
    if (A > kTwoLevelFrom) {
        const int n_super = (A + kSuper - 1) / kSuper;
        super_before = scratch;      // n_super * E int32
        launch_pdl(super_histogram_kernel, dim3(n_super), dim3(256), 0, s, A, p.E, topk_idx, super_before,
                   diag_record_ptr());
        launch_pdl(super_scan_kernel, dim3(1), dim3(256), 0, s, n_super, p.E, super_before);
        count_launches(2);
    }
    if (p.dtype == MONDE_BF16)
        launch_pdl(permute_gather_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), 0, s,
            A, p.E, p.top_k, p.d_model, static_cast<const __nv_bfloat16*>(x), topk_idx, offsets, super_before, perm,
            inv_perm, static_cast<__nv_bfloat16*>(x_perm), diag_record_ptr());
    else
        launch_pdl(permute_gather_kernel<float>, dim3(grid), dim3(kThreads), 0, s,
            A, p.E, p.top_k, p.d_model, static_cast<const float*>(x), topk_idx, offsets, super_before, perm, inv_perm,
            static_cast<float*>(x_perm), diag_record_ptr());
    return launched();
}

int launch_combine(const monde_problem& p, const void* y_perm, const int32_t* inv_perm,
                   const float* topk_w, void* out, cudaStream_t s) {
    const int V = p.dtype == MONDE_BF16 ? 8 : 4;
    const int64_t n = static_cast<int64_t>(p.T) * (p.d_model / V);
    const int grid = static_cast<int>((n + 255) / 256);
    if (p.dtype == MONDE_BF16)
        launch_pdl(combine_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, s,
            p.T, p.d_model, p.top_k, static_cast<const __nv_bfloat16*>(y_perm), inv_perm, topk_w,
            static_cast<__nv_bfloat16*>(out), diag_record_ptr());
    else
        launch_pdl(combine_kernel<float>, dim3(grid), dim3(256), 0, s, p.T, p.d_model, p.top_k, static_cast<const float*>(y_perm),
                                                   inv_perm, topk_w, static_cast<float*>(out), diag_record_ptr());
    return launched();
}

}  // namespace monde
