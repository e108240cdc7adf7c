// Stable counting-sort permutation of assignments into expert-contiguous order, fused
// with the row gather.  Deterministic: positions follow from counts alone, never from
// the order in which threads run.  The counts per 16-token chunk come from the router.
// Paper: Section 2.1 (routing to experts); Section 4.1 (drop-less, padding-less).
#include "common.cuh"

namespace monde {

namespace {

constexpr int kThreads = 128;        // four warps
constexpr int kRowsPerWarp = 4;      // rows a warp copies together
constexpr int kMaxChunkRows = kChunkTokens * kMaxTopK;   // assignments of one chunk

// CTA c owns the assignments of chunk c (16 tokens, 16 * k assignments), the same chunks the router
// CTAs own.  The position of assignment a with expert e is
//     offsets[e] + (assignments to e in earlier super-chunks)           <- super_before, from the router's tail
//                + (assignments to e in earlier chunks of this super-chunk)   <- at most 15 one-byte counts
//                + (earlier assignments to e inside this chunk)         <- compared in shared memory
// every term an integer read or counted in a fixed way: positions never depend on the order in which
// threads or CTAs run, and no CTA looks at another chunk's assignment list.
template <typename T>
__global__ void __launch_bounds__(kThreads) permute_gather_kernel(
        int A, int E, int k, int d, const T* __restrict__ x, const int32_t* __restrict__ topk_idx,
        const int32_t* __restrict__ offsets, const uint8_t* __restrict__ chunk_counts,
        const int32_t* __restrict__ super_before, int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
        T* __restrict__ x_perm) {
    __shared__ int s_e[kMaxChunkRows];
    __shared__ int s_pos[kMaxChunkRows];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk = blockIdx.x;
    const int rows_per_chunk = kChunkTokens * k;
    const int first = chunk * rows_per_chunk;
    const int n_rows = min(rows_per_chunk, A - first);
    pdl_launch_dependents();
    pdl_wait();
    // The rows this warp will copy are known before their positions are: the first vectors of its first
    // rows are requested now, so that trip to memory overlaps the position computation.
    constexpr int V = Vec16<T>::N;
    constexpr int kIter = 3;                         // vectors per lane and row in flight
    const int vec_per_row = d / V;
    const uint4* src[kRowsPerWarp];
    uint4 v[kIter][kRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r) {
        const int a = warp * kRowsPerWarp + r;       // row of the chunk
        src[r] = a < n_rows ? reinterpret_cast<const uint4*>(x + static_cast<int64_t>((first + a) / k) * d) : nullptr;
    }
#pragma unroll
    for (int it = 0; it < kIter; ++it)
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r)
            if (src[r] != nullptr && lane + 32 * it < vec_per_row) v[it][r] = src[r][lane + 32 * it];
    // positions: thread a handles assignment first + a
    int e = -1, base = 0;
    if (tid < n_rows) {
        e = topk_idx[first + tid];
        const int sc = chunk / kSuperChunks, c0 = sc * kSuperChunks;
        base = offsets[e] + super_before[static_cast<size_t>(sc) * E + e];
        int earlier = 0;
#pragma unroll
        for (int c = 0; c < kSuperChunks - 1; ++c)    // independent one-byte loads: one trip to L2
            earlier += c0 + c < chunk ? static_cast<int>(__ldg(chunk_counts + static_cast<size_t>(c0 + c) * E + e)) : 0;
        base += earlier;
    }
    if (tid < kMaxChunkRows) s_e[tid] = e;
    __syncthreads();
    if (tid < n_rows) {
        int rank = 0;
        for (int a = 0; a < tid; ++a) rank += s_e[a] == e;
        const int pos = base + rank;
        perm[pos] = first + tid;
        inv_perm[first + tid] = pos;
        s_pos[tid] = pos;
    }
    __syncthreads();
    // Row gather with 16-byte accesses; a warp's rows advance together, kIter vectors per lane and
    // row requested before any is stored (one trip to memory per batch, not per vector).
    for (int r0 = warp * kRowsPerWarp; r0 < n_rows; r0 += (kThreads / 32) * kRowsPerWarp) {
        uint4* dst[kRowsPerWarp];
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r) {
            const int a = r0 + r;
            dst[r] = a < n_rows ? reinterpret_cast<uint4*>(x_perm + static_cast<int64_t>(s_pos[a]) * d) : nullptr;
            if (r0 != warp * kRowsPerWarp)           // later row groups (k > 1): their sources were not set up above
                src[r] = a < n_rows ? reinterpret_cast<const uint4*>(x + static_cast<int64_t>((first + a) / k) * d) : nullptr;
        }
        for (int i0 = lane; i0 < vec_per_row; i0 += 32 * kIter) {
            if (i0 != lane || r0 != warp * kRowsPerWarp) {      // the very first batch is already in registers
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
}

// out[t,:] = sum_j w[t,j] * y_perm[inv_perm[t*k+j],:]; one thread per 16-byte vector.
template <typename T>
__global__ void __launch_bounds__(256) combine_kernel(
        int T_tokens, int d, int k, const T* __restrict__ y_perm, const int32_t* __restrict__ inv_perm,
        const float* __restrict__ topk_w, T* __restrict__ out) {
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
    const int A = p.T * p.top_k;
    const WsLayout L = ws_layout(p);
    const char* base = static_cast<const char*>(ws);
    const uint8_t* chunk_counts = reinterpret_cast<const uint8_t*>(base + L.chunk_counts_off);
    const int32_t* super_before = reinterpret_cast<const int32_t*>(base + L.super_before_off);
    if (p.dtype == MONDE_BF16)
        launch_pdl(permute_gather_kernel<__nv_bfloat16>, dim3(L.n_chunks), dim3(kThreads), 0, s,
            A, p.E, p.top_k, p.d_model, static_cast<const __nv_bfloat16*>(x), topk_idx, offsets, chunk_counts,
            super_before, perm, inv_perm, static_cast<__nv_bfloat16*>(x_perm));
    else
        launch_pdl(permute_gather_kernel<float>, dim3(L.n_chunks), dim3(kThreads), 0, s,
            A, p.E, p.top_k, p.d_model, static_cast<const float*>(x), topk_idx, offsets, chunk_counts, super_before,
            perm, inv_perm, static_cast<float*>(x_perm));
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
            static_cast<__nv_bfloat16*>(out));
    else
        launch_pdl(combine_kernel<float>, dim3(grid), dim3(256), 0, s, p.T, p.d_model, p.top_k, static_cast<const float*>(y_perm),
                                                   inv_perm, topk_w, static_cast<float*>(out));
    return launched();
}

}  // namespace monde
