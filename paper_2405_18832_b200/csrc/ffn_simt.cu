// Plain CUDA-core expert linear layer: Out[r,n] = act?(bias[e,n] + sum_k In[r,k]*W[e,n,k]).
// This is the arithmetic path of fp32 problems (tensor cores would round fp32 inputs),
// and a debugging aid that can stand in for the tensor-core kernels on bf16 problems.
// Paper: Section 2.1 (expert = two linear layers and an activation); Section 3.4
// (gemm / gemm+relu kernels).
#include "common.cuh"

namespace monde {

namespace {

constexpr int kRows = 8;    // rows of the expert's segment handled per pass
constexpr int kWarps = 8;   // output features per CTA (one per warp)

template <typename T>
__global__ void __launch_bounds__(kWarps * 32) linear_simt_kernel(
        int act, int K, int N, const T* __restrict__ in, const T* __restrict__ W, const T* __restrict__ bias,
        const int32_t* __restrict__ offsets, const int32_t* __restrict__ ids, const int32_t* __restrict__ n_ids,
        T* __restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    if (static_cast<int>(blockIdx.y) >= *n_ids) return;
    constexpr int V = Vec16<T>::N;
    const int e = ids[blockIdx.y];
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (n >= N) return;
    const int row_begin = offsets[e], row_end = offsets[e + 1];
    const T* w = W + (static_cast<int64_t>(e) * N + n) * K;
    const float b = bias != nullptr ? to_float(bias[static_cast<int64_t>(e) * N + n]) : 0.0f;
    for (int r0 = row_begin; r0 < row_end; r0 += kRows) {
        float acc[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) acc[r] = 0.0f;
        for (int i = lane * V; i < K; i += 32 * V) {
            float wv[V];
            Vec16<T>::load(w + i, wv);
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                if (r0 + r < row_end) {
                    float xv[V];
                    Vec16<T>::load(in + static_cast<int64_t>(r0 + r) * K + i, xv);
#pragma unroll
                    for (int v = 0; v < V; ++v) acc[r] = fmaf(xv[v], wv[v], acc[r]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], o);
        }
        if (lane < kRows && r0 + lane < row_end) {
            float v = 0.0f;
#pragma unroll
            for (int r = 0; r < kRows; ++r) if (lane == r) v = acc[r];
            v += b;
            if (act >= 0) v = apply_act(v, act);
            out[static_cast<int64_t>(r0 + lane) * N + n] = from_float<T>(v);
        }
    }
}

}  // namespace

int launch_linear_simt(int dtype, int act_or_neg1, int E, int K, int N, const void* in, const void* W,
                       const void* bias, const int32_t* offsets, const int32_t* ids, const int32_t* n_ids,
                       void* out, cudaStream_t s) {
    dim3 grid((N + kWarps - 1) / kWarps, E);
    if (dtype == MONDE_BF16)
        launch_pdl(linear_simt_kernel<__nv_bfloat16>, grid, dim3(kWarps * 32), 0, s,
            act_or_neg1, K, N, static_cast<const __nv_bfloat16*>(in), static_cast<const __nv_bfloat16*>(W),
            static_cast<const __nv_bfloat16*>(bias), offsets, ids, n_ids, static_cast<__nv_bfloat16*>(out));
    else
        launch_pdl(linear_simt_kernel<float>, grid, dim3(kWarps * 32), 0, s,
            act_or_neg1, K, N, static_cast<const float*>(in), static_cast<const float*>(W),
            static_cast<const float*>(bias), offsets, ids, n_ids, static_cast<float*>(out));
    return launched();
}

}  // namespace monde
