// Gate GEMM + softmax + top-k (one warp per token, warp-shuffle reductions), and the
// shared-memory histogram / hot-cold classification / scan over experts.
// Paper: Section 2.1 (gating network, score map, top-k routing); Section 2.2 (hot and
// cold experts by token count); Eq. 5 (activated = at least one token).
#include "common.cuh"

namespace monde {

namespace {

constexpr int kSlots = kMaxExperts / 32;  // logits per lane: expert e lives in lane e%32, slot e/32

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

// Softmax over all E logits and the k best of them, for one token held by one warp.
// logit[s] of lane l is expert s*32+l (-inf beyond E).
__device__ __forceinline__ void softmax_topk_store(const float (&logit)[kSlots], int E, int k, int renorm,
                                                   int64_t t, int lane, int32_t* __restrict__ topk_idx,
                                                   float* __restrict__ topk_w, float* __restrict__ probs) {
    float m = -INFINITY;
#pragma unroll
    for (int s = 0; s < kSlots; ++s) m = fmaxf(m, logit[s]);
    m = warp_max(m);
    float ex[kSlots];
    float denom = 0.0f;
#pragma unroll
    for (int s = 0; s < kSlots; ++s) {
        ex[s] = (s * 32 + lane < E) ? expf(logit[s] - m) : 0.0f;
        denom += ex[s];
    }
    denom = warp_sum(denom);
    if (probs != nullptr) {
#pragma unroll
        for (int s = 0; s < kSlots; ++s)
            if (s * 32 + lane < E) probs[t * E + s * 32 + lane] = ex[s] / denom;
    }
    uint32_t taken = 0;
    float sel_p[kMaxTopK];
    int sel_e[kMaxTopK];
    float mass = 0.0f;
#pragma unroll
    for (int j = 0; j < kMaxTopK; ++j) {
        if (j < k) {
            float bv = -INFINITY;
            int be = 0x7fffffff;
            float bp = 0.0f;
#pragma unroll
            for (int s = 0; s < kSlots; ++s) {
                const int e = s * 32 + lane;
                if (e < E && !((taken >> s) & 1u) && (logit[s] > bv || be == 0x7fffffff)) {
                    bv = logit[s]; be = e; bp = ex[s];
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oe = __shfl_xor_sync(0xffffffffu, be, o);
                const float op = __shfl_xor_sync(0xffffffffu, bp, o);
                if (oe != 0x7fffffff && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be))) {
                    bv = ov; be = oe; bp = op;
                }
            }
            if ((be & 31) == lane) taken |= 1u << (be >> 5);
            sel_e[j] = be;
            sel_p[j] = bp / denom;
            mass += sel_p[j];
        }
    }
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < kMaxTopK; ++j) {
            if (j < k) {
                topk_idx[t * k + j] = sel_e[j];
                topk_w[t * k + j] = renorm ? sel_p[j] / mass : sel_p[j];
            }
        }
    }
}

// One warp per token; lanes split d_model with 16-byte loads.
template <typename T>
__global__ void __launch_bounds__(128) route_warp_per_token_kernel(
        int T_tokens, int d, int E, int k, int renorm, const T* __restrict__ x, const T* __restrict__ Wg,
        const float* __restrict__ bg, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
        float* __restrict__ probs) {
    constexpr int V = Vec16<T>::N;
    const int lane = threadIdx.x & 31;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T_tokens) return;
    const T* xr = x + t * d;
    float logit[kSlots];
#pragma unroll
    for (int s = 0; s < kSlots; ++s) logit[s] = -INFINITY;
#pragma unroll
    for (int s = 0; s < kSlots; ++s) {
        if (s * 32 < E) {
            for (int le = 0; le < 32 && s * 32 + le < E; ++le) {
                const int e = s * 32 + le;
                const T* wr = Wg + static_cast<int64_t>(e) * d;
                float acc = 0.0f;
                for (int i = lane * V; i < d; i += 32 * V) {
                    float a[V], b[V];
                    Vec16<T>::load(xr + i, a);
                    Vec16<T>::load(wr + i, b);
#pragma unroll
                    for (int v = 0; v < V; ++v) acc = fmaf(a[v], b[v], acc);
                }
                acc = warp_sum(acc);
                if (bg != nullptr) acc += bg[e];
                if (lane == le) logit[s] = acc;
            }
        }
    }
    softmax_topk_store(logit, E, k, renorm, t, lane, topk_idx, topk_w, probs);
}

// Histogram of assignments per expert (shared-memory atomics on integers: the sum does
// not depend on order), then classification, compaction and exclusive scan by one warp.
__global__ void __launch_bounds__(1024) histogram_classify_scan_kernel(
        int A, int E, int theta, const int32_t* __restrict__ topk_idx, int32_t* __restrict__ counts,
        int32_t* __restrict__ offsets, uint8_t* __restrict__ cls, int32_t* __restrict__ hot_ids,
        int32_t* __restrict__ cold_ids, int32_t* __restrict__ n_hot_cold) {
    __shared__ int hist[kMaxExperts];
    for (int e = threadIdx.x; e < kMaxExperts; e += blockDim.x) hist[e] = 0;
    __syncthreads();
    for (int a = threadIdx.x; a < A; a += blockDim.x) atomicAdd(&hist[topk_idx[a]], 1);
    __syncthreads();
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    // lane owns experts [lane*8, lane*8+8)
    int c[kSlots], sum = 0, nh = 0, nc = 0;
#pragma unroll
    for (int i = 0; i < kSlots; ++i) {
        const int e = lane * kSlots + i;
        c[i] = e < E ? hist[e] : 0;
        sum += c[i];
        nh += (c[i] > 0 && c[i] >= theta);
        nc += (c[i] > 0 && c[i] < theta);
    }
    int ps = sum, ph = nh, pc = nc;   // inclusive scans across lanes
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, ps, o);
        const int b = __shfl_up_sync(0xffffffffu, ph, o);
        const int d = __shfl_up_sync(0xffffffffu, pc, o);
        if (lane >= o) { ps += a; ph += b; pc += d; }
    }
    int off = ps - sum, ih = ph - nh, ic = pc - nc;
#pragma unroll
    for (int i = 0; i < kSlots; ++i) {
        const int e = lane * kSlots + i;
        if (e < E) {
            counts[e] = c[i];
            offsets[e] = off;
            uint8_t k = 0;
            if (c[i] > 0) {
                if (c[i] >= theta) { k = 2; hot_ids[ih++] = e; }
                else { k = 1; cold_ids[ic++] = e; }
            }
            cls[e] = k;
            off += c[i];
        }
    }
    if (lane == 31) {
        offsets[E] = ps;
        n_hot_cold[0] = ph;
        n_hot_cold[1] = pc;
    }
}

}  // namespace

int launch_route(const monde_problem& p, const void* x, const void* Wg, const float* bg,
                 int32_t* topk_idx, float* topk_w, float* probs, cudaStream_t s) {
    const int warps = 4;
    const int grid = (p.T + warps - 1) / warps;
    if (p.dtype == MONDE_BF16)
        route_warp_per_token_kernel<__nv_bfloat16><<<grid, warps * 32, 0, s>>>(
            p.T, p.d_model, p.E, p.top_k, p.renormalize, static_cast<const __nv_bfloat16*>(x),
            static_cast<const __nv_bfloat16*>(Wg), bg, topk_idx, topk_w, probs);
    else
        route_warp_per_token_kernel<float><<<grid, warps * 32, 0, s>>>(
            p.T, p.d_model, p.E, p.top_k, p.renormalize, static_cast<const float*>(x),
            static_cast<const float*>(Wg), bg, topk_idx, topk_w, probs);
    return launched();
}

int launch_histogram_classify_scan(const monde_problem& p, const int32_t* topk_idx, int32_t* counts,
                                   int32_t* offsets, uint8_t* cls, int32_t* hot_ids, int32_t* cold_ids,
                                   int32_t* n_hot_cold, cudaStream_t s) {
    histogram_classify_scan_kernel<<<1, 1024, 0, s>>>(p.T * p.top_k, p.E, p.hot_threshold, topk_idx, counts,
                                                      offsets, cls, hot_ids, cold_ids, n_hot_cold);
    return launched();
}

}  // namespace monde
