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

struct HistArgs {
    int A, E, theta;
    int32_t* counts;
    int32_t* offsets;
    uint8_t* cls;
    int32_t* hot_ids;
    int32_t* cold_ids;
    int32_t* n_hot_cold;
    int32_t* ticket;      // CTAs of the router that have finished (left at zero)
};

// Histogram of assignments per expert (shared-memory atomics on integers: the sum does
// not depend on order), then classification, compaction and exclusive scan by one warp.
// Runs in one CTA of any size.
__device__ void histogram_classify_scan(const HistArgs& h, const int32_t* __restrict__ topk_idx, int* hist) {
    for (int e = threadIdx.x; e < kMaxExperts; e += blockDim.x) hist[e] = 0;
    __syncthreads();
    // The loads are batched (four 16-byte loads per thread in flight): this runs in the last CTA
    // alone, after everything else, and one load per loop iteration would put A / blockDim.x trips
    // to L2 on the critical path of the call.
    const int A4 = (reinterpret_cast<uintptr_t>(topk_idx) & 15) == 0 ? h.A >> 2 : 0;
    const int4* idx4 = reinterpret_cast<const int4*>(topk_idx);
    for (int i = threadIdx.x; i < A4; i += 4 * blockDim.x) {
        int4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int q = i + j * blockDim.x;
            v[j] = q < A4 ? __ldcg(idx4 + q) : make_int4(-1, -1, -1, -1);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (v[j].x < 0) continue;
            atomicAdd(&hist[v[j].x], 1);
            atomicAdd(&hist[v[j].y], 1);
            atomicAdd(&hist[v[j].z], 1);
            atomicAdd(&hist[v[j].w], 1);
        }
    }
    for (int a = A4 * 4 + threadIdx.x; a < h.A; a += blockDim.x) atomicAdd(&hist[__ldcg(topk_idx + a)], 1);
    __syncthreads();
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    // lane owns experts [lane*8, lane*8+8)
    int c[kSlots], sum = 0, nh = 0, nc = 0;
#pragma unroll
    for (int i = 0; i < kSlots; ++i) {
        const int e = lane * kSlots + i;
        c[i] = e < h.E ? hist[e] : 0;
        sum += c[i];
        nh += (c[i] > 0 && c[i] >= h.theta);
        nc += (c[i] > 0 && c[i] < h.theta);
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
        if (e < h.E) {
            h.counts[e] = c[i];
            h.offsets[e] = off;
            uint8_t k = 0;
            if (c[i] > 0) {
                if (c[i] >= h.theta) { k = 2; h.hot_ids[ih++] = e; }
                else { k = 1; h.cold_ids[ic++] = e; }
            }
            h.cls[e] = k;
            off += c[i];
        }
    }
    if (lane == 31) {
        h.offsets[h.E] = ps;
        h.n_hot_cold[0] = ph;
        h.n_hot_cold[1] = pc;
    }
}

// Called by every thread of every router CTA after its top-k stores: the CTA that finishes
// last runs the histogram, so routing is one launch.
__device__ void finish_route(const HistArgs& h, const int32_t* topk_idx, int finishers = 0) {
    __shared__ int s_hist[kMaxExperts];
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (finishers == 0) finishers = static_cast<int>(gridDim.x);     // default: every CTA of the launch arrives
    if (threadIdx.x == 0) s_last = atomicAdd(h.ticket, 1) == finishers - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (threadIdx.x == 0) *h.ticket = 0;
    histogram_classify_scan(h, topk_idx, s_hist);
}

// Stand-alone form, used when there are no tokens (every count is zero).
__global__ void __launch_bounds__(256) histogram_only_kernel(HistArgs h, const int32_t* topk_idx) {
    __shared__ int s_hist[kMaxExperts];
    pdl_launch_dependents();
    pdl_wait();
    histogram_classify_scan(h, topk_idx, s_hist);
}

// One warp per token; lanes split d_model with 16-byte loads.
template <typename T>
__global__ void __launch_bounds__(128) route_warp_per_token_kernel(
        int T_tokens, int d, int E, int k, int renorm, const T* __restrict__ x, const T* __restrict__ Wg,
        const float* __restrict__ bg, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
        float* __restrict__ probs, const HistArgs hist) {
    constexpr int V = Vec16<T>::N;
    const int lane = threadIdx.x & 31;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    pdl_launch_dependents();
    pdl_wait();
    if (t < T_tokens) {
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
    finish_route(hist, topk_idx);
}

// ---- bf16 gate on the warp-level tensor-core path -------------------------------------
// CTA = 16 tokens x all experts; each of the 4 warps owns a contiguous quarter of the
// (padded) expert range as 8-wide MMA column tiles.  Fragments are loaded straight from
// global memory with 16-byte loads: lane (g, t) reads 8 consecutive k of row g, which
// feeds the k-slots of two m16n8k16 MMAs.  The k index inside an MMA is permuted the same
// way for both operands, which leaves every dot product unchanged.  Products of two bf16
// values are exact in fp32 and accumulation is fp32, so logits keep fp32 accuracy.
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// kTilesPerWarp: 8-expert column tiles per warp, padded E = 32 * kTilesPerWarp.  kDeep: grids of at most
// one CTA per SM keep the loads of several K steps in flight (about 128 registers); larger grids keep
// two CTAs per SM (64 registers) and load a step at a time.
template <int kTilesPerWarp, bool kDeep>
__global__ void __launch_bounds__(512, (kDeep || kTilesPerWarp >= 8) ? 1 : 2) route_mma_kernel(
        int T_tokens, int d, int E, int k, int renorm, const __nv_bfloat16* __restrict__ x,
        const __nv_bfloat16* __restrict__ Wg, const float* __restrict__ bg, int32_t* __restrict__ topk_idx,
        float* __restrict__ topk_w, float* __restrict__ probs, const HistArgs hist) {
    // 16 warps = 4 expert quarters x 4 interleaved K quarters: many independent loads in flight
    // per CTA, which is what a 32-token decode batch (two CTAs in the whole grid) needs.
    constexpr int kEPad = 32 * kTilesPerWarp;
    constexpr int kRow = kEPad + 1;
    extern __shared__ float s_part[];                 // [4 K quarters][16 tokens][kRow]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int eq = warp & 3, kq = warp >> 2;
    const int g = lane >> 2, t4 = lane & 3;
    const int tok0 = blockIdx.x * 16;
    pdl_launch_dependents();
    pdl_wait();
    const int r0 = min(tok0 + g, T_tokens - 1), r1 = min(tok0 + g + 8, T_tokens - 1);
    const uint4* xa = reinterpret_cast<const uint4*>(x + static_cast<int64_t>(r0) * d) + t4;
    const uint4* xb = reinterpret_cast<const uint4*>(x + static_cast<int64_t>(r1) * d) + t4;
    const uint4* wp[kTilesPerWarp];
#pragma unroll
    for (int j = 0; j < kTilesPerWarp; ++j) {
        const int e = min(eq * (8 * kTilesPerWarp) + j * 8 + g, E - 1);
        wp[j] = reinterpret_cast<const uint4*>(Wg + static_cast<int64_t>(e) * d) + t4;
    }
    float acc[kTilesPerWarp][4];
#pragma unroll
    for (int j = 0; j < kTilesPerWarp; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[j][i] = 0.0f;
    const int steps = d / 32;               // 32 k per step: 4 lanes x 8 elements
    // Loads of several steps are issued together and the MMAs follow: a step at a time would put one
    // trip to memory per step on the critical path of a kernel that is all latency.
    constexpr int kBatch = (!kDeep || kTilesPerWarp >= 8) ? 1 : 20 / (2 + kTilesPerWarp);   // about 80 registers of loads in flight
    for (int s0 = kq; s0 < steps; s0 += 4 * kBatch) {
        uint4 a[kBatch], b[kBatch], w[kBatch][kTilesPerWarp];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int s = s0 + 4 * i;
            if (s < steps) {
                a[i] = xa[s * 4];
                b[i] = xb[s * 4];
#pragma unroll
                for (int j = 0; j < kTilesPerWarp; ++j) w[i][j] = wp[j][s * 4];
            }
        }
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            if (s0 + 4 * i < steps) {
#pragma unroll
                for (int j = 0; j < kTilesPerWarp; ++j) {
                    mma_bf16_16816(acc[j], a[i].x, b[i].x, a[i].y, b[i].y, w[i][j].x, w[i][j].y);
                    mma_bf16_16816(acc[j], a[i].z, b[i].z, a[i].w, b[i].w, w[i][j].z, w[i][j].w);
                }
            }
        }
    }
    float* part = s_part + kq * (16 * kRow);
#pragma unroll
    for (int j = 0; j < kTilesPerWarp; ++j) {
        const int e = eq * (8 * kTilesPerWarp) + j * 8 + t4 * 2;
        part[g * kRow + e] = acc[j][0];
        part[g * kRow + e + 1] = acc[j][1];
        part[(g + 8) * kRow + e] = acc[j][2];
        part[(g + 8) * kRow + e + 1] = acc[j][3];
    }
    __syncthreads();
    const int64_t t = tok0 + warp;          // one warp per token for softmax and top-k
    if (t < T_tokens) {
        float logit[kSlots];
#pragma unroll
        for (int s = 0; s < kSlots; ++s) {
            const int e = s * 32 + lane;
            if (s < kTilesPerWarp && e < E) {
                const float* p = s_part + warp * kRow + e;    // K quarters summed in a fixed order
                logit[s] = ((p[0] + p[16 * kRow]) + (p[32 * kRow] + p[48 * kRow])) + (bg != nullptr ? bg[e] : 0.0f);
            } else {
                logit[s] = -INFINITY;
            }
        }
        softmax_topk_store(logit, E, k, renorm, t, lane, topk_idx, topk_w, probs);
    }
    finish_route(hist, topk_idx);
}

// ---- small batches: the gate GEMM dealt over (chunk, 8 experts) CTAs -----------------------------
// A batch of a few dozen tokens has one or two 16-token chunks; with one CTA per chunk a decode step
// would read the whole gate matrix through one or two SMs.  Here CTA (chunk c, octet o) computes the
// logits of 16 tokens against experts [8o, 8o+8): its 16 warps split K sixteen ways (all loads of
// the CTA are in flight together: one trip to memory), partial sums meet in shared memory and are
// added in warp order, and the 16 x 8 logits go to the workspace.  The CTA that completes a chunk's
// logits (per-chunk ticket) runs softmax and top-k for the chunk, then the usual tail.
__global__ void __launch_bounds__(512, 1) route_split_kernel(
        int T_tokens, int d, int E, int k, int renorm, const __nv_bfloat16* __restrict__ x,
        const __nv_bfloat16* __restrict__ Wg, const float* __restrict__ bg, int32_t* __restrict__ topk_idx,
        float* __restrict__ topk_w, float* __restrict__ probs, float* __restrict__ logits_ws,
        int32_t* __restrict__ tile_tickets, const HistArgs hist) {
    __shared__ float s_part[16][16][9];            // [warp][token][expert of the octet]
    __shared__ int s_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t4 = lane & 3;
    const int chunk = blockIdx.x, oct = blockIdx.y, n_oct = gridDim.y;
    const int tok0 = chunk * 16;
    pdl_launch_dependents();
    pdl_wait();
    const int r0 = min(tok0 + g, T_tokens - 1), r1 = min(tok0 + g + 8, T_tokens - 1);
    const uint4* xa = reinterpret_cast<const uint4*>(x + static_cast<int64_t>(r0) * d) + t4;
    const uint4* xb = reinterpret_cast<const uint4*>(x + static_cast<int64_t>(r1) * d) + t4;
    const uint4* wp = reinterpret_cast<const uint4*>(Wg + static_cast<int64_t>(min(oct * 8 + g, E - 1)) * d) + t4;
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    const int steps = d / 32;               // 32 k per step: 4 lanes x 8 elements; warp w takes steps w, w+16, ...
    constexpr int kBatch = 4;
    for (int s0 = warp; s0 < steps; s0 += 16 * kBatch) {
        uint4 a[kBatch], b[kBatch], w[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int sidx = s0 + 16 * i;
            if (sidx < steps) {
                a[i] = xa[sidx * 4];
                b[i] = xb[sidx * 4];
                w[i] = wp[sidx * 4];
            }
        }
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            if (s0 + 16 * i < steps) {
                mma_bf16_16816(acc, a[i].x, b[i].x, a[i].y, b[i].y, w[i].x, w[i].y);
                mma_bf16_16816(acc, a[i].z, b[i].z, a[i].w, b[i].w, w[i].z, w[i].w);
            }
        }
    }
    s_part[warp][g][t4 * 2] = acc[0];
    s_part[warp][g][t4 * 2 + 1] = acc[1];
    s_part[warp][g + 8][t4 * 2] = acc[2];
    s_part[warp][g + 8][t4 * 2 + 1] = acc[3];
    __syncthreads();
    if (threadIdx.x < 128) {               // 16 tokens x 8 experts, the 16 K slices added in warp order
        const int tk = threadIdx.x >> 3, eo = threadIdx.x & 7;
        float sum = 0.0f;
#pragma unroll
        for (int w = 0; w < 16; ++w) sum += s_part[w][tk][eo];
        const int e = oct * 8 + eo;
        if (tok0 + tk < T_tokens && e < E)
            logits_ws[static_cast<int64_t>(tok0 + tk) * kMaxExperts + e] = sum + (bg != nullptr ? bg[e] : 0.0f);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(tile_tickets + chunk, 1) == n_oct - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (threadIdx.x == 0) tile_tickets[chunk] = 0;
    const int64_t t = tok0 + warp;          // one warp per token for softmax and top-k
    if (t < T_tokens) {
        float logit[kSlots];
#pragma unroll
        for (int sl = 0; sl < kSlots; ++sl) {
            const int e = sl * 32 + lane;
            logit[sl] = e < E ? __ldcg(logits_ws + t * kMaxExperts + e) : -INFINITY;
        }
        softmax_topk_store(logit, E, k, renorm, t, lane, topk_idx, topk_w, probs);
    }
    finish_route(hist, topk_idx, gridDim.x);
}

template <int kTilesPerWarp>
cudaError_t route_mma_attributes() {
    constexpr int kSmem = 4 * 16 * (32 * kTilesPerWarp + 1) * 4;
    const cudaError_t e = cudaFuncSetAttribute(route_mma_kernel<kTilesPerWarp, false>,
                                               cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    return e != cudaSuccess ? e : cudaFuncSetAttribute(route_mma_kernel<kTilesPerWarp, true>,
                                                       cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
}

template <int kTilesPerWarp>
int launch_route_mma(const monde_problem& p, const void* x, const void* Wg, const float* bg, int32_t* topk_idx,
                     float* topk_w, float* probs, const HistArgs& hist, cudaStream_t s) {
    constexpr int kSmem = 4 * 16 * (32 * kTilesPerWarp + 1) * 4;
    if (kSmem > 48 * 1024) {      // more dynamic shared memory than the default limit: opt in, once per device
        constexpr int key = kTilesPerWarp == 1 ? kSetupRoute1 : kTilesPerWarp == 2 ? kSetupRoute2
                          : kTilesPerWarp == 4 ? kSetupRoute4 : kSetupRoute8;
        if (per_device_once(key, route_mma_attributes<kTilesPerWarp>) != cudaSuccess) return MONDE_ERR_CUDA;
    }
    const int grid = (p.T + 15) / 16;
    const int sms = current_sm_count();
    if (grid <= sms)
        launch_pdl(route_mma_kernel<kTilesPerWarp, true>, dim3(grid), dim3(512), kSmem, s,
            p.T, p.d_model, p.E, p.top_k, p.renormalize, static_cast<const __nv_bfloat16*>(x),
            static_cast<const __nv_bfloat16*>(Wg), bg, topk_idx, topk_w, probs, hist);
    else
        launch_pdl(route_mma_kernel<kTilesPerWarp, false>, dim3(grid), dim3(512), kSmem, s,
            p.T, p.d_model, p.E, p.top_k, p.renormalize, static_cast<const __nv_bfloat16*>(x),
            static_cast<const __nv_bfloat16*>(Wg), bg, topk_idx, topk_w, probs, hist);
    return MONDE_OK;
}

// The paper's own placement rule (Section 3.3, Eq. 3-6): the H experts with the most tokens are
// hot, H = floor(share * Expert_Activ) with share = alpha * BW_a / (BW_b + BW_a) and Expert_Activ
// the number of experts with at least one token (Eq. 5); equal counts: the smaller id is hotter.
// One CTA of 256 threads: thread e ranks expert e against all others.
__global__ void __launch_bounds__(kMaxExperts) classify_top_h_kernel(
        int E, double share, const int32_t* __restrict__ counts, uint8_t* __restrict__ cls,
        int32_t* __restrict__ hot_ids, int32_t* __restrict__ cold_ids, int32_t* __restrict__ n_hot_cold) {
    __shared__ int s_cnt[kMaxExperts];
    __shared__ int s_cls[kMaxExperts];
    __shared__ int s_active;
    pdl_launch_dependents();
    pdl_wait();
    const int e = threadIdx.x;
    if (e == 0) s_active = 0;
    s_cnt[e] = e < E ? counts[e] : 0;
    __syncthreads();
    const int c = s_cnt[e];
    if (c > 0) atomicAdd(&s_active, 1);
    int rank = 0;
    for (int o = 0; o < E; ++o) rank += (s_cnt[o] > c) || (s_cnt[o] == c && o < e);
    __syncthreads();
    const double h_real = share * static_cast<double>(s_active);
    int H = h_real <= 0.0 ? 0 : static_cast<int>(floor(h_real));
    H = min(H, s_active);
    const int k = c > 0 ? (rank < H ? 2 : 1) : 0;
    s_cls[e] = k;
    if (e < E) cls[e] = static_cast<uint8_t>(k);
    __syncthreads();
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;       // lane owns experts [lane*8, lane*8+8): ascending compaction
    int nh = 0, nc = 0;
#pragma unroll
    for (int i = 0; i < kSlots; ++i) {
        nh += s_cls[lane * kSlots + i] == 2;
        nc += s_cls[lane * kSlots + i] == 1;
    }
    int ph = nh, pc = nc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, ph, o);
        const int b = __shfl_up_sync(0xffffffffu, pc, o);
        if (lane >= o) { ph += a; pc += b; }
    }
    int ih = ph - nh, ic = pc - nc;
#pragma unroll
    for (int i = 0; i < kSlots; ++i) {
        const int x = lane * kSlots + i;
        if (s_cls[x] == 2) hot_ids[ih++] = x;
        else if (s_cls[x] == 1) cold_ids[ic++] = x;
    }
    if (lane == 31) {
        n_hot_cold[0] = ph;
        n_hot_cold[1] = pc;
    }
}

}  // namespace

int launch_route(const monde_problem& p, const void* x, const void* Wg, const float* bg,
                 int32_t* topk_idx, float* topk_w, float* probs, int32_t* counts, int32_t* offsets, uint8_t* cls,
                 int32_t* hot_ids, int32_t* cold_ids, int32_t* n_hot_cold, void* ws, cudaStream_t s) {
    char* base = static_cast<char*>(ws);
    int32_t* ticket = reinterpret_cast<int32_t*>(base + WsLayout::kRouteTicket);
    const HistArgs hist{p.T * p.top_k, p.E, p.hot_threshold, counts, offsets, cls, hot_ids, cold_ids, n_hot_cold, ticket};
    if (p.T == 0) {
        launch_pdl(histogram_only_kernel, dim3(1), dim3(256), 0, s, hist, topk_idx);
        return launched();
    }
    if (p.dtype == MONDE_BF16 && p.T <= kSplitRouteMaxTokens) {
        // at most 16 chunks: their tickets follow the call's own in the workspace header
        launch_pdl(route_split_kernel, dim3((p.T + 15) / 16, (p.E + 7) / 8), dim3(512), 0, s,
            p.T, p.d_model, p.E, p.top_k, p.renormalize, static_cast<const __nv_bfloat16*>(x),
            static_cast<const __nv_bfloat16*>(Wg), bg, topk_idx, topk_w, probs,
            reinterpret_cast<float*>(base + ws_layout(p).logits_off), ticket + 1, hist);
        return launched();
    }
    if (p.dtype == MONDE_BF16) {
        int st;
        if (p.E <= 32) st = launch_route_mma<1>(p, x, Wg, bg, topk_idx, topk_w, probs, hist, s);
        else if (p.E <= 64) st = launch_route_mma<2>(p, x, Wg, bg, topk_idx, topk_w, probs, hist, s);
        else if (p.E <= 128) st = launch_route_mma<4>(p, x, Wg, bg, topk_idx, topk_w, probs, hist, s);
        else st = launch_route_mma<8>(p, x, Wg, bg, topk_idx, topk_w, probs, hist, s);
        if (st != MONDE_OK) return st;
    } else {
        const int warps = 4;
        launch_pdl(route_warp_per_token_kernel<float>, dim3((p.T + warps - 1) / warps), dim3(warps * 32), 0, s,
            p.T, p.d_model, p.E, p.top_k, p.renormalize, static_cast<const float*>(x),
            static_cast<const float*>(Wg), bg, topk_idx, topk_w, probs, hist);
    }
    return launched();
}

int launch_classify_top_h(const monde_problem& p, double share, const int32_t* counts, uint8_t* cls,
                          int32_t* hot_ids, int32_t* cold_ids, int32_t* n_hot_cold, cudaStream_t s) {
    launch_pdl(classify_top_h_kernel, dim3(1), dim3(kMaxExperts), 0, s, p.E, share, counts, cls, hot_ids, cold_ids,
               n_hot_cold);
    return launched();
}

}  // namespace monde
