// bf16 expert linear layers on the 5th-generation tensor cores (tcgen05, accumulators in
// tensor memory), operands staged in shared memory by TMA.
//
// Paper: Section 3.1 describes an expert computation as C = A x B with A the routed
// tokens (small height for cold experts) and B the expert parameters (width d_model or
// d_ff); Section 2.2 separates hot experts (many tokens) from cold, memory-bound ones;
// Section 3.4 names the gemm and gemm+activation kernels.  Here every expert GEMM is
// issued "weights as rows": the 128-row MMA dimension holds 128 output features of the
// expert's weight matrix and the MMA N dimension holds the tokens, so an expert with m
// tokens costs one pass over its weights with N = m rounded up to 16.  The two classes
// are two instantiations of the same kernel:
//   cold: token tile <= 64, 8-stage ring of 24 KB stages -> a deep queue of weight bytes
//         in flight per SM; the tensor core is idle most of the time and HBM sets the pace;
//   hot : token tile <= 256 (a full-rate 128 x 256 MMA), 4-stage ring of 48 KB stages.
// Warp roles: warp 0 issues TMA, warp 1 issues MMAs and owns the TMEM allocation, warps
// 2-5 drain the accumulator (bias + activation fused) while the next tile's MMAs run into
// the second accumulator buffer.  CTAs are persistent and walk a device-built list of
// (expert, feature tile, token tile) units, so counts never travel to the host.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "sm100.cuh"

namespace monde {

namespace {

using namespace sm100;

constexpr int kThreads = 192;
constexpr int kBlockK = 64;           // K elements per stage: one 128-byte swizzle row
constexpr int kTileRows = 128;        // output features per unit = MMA M
constexpr int kABytes = kTileRows * 128;
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // every device-side wait gives up after 2 s

enum WaitSite { kSiteProducerEmpty = 1, kSiteMmaFull = 2, kSiteMmaTmemEmpty = 3, kSiteEpilogueTmemFull = 4 };

template <int kTokTile, int kStages>
struct Cfg {
    static constexpr int kBBytes = kTokTile * 128;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTileBytes = kStages * kStageBytes;
    static constexpr int kNumBars = 2 * kStages + 4;
    static constexpr int kTableInts = 6 * (kMaxExperts + 1);
    static constexpr int kSmemBytes = 1024 + kTileBytes + kNumBars * 8 + 64 + kTableInts * 4;
    static constexpr int kTmemCols = 2 * kTokTile < 32 ? 32 : 2 * kTokTile;   // power of two for 64 / 256
};

struct Unit {
    int e;        // expert id
    int row0;     // first row of the token tile in the expert-contiguous buffers
    int rows;     // valid token rows in the tile
    int nt;       // rows rounded up to a multiple of 16 (MMA N)
    int n0;       // first output feature of the tile
};

struct UnitTable {
    int* prefix;  // [n+1] exclusive prefix of units per listed expert
    int* e;
    int* off;
    int* m;
    int* tt;      // token tiles
    int* per;     // tokens per tile (multiple of 16)
    __device__ __forceinline__ Unit decode(int u, int& cursor) const {
        while (u >= prefix[cursor + 1]) ++cursor;
        const int local = u - prefix[cursor];
        const int tok = local % tt[cursor];
        Unit r;
        r.e = e[cursor];
        r.n0 = (local / tt[cursor]) * kTileRows;
        const int r_in_e = tok * per[cursor];
        r.rows = min(per[cursor], m[cursor] - r_in_e);
        r.nt = (r.rows + 15) & ~15;
        r.row0 = off[cursor] + r_in_e;
        return r;
    }
};

__device__ __forceinline__ void report_timeout(int32_t* status, volatile int* abort_flag, int site) {
    *abort_flag = 1;
    if (atomicCAS(status, 0, MONDE_ERR_TIMEOUT) == 0) status[1] = site;
}

// Out[row, n] = act?(bias[e, n] + sum_k In[row, k] * W[e, n, k]) for the rows of the listed experts.
template <int kTokTile, int kStages>
__global__ void __launch_bounds__(kThreads, 1) expert_gemm_kernel(
        const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_in,
        int K, int N, int act, const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ out,
        const int32_t* __restrict__ counts, const int32_t* __restrict__ offsets,
        const int32_t* __restrict__ ids, const int32_t* __restrict__ n_ids, int32_t* status) {
    using C = Cfg<kTokTile, kStages>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kTileBytes);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + C::kNumBars);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* tab = reinterpret_cast<int*>(tmem_slot + 16);
    UnitTable ut;
    ut.prefix = tab;
    ut.e = tab + (kMaxExperts + 1);
    ut.off = ut.e + (kMaxExperts + 1);
    ut.m = ut.off + (kMaxExperts + 1);
    ut.tt = ut.m + (kMaxExperts + 1);
    ut.per = ut.tt + (kMaxExperts + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_list = min(*n_ids, kMaxExperts);
    const int n_tiles = (N + kTileRows - 1) / kTileRows;
    const int k_blocks = K / kBlockK;

    // ---- set-up: unit table, barriers, tensor memory --------------------------------
    for (int i = tid; i < n_list; i += kThreads) {
        const int e = ids[i];
        const int m = counts[e];
        const int tt = (m + kTokTile - 1) / kTokTile;
        const int per = tt > 0 ? (((m + tt - 1) / tt + 15) & ~15) : 16;
        ut.e[i] = e;
        ut.off[i] = offsets[e];
        ut.m[i] = m;
        ut.tt[i] = tt > 0 ? tt : 1;
        ut.per[i] = per;
        ut.prefix[i + 1] = tt * n_tiles;
    }
    if (tid == 0) {
        ut.prefix[0] = 0;
        *abort_flag = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);             // full: producer's expect_tx arrival
            mbar_init(smem_u32(&bars[kStages + s]), 1);   // empty: one tcgen05.commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars[2 * kStages + b]), 1);       // accumulator full: one commit
            mbar_init(smem_u32(&bars[2 * kStages + 2 + b]), 4);   // accumulator drained: 4 epilogue warps
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 0) {   // inclusive scan of the per-expert unit counts, 8 entries per lane
        int v[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int idx = lane * 8 + i;
            v[i] = idx < n_list ? ut.prefix[idx + 1] : 0;
            sum += v[i];
        }
        int inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        int run = inc - sum;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int idx = lane * 8 + i;
            run += v[i];
            if (idx < n_list) ut.prefix[idx + 1] = run;
        }
    } else if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const int total_units = ut.prefix[n_list];
    const uint32_t tiles_u32 = smem_u32(smem);

    if (warp == 0) {
        // ---- TMA producer ------------------------------------------------------------
        if (lane == 0) {
            prefetch_tensormap(&map_w);
            prefetch_tensormap(&map_in);
            const uint64_t pol_w = policy_evict_first();   // weights are read once
            const uint64_t pol_x = policy_evict_last();    // token tiles are re-read by every feature tile
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int u = blockIdx.x; ok && u < total_units; u += gridDim.x) {
                const Unit un = ut.decode(u, cursor);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(&bars[kStages + stage]), phase ^ 1u, abort_flag, kWaitLimitNs)) {
                        report_timeout(status, abort_flag, kSiteProducerEmpty);
                        ok = false;
                        break;
                    }
                    const uint32_t full = smem_u32(&bars[stage]);
                    const uint32_t a_dst = tiles_u32 + stage * C::kStageBytes;
                    mbar_arrive_expect_tx(full, kABytes + un.nt * 128);
                    tma_load_2d(a_dst, &map_w, full, kb * kBlockK, un.e * N + un.n0, pol_w);
                    for (int j = 0; j < un.nt; j += 16)
                        tma_load_2d(a_dst + kABytes + j * 128, &map_in, full, kb * kBlockK, un.row0 + j, pol_x);
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer --------------------------------------------------------------
        if (lane == 0) {
            int stage = 0, cursor = 0, it = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int u = blockIdx.x; ok && u < total_units; u += gridDim.x, ++it) {
                const Unit un = ut.decode(u, cursor);
                const int b = it & 1;
                const uint32_t tphase = (it >> 1) & 1;
                if (!mbar_wait(smem_u32(&bars[2 * kStages + 2 + b]), tphase ^ 1u, abort_flag, kWaitLimitNs)) {
                    report_timeout(status, abort_flag, kSiteMmaTmemEmpty);
                    break;
                }
                tc_fence_after_sync();
                const uint32_t idesc = idesc_bf16_m128(un.nt);
                const uint32_t d_tmem = tmem_base + b * kTokTile;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(&bars[stage]), phase, abort_flag, kWaitLimitNs)) {
                        report_timeout(status, abort_flag, kSiteMmaFull);
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t a_addr = tiles_u32 + stage * C::kStageBytes;
                    const uint64_t a_desc = smem_desc_sw128(a_addr);
                    const uint64_t b_desc = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
                    for (int k4 = 0; k4 < kBlockK / 16; ++k4)
                        umma_bf16(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, (kb | k4) != 0);
                    umma_commit(smem_u32(&bars[kStages + stage]));   // stage reusable once these MMAs finish
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(smem_u32(&bars[2 * kStages + b]));   // accumulator complete
            }
        }
    } else {
        // ---- epilogue: TMEM -> registers -> bias, activation -> global ----------------
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        int cursor = 0, it = 0;
        for (int u = blockIdx.x; u < total_units; u += gridDim.x, ++it) {
            const Unit un = ut.decode(u, cursor);
            const int b = it & 1;
            const uint32_t tphase = (it >> 1) & 1;
            if (!mbar_wait(smem_u32(&bars[2 * kStages + b]), tphase, abort_flag, kWaitLimitNs)) {
                report_timeout(status, abort_flag, kSiteEpilogueTmemFull);
                break;
            }
            tc_fence_after_sync();
            const int n = un.n0 + q * 32 + lane;
            const bool n_ok = n < N;
            const float bias_v = (bias != nullptr && n_ok) ? __bfloat162float(bias[static_cast<int64_t>(un.e) * N + n]) : 0.0f;
            const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * kTokTile;
            __nv_bfloat16* dst = out + static_cast<int64_t>(un.row0) * N + n;
            for (int c0 = 0; c0 < un.nt; c0 += 16) {
                uint32_t v[16];
                tmem_ld_16(t_addr + c0, v);
                tmem_ld_wait();
                if (n_ok) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (c0 + j < un.rows) {
                            float r = __uint_as_float(v[j]) + bias_v;
                            if (act >= 0) r = apply_act(r, act);
                            dst[static_cast<int64_t>(c0 + j) * N] = __float2bfloat16_rn(r);
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars[2 * kStages + 2 + b]));
        }
    }

    // ---- teardown --------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ---- host side -----------------------------------------------------------------------

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Row-major bf16 matrix [rows, cols] viewed through boxes of box_rows x 64 columns, 128-byte swizzle.
bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBlockK), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        return v > 0 ? v : 148;
    }();
    return n;
}

template <int kTokTile, int kStages>
int launch_one(int E, int rows_total, int K, int N, int act, const void* in, const void* W, const void* bias,
               void* out, const int32_t* counts, const int32_t* offsets, const int32_t* ids,
               const int32_t* n_ids, int32_t* status, cudaStream_t s) {
    using C = Cfg<kTokTile, kStages>;
    auto kernel = expert_gemm_kernel<kTokTile, kStages>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    });
    if (attr_err != cudaSuccess) return MONDE_ERR_CUDA;
    CUtensorMap map_w, map_in;
    if (!make_map(&map_w, W, static_cast<uint64_t>(E) * N, K, kTileRows)) return MONDE_ERR_CUDA;
    if (!make_map(&map_in, in, rows_total, K, 16)) return MONDE_ERR_CUDA;
    kernel<<<sm_count(), kThreads, C::kSmemBytes, s>>>(
        map_w, map_in, K, N, act, static_cast<const __nv_bfloat16*>(bias), static_cast<__nv_bfloat16*>(out), counts,
        offsets, ids, n_ids, status);
    return launched();
}

}  // namespace

int launch_ffn_bf16(const monde_problem& p, const void* x_perm, const void* W1, const void* b1,
                    const void* W2, const void* b2, const int32_t* counts, const int32_t* offsets,
                    const int32_t* hot_ids, const int32_t* cold_ids, const int32_t* n_hot_cold,
                    void* y_perm, void* ws, cudaStream_t s) {
    void* h = static_cast<char*>(ws) + WsLayout::kHidden;
    int32_t* status = reinterpret_cast<int32_t*>(static_cast<char*>(ws) + WsLayout::kStatus);
    const int A = p.T * p.top_k;
    int st;
    // cold class: weight-streaming configuration
    st = launch_one<64, 8>(p.E, A, p.d_model, p.d_ff, p.act, x_perm, W1, b1, h, counts, offsets, cold_ids,
                           n_hot_cold + 1, status, s);
    if (st != MONDE_OK) return st;
    // hot class: wide token tiles
    st = launch_one<256, 4>(p.E, A, p.d_model, p.d_ff, p.act, x_perm, W1, b1, h, counts, offsets, hot_ids,
                            n_hot_cold, status, s);
    if (st != MONDE_OK) return st;
    st = launch_one<64, 8>(p.E, A, p.d_ff, p.d_model, -1, h, W2, b2, y_perm, counts, offsets, cold_ids,
                           n_hot_cold + 1, status, s);
    if (st != MONDE_OK) return st;
    return launch_one<256, 4>(p.E, A, p.d_ff, p.d_model, -1, h, W2, b2, y_perm, counts, offsets, hot_ids,
                              n_hot_cold, status, s);
}

}  // namespace monde
