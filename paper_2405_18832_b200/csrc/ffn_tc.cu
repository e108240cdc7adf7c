// bf16 expert FFN on the 5th-generation tensor cores (tcgen05, accumulators in tensor
// memory), operands staged in shared memory by TMA; one persistent launch runs both
// linear layers of every activated expert, hot and cold.
//
// Paper: Section 3.1 describes an expert computation as C = A x B with A the routed
// tokens (small height for cold experts) and B the expert parameters (width d_model or
// d_ff); Section 2.2 separates hot experts (many tokens) from cold, memory-bound ones;
// Section 3.3 runs the two classes side by side on the hardware that suits each;
// Section 3.4 names the gemm and gemm+activation kernels.
//
// Every expert GEMM is issued "weights as rows": the 128-row MMA dimension holds 128
// output features of the expert's weight matrix and the MMA N dimension holds the tokens,
// so an expert with m tokens costs one pass over its weights with N = m rounded up to 16.
// The class chosen by the router selects the tiling of a work unit:
//   hot : token tile <= 256 (a full-rate 128 x 256 MMA), 4-stage ring of 48 KB stages;
//   cold: token tile <= 64, 8-stage ring of 24 KB stages -> a deep queue of weight bytes in
//         flight per SM; the tensor core idles most of the time and HBM sets the pace.
// Work units (expert, 128-feature tile, token tile) are ordered hot-first-layer,
// hot-second-layer, cold-first-layer, cold-second-layer and dealt round-robin to one
// persistent CTA per SM.  A second-layer unit needs the hidden rows of its token tile,
// which are produced by first-layer units earlier in the same order: per-token-tile
// counters in the workspace carry that dependency, and the TMA producer streams the
// unit's weights while it waits, so weight traffic never stalls at the layer boundary.
// Warp roles: warp 0 issues TMA, warp 1 issues MMAs and owns the TMEM allocation, warps
// 2-5 drain the accumulator (bias + activation fused) while the next unit's MMAs run into
// the second accumulator buffer.  Counts never travel to the host.
#include <cuda.h>

#include <cstdlib>
#include <mutex>

#include "common.cuh"
#include "sm100.cuh"

namespace monde {

unsigned long long* g_trace = nullptr;
int g_trace_slots = 0;

namespace {

using namespace sm100;

constexpr int kThreads = 224;       // producer, MMA, 4 epilogue warps, publisher
constexpr int kBlockK = 64;           // K elements per stage: one 128-byte swizzle row
constexpr int kTileRows = 128;        // output features per unit = MMA M
constexpr int kABytes = kTileRows * 128;
constexpr int kMaxStages = 8;
constexpr int kHotTokTile = 256, kHotStages = 4;     // 4 x (16 KB + 32 KB)
constexpr int kColdTokTile = 64, kColdStages = 8;    // 8 x (16 KB +  8 KB)
constexpr int kTileBytes = 192 * 1024;
constexpr int kNumBars = 2 * kMaxStages + 6;
constexpr int kTableInts = 6 * (kMaxExperts + 1);
constexpr int kStageOutBytes = 2 * 16 * kTileRows * 2;
constexpr int kSmemBytes = 1024 + kTileBytes + kNumBars * 8 + 64 + kTableInts * 4 + kStageOutBytes + 16;
constexpr int kTmemCols = 512;        // two accumulator buffers of 256 fp32 columns
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // every device-side wait gives up after 2 s

enum WaitSite { kSiteProducerEmpty = 1, kSiteMmaFull = 2, kSiteMmaTmemEmpty = 3, kSiteEpilogueTmemFull = 4,
                kSiteHiddenReady = 5, kSiteDrain = 6 };

struct FfnParams {
    int d_model, d_ff, act;
    const __nv_bfloat16* b1;
    const __nv_bfloat16* b2;
    __nv_bfloat16* h;
    __nv_bfloat16* y;
    const int32_t* counts;
    const int32_t* offsets;
    const int32_t* hot_ids;
    const int32_t* cold_ids;
    const int32_t* n_hot_cold;
    int32_t* status;       // {status, site}
    int32_t* ticket;       // CTAs that have finished
    int32_t* ready;        // per token tile: first-layer units finished
    unsigned long long* trace;   // diagnostic timeline (null in normal use): [cta][unit slot][8]
    int trace_slots;
};

// Diagnostic timeline: slot 0 unit id, 1-2 producer first/last issue, 3-4 MMA first full / commit,
// 5-6 epilogue start / end (global timer, ns).
__device__ __forceinline__ void trace_mark(const FfnParams& P, int it, int slot, unsigned long long v) {
    if (P.trace != nullptr && it < P.trace_slots)
        P.trace[(static_cast<size_t>(blockIdx.x) * P.trace_slots + it) * 8 + slot] = v;
}
__device__ __forceinline__ void trace_time(const FfnParams& P, int it, int slot) {
    if (P.trace != nullptr && it < P.trace_slots)
        P.trace[(static_cast<size_t>(blockIdx.x) * P.trace_slots + it) * 8 + slot] = global_timer_ns();
}

struct Unit {
    int e;        // expert id
    int row0;     // first row of the token tile in the expert-contiguous buffers
    int rows;     // valid token rows in the tile
    int nt;       // rows rounded up to a multiple of 16 (MMA N)
    int n0;       // first output feature of the tile
    int layer;    // 0: h = act(x W1^T + b1), 1: y = h W2^T + b2
    int cold;     // class: selects the stage geometry
    int ready_idx;  // token-tile index into the dependency counters
};

// Per-CTA copy of the unit list in shared memory.  Entries 0..n_hot-1 are the hot experts,
// n_hot..n_hot+n_cold-1 the cold ones; tt_prefix is the exclusive prefix of token tiles.
struct UnitTable {
    int* tt_prefix;   // [n+1]
    int* e;
    int* off;
    int* m;
    int* tt;          // token tiles of this expert
    int* per;         // tokens per tile (multiple of 16)
    int n_hot, n_all, nt1, nt2;      // 128-feature tiles of layer 1 (d_ff) and layer 2 (d_model)
    int seg[5];                      // unit index where each (class, layer) segment starts

    __device__ __forceinline__ Unit decode(int u) const {
        int sgm = 0;
        while (u >= seg[sgm + 1]) ++sgm;
        Unit r;
        r.cold = sgm >> 1;
        r.layer = sgm & 1;
        const int ntl = r.layer ? nt2 : nt1;
        const int lo_entry = r.cold ? n_hot : 0;
        const int tt_base = tt_prefix[lo_entry];
        const int v = u - seg[sgm];
        int lo = lo_entry, hi = (r.cold ? n_all : n_hot) - 1;      // largest entry with block start <= v
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if ((tt_prefix[mid] - tt_base) * ntl <= v) lo = mid; else hi = mid - 1;
        }
        const int local = v - (tt_prefix[lo] - tt_base) * ntl;
        const int tok = local % tt[lo];
        r.e = e[lo];
        r.n0 = (local / tt[lo]) * kTileRows;
        const int r_in_e = tok * per[lo];
        r.rows = min(per[lo], m[lo] - r_in_e);
        r.nt = (r.rows + 15) & ~15;
        r.row0 = off[lo] + r_in_e;
        r.ready_idx = tt_prefix[lo] + tok;
        return r;
    }
};

__device__ __forceinline__ void report_timeout(int32_t* status, volatile int* abort_flag, int site) {
    *abort_flag = 1;
    if (atomicCAS(status, 0, MONDE_ERR_TIMEOUT) == 0) status[1] = site;
}

// erf by the rational approximation 7.1.26 of Abramowitz & Stegun (|error| <= 1.5e-7, far
// below one bf16 rounding of the result); a dozen instructions instead of a library call.
__device__ __forceinline__ float erf_as(float x) {
    const float ax = fabsf(x);
    const float t = __frcp_rn(fmaf(0.3275911f, ax, 1.0f));
    float p = fmaf(1.061405429f, t, -1.453152027f);
    p = fmaf(p, t, 1.421413741f);
    p = fmaf(p, t, -0.284496736f);
    p = fmaf(p, t, 0.254829592f);
    const float r = 1.0f - p * t * __expf(-ax * ax);
    return copysignf(r, x);
}
template <int kAct>
__device__ __forceinline__ float activate(float v) {
    if (kAct == MONDE_ACT_RELU) return fmaxf(v, 0.0f);
    return 0.5f * v * (1.0f + erf_as(v * 0.70710678118654752440f));
}

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

template <int kAct>
__global__ void __launch_bounds__(kThreads, 1) expert_ffn_kernel(
        const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_w2,
        const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_h, const FfnParams P) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kTileBytes);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* tab = reinterpret_cast<int*>(tmem_slot + 16);
    __nv_bfloat16* stg = reinterpret_cast<__nv_bfloat16*>(                     // 2 x [16 tokens][128 features]
        (reinterpret_cast<uintptr_t>(tab + kTableInts) + 15) & ~uintptr_t(15));
    UnitTable ut;
    ut.tt_prefix = tab;
    ut.e = tab + (kMaxExperts + 1);
    ut.off = ut.e + (kMaxExperts + 1);
    ut.m = ut.off + (kMaxExperts + 1);
    ut.tt = ut.m + (kMaxExperts + 1);
    ut.per = ut.tt + (kMaxExperts + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    ut.n_hot = min(P.n_hot_cold[0], kMaxExperts);
    ut.n_all = min(ut.n_hot + P.n_hot_cold[1], kMaxExperts);
    ut.nt1 = (P.d_ff + kTileRows - 1) / kTileRows;
    ut.nt2 = (P.d_model + kTileRows - 1) / kTileRows;

    // ---- set-up: unit table, barriers, tensor memory --------------------------------
    for (int i = tid; i < ut.n_all; i += kThreads) {
        const bool cold = i >= ut.n_hot;
        const int e = cold ? P.cold_ids[i - ut.n_hot] : P.hot_ids[i];
        const int tile = cold ? kColdTokTile : kHotTokTile;
        const int m = P.counts[e];
        const int tt = max(1, (m + tile - 1) / tile);
        ut.e[i] = e;
        ut.off[i] = P.offsets[e];
        ut.m[i] = m;
        ut.tt[i] = tt;
        ut.per[i] = ((m + tt - 1) / tt + 15) & ~15;
        ut.tt_prefix[i + 1] = tt;
    }
    if (tid == 0) {
        ut.tt_prefix[0] = 0;
        *abort_flag = 0;
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&bars[s]), 1);               // full: producer's expect_tx arrival
            mbar_init(smem_u32(&bars[kMaxStages + s]), 1);  // empty: one tcgen05.commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars[2 * kMaxStages + b]), 1);       // accumulator full: one commit
            mbar_init(smem_u32(&bars[2 * kMaxStages + 2 + b]), 4);   // accumulator drained: 4 epilogue warps
            mbar_init(smem_u32(&bars[2 * kMaxStages + 4 + b]), 4);   // output rows stored: 4 epilogue warps
        }
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 0) {   // inclusive scan of the per-expert token-tile counts, 8 entries per lane
        int v[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int idx = lane * 8 + i;
            v[i] = idx < ut.n_all ? ut.tt_prefix[idx + 1] : 0;
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
            if (idx < ut.n_all) ut.tt_prefix[idx + 1] = run;
        }
    } else if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const int tt_hot = ut.tt_prefix[ut.n_hot], tt_all = ut.tt_prefix[ut.n_all];
    ut.seg[0] = 0;
    ut.seg[1] = tt_hot * ut.nt1;
    ut.seg[2] = ut.seg[1] + tt_hot * ut.nt2;
    ut.seg[3] = ut.seg[2] + (tt_all - tt_hot) * ut.nt1;
    ut.seg[4] = ut.seg[3] + (tt_all - tt_hot) * ut.nt2;
    const int total_units = ut.seg[4];
    const uint32_t tiles_u32 = smem_u32(smem);
    const int ready_target = ut.nt1;

    if (warp == 0) {
        // ---- TMA producer ------------------------------------------------------------
        if (lane == 0) {
            prefetch_tensormap(&map_w1);
            prefetch_tensormap(&map_w2);
            prefetch_tensormap(&map_x);
            prefetch_tensormap(&map_h);
            const uint64_t pol_w = policy_evict_first();   // weights are read once
            const uint64_t pol_x = policy_evict_last();    // token tiles are re-read by every feature tile
            int stage = 0, cls = -1, stages = kHotStages, stage_bytes = kABytes + kHotTokTile * 128;
            uint32_t fill_bits = 0;     // bit s: parity of the number of fills of stage s
            bool ok = true;
            int pit = 0;
            for (int u = blockIdx.x; ok && u < total_units; u += gridDim.x, ++pit) {
                const Unit un = ut.decode(u);
                trace_mark(P, pit, 0, static_cast<unsigned long long>(u));
                if (un.cold != cls) {
                    // geometry switch: every stage filled so far must have been consumed
                    for (int s = 0; ok && s < stages; ++s)
                        if (!mbar_wait(smem_u32(&bars[kMaxStages + s]), ((fill_bits >> s) & 1u) ^ 1u, abort_flag,
                                       kWaitLimitNs)) {
                            report_timeout(P.status, abort_flag, kSiteDrain);
                            ok = false;
                        }
                    if (!ok) break;
                    cls = un.cold;
                    stages = cls ? kColdStages : kHotStages;
                    stage_bytes = kABytes + (cls ? kColdTokTile : kHotTokTile) * 128;
                    stage = 0;
                }
                const CUtensorMap* mw = un.layer ? &map_w2 : &map_w1;
                const CUtensorMap* mi = un.layer ? &map_h : &map_x;
                const int K = un.layer ? P.d_ff : P.d_model;
                const int N = un.layer ? P.d_model : P.d_ff;
                const int k_blocks = K / kBlockK;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(&bars[kMaxStages + stage]), ((fill_bits >> stage) & 1u) ^ 1u, abort_flag,
                                   kWaitLimitNs)) {
                        report_timeout(P.status, abort_flag, kSiteProducerEmpty);
                        ok = false;
                        break;
                    }
                    if (kb == 0) trace_time(P, pit, 1);
                    const uint32_t full = smem_u32(&bars[stage]);
                    const uint32_t a_dst = tiles_u32 + stage * stage_bytes;
                    mbar_arrive_expect_tx(full, kABytes + un.nt * 128);
                    tma_load_2d(a_dst, mw, full, kb * kBlockK, un.e * N + un.n0, pol_w);
                    if (kb == 0 && un.layer == 1) {
                        // the hidden rows of this token tile must be complete; weights already stream
                        const int32_t* flag = P.ready + un.ready_idx;
                        if (ld_acquire(flag) < ready_target) {
                            const uint64_t t0 = global_timer_ns();
                            while (ld_acquire(flag) < ready_target) {
                                if (*abort_flag != 0 || global_timer_ns() - t0 > kWaitLimitNs) {
                                    report_timeout(P.status, abort_flag, kSiteHiddenReady);
                                    ok = false;
                                    break;
                                }
                            }
                            if (!ok) break;
                        }
                        fence_proxy_async_all();
                    }
                    for (int j = 0; j < un.nt; j += 16)
                        tma_load_2d(a_dst + kABytes + j * 128, mi, full, kb * kBlockK, un.row0 + j, pol_x);
                    fill_bits ^= 1u << stage;
                    if (++stage == stages) stage = 0;
                }
                trace_time(P, pit, 2);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer --------------------------------------------------------------
        if (lane == 0) {
            int stage = 0, it = 0, cls = -1, stages = kHotStages, stage_bytes = kABytes + kHotTokTile * 128;
            uint32_t use_bits = 0;      // bit s: parity of the number of uses of stage s
            bool ok = true;
            for (int u = blockIdx.x; ok && u < total_units; u += gridDim.x, ++it) {
                const Unit un = ut.decode(u);
                if (un.cold != cls) {
                    cls = un.cold;
                    stages = cls ? kColdStages : kHotStages;
                    stage_bytes = kABytes + (cls ? kColdTokTile : kHotTokTile) * 128;
                    stage = 0;
                }
                const int b = it & 1;
                const uint32_t tphase = (it >> 1) & 1;
                if (!mbar_wait(smem_u32(&bars[2 * kMaxStages + 2 + b]), tphase ^ 1u, abort_flag, kWaitLimitNs)) {
                    report_timeout(P.status, abort_flag, kSiteMmaTmemEmpty);
                    break;
                }
                tc_fence_after_sync();
                const uint32_t idesc = idesc_bf16_m128(un.nt);
                const uint32_t d_tmem = tmem_base + b * 256;
                const int k_blocks = (un.layer ? P.d_ff : P.d_model) / kBlockK;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(smem_u32(&bars[stage]), (use_bits >> stage) & 1u, abort_flag, kWaitLimitNs)) {
                        report_timeout(P.status, abort_flag, kSiteMmaFull);
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    if (kb == 0) trace_time(P, it, 3);
                    const uint32_t a_addr = tiles_u32 + stage * stage_bytes;
                    const uint64_t a_desc = smem_desc_sw128(a_addr);
                    const uint64_t b_desc = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
                    for (int k4 = 0; k4 < kBlockK / 16; ++k4)
                        umma_bf16(d_tmem, a_desc + 2 * k4, b_desc + 2 * k4, idesc, (kb | k4) != 0);
                    umma_commit(smem_u32(&bars[kMaxStages + stage]));   // stage reusable once these MMAs finish
                    use_bits ^= 1u << stage;
                    if (++stage == stages) stage = 0;
                }
                if (ok) umma_commit(smem_u32(&bars[2 * kMaxStages + b]));   // accumulator complete
                trace_time(P, it, 4);
            }
        }
    } else if (warp < 6) {
        // ---- epilogue: TMEM -> registers -> bias, activation -> global ----------------
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        int it = 0;
        for (int u = blockIdx.x; u < total_units; u += gridDim.x, ++it) {
            const Unit un = ut.decode(u);
            const int b = it & 1;
            const uint32_t tphase = (it >> 1) & 1;
            const bool got = mbar_wait(smem_u32(&bars[2 * kMaxStages + b]), tphase, abort_flag, kWaitLimitNs);
            if (!got) report_timeout(P.status, abort_flag, kSiteEpilogueTmemFull);
            // the four epilogue warps share a named barrier below: leave together or not at all
            uint32_t all_got;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.u32 q, %1, 0;\n\t"
                "bar.red.and.pred p, 1, 128, q;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(all_got) : "r"(static_cast<uint32_t>(got)) : "memory");
            if (!all_got) break;
            tc_fence_after_sync();
            if (warp == 2 && lane == 0) trace_time(P, it, 5);
            const int N = un.layer ? P.d_model : P.d_ff;
            const __nv_bfloat16* bias = un.layer ? P.b2 : P.b1;
            const int n = un.n0 + q * 32 + lane;
            const float bias_v = (bias != nullptr && n < N) ? __bfloat162float(bias[static_cast<int64_t>(un.e) * N + n]) : 0.0f;
            const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * 256;
            __nv_bfloat16* out = un.layer ? P.y : P.h;
            const int et = tid - 64;                    // 0..127 within the epilogue warps (warps 2-5)
            const int rd_row = et >> 4, rd_col = (et & 15) * 8;
            const bool col_ok = un.n0 + rd_col < N;     // N is a multiple of 64: 8-wide groups are all in or all out
            // 32 accumulator columns (tokens) per TMEM load, the next load in flight while this one
            // is converted; each group of 16 tokens is transposed through shared memory so that
            // global stores are 16-byte pieces of 256-byte contiguous row segments.  The code is
            // kept small on purpose: an unrolled epilogue with an inlined library erf per element
            // overflowed the instruction cache and ran 20x slower.
            auto drain32 = [&](const uint32_t (&v)[32], int c32) {
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    const int c0 = c32 + g * 16;
                    if (c0 < un.nt) {
                        __nv_bfloat16* sb = stg + g * (16 * kTileRows);
                        if (un.layer) {
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                sb[j * kTileRows + q * 32 + lane] = __float2bfloat16_rn(__uint_as_float(v[g * 16 + j]) + bias_v);
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                sb[j * kTileRows + q * 32 + lane] =
                                    __float2bfloat16_rn(activate<kAct>(__uint_as_float(v[g * 16 + j]) + bias_v));
                        }
                        asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            const int r = rd_row + half * 8;
                            if (col_ok && c0 + r < un.rows) {
                                const uint4 val = *reinterpret_cast<const uint4*>(sb + r * kTileRows + rd_col);
                                *reinterpret_cast<uint4*>(out + static_cast<int64_t>(un.row0 + c0 + r) * N + un.n0 + rd_col) = val;
                            }
                        }
                    }
                }
            };
            uint32_t va[32], vb[32];
            tmem_ld_32(t_addr, va);
            for (int c32 = 0; c32 < un.nt; c32 += 64) {
                tmem_ld_wait();
                if (c32 + 32 < un.nt) tmem_ld_32(t_addr + c32 + 32, vb);
                drain32(va, c32);
                if (c32 + 32 < un.nt) {
                    tmem_ld_wait();
                    if (c32 + 64 < un.nt) tmem_ld_32(t_addr + c32 + 64, va);
                    drain32(vb, c32 + 32);
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&bars[2 * kMaxStages + 2 + b]));   // accumulator buffer free
                mbar_arrive(smem_u32(&bars[2 * kMaxStages + 4 + b]));   // rows stored (release, CTA scope)
                if (warp == 2) trace_time(P, it, 6);
            }
        }
    } else if (warp == 6) {
        // ---- publisher: makes finished hidden rows visible device-wide -------------------
        // The device-scope fence has to wait until the epilogue's stores have reached L2, which
        // takes microseconds while TMA loads saturate the memory system; doing it here keeps
        // that wait off the epilogue warps.  Order: epilogue stores -> mbarrier (release/acquire
        // at CTA scope) -> this thread's device-scope fence (cumulative) -> counter increment.
        if (lane == 0) {
            int it = 0;
            for (int u = blockIdx.x; u < total_units; u += gridDim.x, ++it) {
                const Unit un = ut.decode(u);
                const int b = it & 1;
                if (!mbar_wait(smem_u32(&bars[2 * kMaxStages + 4 + b]), (it >> 1) & 1, abort_flag, kWaitLimitNs))
                    break;   // the role that stalled has already reported
                if (un.layer == 0) {
                    __threadfence();
                    fence_proxy_async_all();
                    atomicAdd(P.ready + un.ready_idx, 1);
                }
            }
        }
    }

    // ---- teardown --------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    // The last CTA to finish leaves the dependency counters at zero for the next call.
    if (warp == 2) {
        int last = 0;
        if (lane == 0) {
            __threadfence();
            last = atomicAdd(P.ticket, 1) == static_cast<int>(gridDim.x) - 1;
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            for (int i = lane; i < tt_all; i += 32) P.ready[i] = 0;
            if (lane == 0) *P.ticket = 0;
        }
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

}  // namespace

int launch_ffn_bf16(const monde_problem& p, const void* x_perm, const void* W1, const void* b1,
                    const void* W2, const void* b2, const int32_t* counts, const int32_t* offsets,
                    const int32_t* hot_ids, const int32_t* cold_ids, const int32_t* n_hot_cold,
                    void* y_perm, void* ws, cudaStream_t s) {
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(expert_ffn_kernel<MONDE_ACT_RELU>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (attr_err == cudaSuccess)
            attr_err = cudaFuncSetAttribute(expert_ffn_kernel<MONDE_ACT_GELU_ERF>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    });
    if (attr_err != cudaSuccess) return MONDE_ERR_CUDA;
    char* base = static_cast<char*>(ws);
    const uint64_t A = static_cast<uint64_t>(p.T) * p.top_k;
    FfnParams P;
    P.d_model = p.d_model;
    P.d_ff = p.d_ff;
    P.act = p.act;
    P.b1 = static_cast<const __nv_bfloat16*>(b1);
    P.b2 = static_cast<const __nv_bfloat16*>(b2);
    P.h = reinterpret_cast<__nv_bfloat16*>(base + WsLayout::kHidden);
    P.y = static_cast<__nv_bfloat16*>(y_perm);
    P.counts = counts;
    P.offsets = offsets;
    P.hot_ids = hot_ids;
    P.cold_ids = cold_ids;
    P.n_hot_cold = n_hot_cold;
    P.status = reinterpret_cast<int32_t*>(base + WsLayout::kStatus);
    P.ticket = reinterpret_cast<int32_t*>(base + WsLayout::kCounters);
    P.ready = reinterpret_cast<int32_t*>(base + WsLayout::kTiles);
    P.trace = g_trace;
    P.trace_slots = g_trace_slots;
    CUtensorMap map_w1, map_w2, map_x, map_h;
    if (!make_map(&map_w1, W1, static_cast<uint64_t>(p.E) * p.d_ff, p.d_model, kTileRows)) return MONDE_ERR_CUDA;
    if (!make_map(&map_w2, W2, static_cast<uint64_t>(p.E) * p.d_model, p.d_ff, kTileRows)) return MONDE_ERR_CUDA;
    if (!make_map(&map_x, x_perm, A, p.d_model, 16)) return MONDE_ERR_CUDA;
    if (!make_map(&map_h, P.h, A, p.d_ff, 16)) return MONDE_ERR_CUDA;
    if (p.act == MONDE_ACT_RELU)
        expert_ffn_kernel<MONDE_ACT_RELU><<<sm_count(), kThreads, kSmemBytes, s>>>(map_w1, map_w2, map_x, map_h, P);
    else
        expert_ffn_kernel<MONDE_ACT_GELU_ERF><<<sm_count(), kThreads, kSmemBytes, s>>>(map_w1, map_w2, map_x, map_h, P);
    return launched();
}

}  // namespace monde

// Diagnostic hook (not part of the public header): device buffer of 148 * slots * 8 uint64
// that the FFN kernel fills with a per-unit timeline; pass null to switch it off.
extern "C" void monde_internal_set_trace(void* device_buf, int slots) {
    monde::g_trace = static_cast<unsigned long long*>(device_buf);
    monde::g_trace_slots = slots;
}
