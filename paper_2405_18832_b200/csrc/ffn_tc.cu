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
// A unit covers two 128-feature tiles that share one token tile (the token tile is the
// operand that every feature tile re-reads through L2, so pairing halves that traffic).
//   hot : token tile <= 256 (full-rate 128 x 256 MMAs).  For d_model >= 1536 a unit
//         takes two feature tiles (three 32 KB weight stages, three 32 KB token stages), and
//         the two accumulators fill all 512 TMEM columns, so the epilogue is not overlapped
//         with the next unit's MMAs - cheaper than re-reading a 32 KB token tile per 16 KB
//         weight tile.  In those layers a hot expert of at most 128 rows is staged through
//         128-row token stages (four of 16 KB), which leaves room for a fourth weight stage,
//         and its two accumulators fit one of the two 256-column buffers; such experts follow
//         the larger ones in the list.  For smaller layers the exposed epilogue and the halved
//         unit count cost more than they save: one feature tile per unit (six 16 KB weight
//         stages, three 32 KB token stages), two accumulator buffers;
//   cold: token tile = threshold-1 rounded up to 16 (at most 64), two feature tiles per unit,
//         five 32 KB weight stages and four small token stages, two accumulator buffers -> a
//         deep queue of weight bytes in flight per SM; the tensor core idles most of the time
//         and HBM sets the pace.
// Weight tiles (from HBM, long latency) and token tiles (from L2, re-read by every feature
// tile) have separate rings and separate producer warps.
// Work units (expert, 128-feature tile, token tile) form one ordered list: hot first
// layer, hot second layer, cold first layer, cold second layer.  One persistent CTA per SM
// takes the next unit from a device-wide counter.  A second-layer unit needs the hidden
// rows of its token tile, which are produced by first-layer units earlier in the list:
// per-token-tile counters in the workspace carry that dependency (a unit only ever waits
// for units taken before it, so the wait cannot deadlock), and the TMA producer streams
// the unit's weights while it waits, so weight traffic never stalls at the layer boundary.
// Cold second-layer units are long (K = d_ff) and few; they are split along K into up to
// four sub-units so that the end of the run is not a handful of CTAs each streaming a
// megabyte alone.  Sub-units 0..S-2 store fp32 partial tiles in the workspace; the last
// sub-unit (again later in the list than the ones it waits for) adds them in a fixed
// order, so results stay bit-reproducible.
// Warp roles: warp 0 schedules and issues the weight-tile TMA loads, warp 7 the token-tile
// loads, warp 1 issues MMAs and owns the TMEM allocation, warps 2-5 and 8-11 drain the
// accumulator (bias + activation fused) while the next unit's MMAs run into the second
// accumulator buffer, warp 6 publishes finished rows.  Counts never travel to the host.
// Variants of the same kernel: CTA pairs (template parameter kPair: clusters of two CTAs issue
// one 256-row MMA, tcgen05 cta_group::2; opt-in), and a last store that writes rows in token
// order: with the gate weight applied (top-1 routing) or side by side per token for the combine
// kernel to add (top-k > 1); both behind monde_moe_ffn_combine_fwd.
#include <cuda.h>

#include <algorithm>
#include <mutex>

#include "common.cuh"
#include "sm100.cuh"

namespace monde {

namespace {

using namespace sm100;

constexpr int kThreads = 384;       // weight producer, MMA, 4 epilogue warps, publisher, token-tile producer, 4 more epilogue warps
constexpr int kBlockK = 64;           // K elements per stage: one 128-byte swizzle row
constexpr int kTileRows = 128;        // output features per unit = MMA M
constexpr int kABytes = kTileRows * 128;
constexpr int kMaxStagesA = 10;       // weight-tile ring
constexpr int kMaxStagesB = 4;        // token-tile ring
constexpr int kQueue = 4;            // unit ids in flight between the producer and the other roles
constexpr int kClaimAhead = 6;       // K blocks still to load when the producer takes its next unit
constexpr int kHotTokTile = 256;
constexpr int kSmallHotRows = 128;   // hot experts with at most this many rows: token-tile stages of 128 rows, one more weight stage
constexpr int kTilesPerUnit = 2;      // a unit covers two 128-feature tiles that share one token tile
constexpr int kTileBytes = 200 * 1024;   // operand rings: with 16-row cold token tiles this is six 32 KB weight stages + four token stages
constexpr int kMailSlots = 8;        // unit indices in flight from the leader of a CTA pair to the other CTA
constexpr int kNumBars = 2 * kMaxStagesA + 2 * kMaxStagesB + 6 + 2 * kQueue + kMailSlots + 1;   // + the MMA issuer's way-out barrier
constexpr int kTableInts = 6 * (kMaxExperts + 1);
constexpr int kStageOutBytes = 2 * 2 * 16 * kTileRows * 2;   // per epilogue warp set: two staging buffers of 16 tokens x 128 features
constexpr int kSmemBytes = 1024 + kTileBytes + kNumBars * 8 + 64 + kQueue * 64 + kTableInts * 4 + kStageOutBytes + 16;
constexpr int kTmemCols = 512;        // two accumulator buffers of 256 fp32 columns
constexpr uint64_t kDrainLimitNs = 200000ull;      // on the way out after a wait gave up: time allowed for copies and MMAs in flight to land

enum WaitSite { kSiteProducerEmpty = 1, kSiteMmaFull = 2, kSiteMmaTmemEmpty = 3, kSiteEpilogueTmemFull = 4,
                kSiteHiddenReady = 5, kSiteDrain = 6, kSiteQueue = 7, kSitePartials = 8 };

struct FfnParams {
    int E, d_model, d_ff, act;
    int cold_tile;                // token tile of the cold class
    int pair_mask;                // bit (class * 2 + layer): units of that segment take two feature tiles
    int n_split;                  // K-splits of a cold second-layer unit (1 = none)
    int split_major;              // ordering of the K-split sub-units (see UnitTable::decode)
    const __nv_bfloat16* b1;
    const __nv_bfloat16* b2;
    __nv_bfloat16* h;
    __nv_bfloat16* y;
    const uint8_t* cls;
    const int32_t* counts;
    const int32_t* offsets;
    int32_t* status;       // {status, site}
    int32_t* ticket;       // CTAs that have finished
    int32_t* next_unit;    // device-wide unit counter
    int32_t* part_done;    // per cold second-layer tile: partial tiles finished
    float* partials;       // [tile][split][cold_tile tokens][128 features] fp32
    int32_t* ready;        // per token tile: first-layer units finished
    const int32_t* fuse_perm;    // fused combine: assignment id of every row; null = store y in expert-contiguous order
    const float* fuse_w;         // gate weight per assignment (top-1); null = rows go out unweighted, in assignment order
    __nv_bfloat16* fuse_out;     // out [T, d_model] (top-1) or the token-ordered staging rows [T * top_k, d_model]
    DiagRecord* diag;            // range-check record of the diagnostics build (null otherwise)
    int A;                       // rows of x_perm / h / y_perm
    unsigned long long* trace;   // diagnostic timeline (null in normal use): [cta][unit slot][8]
    int trace_slots;
    int hold_ready;              // diagnostic: first-layer units do not publish their rows
    unsigned long long wait_ns;  // bound of a wait for another unit's results; waits inside the CTA get twice that
};

// Diagnostic timeline: slot 0 unit id, 1-2 producer first/last issue, 3-4 MMA first full / commit,
// 5-6 epilogue start / end (global timer, ns), 7 time the MMA issuer spent waiting for operands (ns).
__device__ __forceinline__ void trace_mark(const FfnParams& P, int it, int slot, unsigned long long v) {
    if (P.trace != nullptr && it < P.trace_slots)
        P.trace[(static_cast<size_t>(blockIdx.x) * P.trace_slots + it) * 8 + slot] = v;
}
__device__ __forceinline__ void trace_time(const FfnParams& P, int it, int slot) {
    if (P.trace != nullptr && it < P.trace_slots)
        P.trace[(static_cast<size_t>(blockIdx.x) * P.trace_slots + it) * 8 + slot] = global_timer_ns();
}

struct Unit {
    int id;       // position in the unit list, -1 = end of list
    int e;        // expert id
    int row0;     // first row of the token tile in the expert-contiguous buffers
    int rows;     // valid token rows in the tile
    int nt;       // rows rounded up to a multiple of 16 (MMA N)
    int n0;       // first output feature of the tile
    int layer;    // 0: h = act(x W1^T + b1), 1: y = h W2^T + b2
    int cold;     // class, selects the stage geometry: 0 hot, 1 cold, 2 hot with at most kSmallHotRows rows
    int ready_idx;  // token-tile index into the dependency counters
    int kb0, kb1;   // K blocks [kb0, kb1) of the reduction handled by this unit
    int split;      // sub-unit index along K, n_split - 1 = the one that finishes the tile
    int n_split;    // sub-units of this tile (1 unless cold second layer)
    int tile_idx;   // cold second-layer unit index (partials / part_done)
    int tiles;      // 128-feature tiles of this unit (1 or 2) sharing one token tile
    int wide;       // 1: the unit's accumulators occupy all 512 TMEM columns (hot, two tiles)
};

static_assert(sizeof(Unit) <= 64, "unit queue slots are 64 bytes");

// Per-CTA copy of the unit list in shared memory.  Entries 0..n_hot-1 are the hot experts (those
// with more than kSmallHotRows rows first, so that each stage geometry is one run of the list),
// n_hot..n_hot+n_cold-1 the cold ones; tt_prefix is the exclusive prefix of token tiles.
struct UnitTable {
    int* tt_prefix;   // [n+1]
    int* e;
    int* off;
    int* m;
    int* tt;          // token tiles of this expert
    int* per;         // tokens per tile (multiple of 16)
    int n_hot, n_all, nt1, nt2;      // 128-feature tiles of layer 1 (d_ff) and layer 2 (d_model)
    int upt[6];                      // units per token tile, by class * 2 + layer (class 2 = class 0)
    int tpu[6];                      // feature tiles per unit, likewise
    int kblocks1, kblocks2;          // 64-wide K blocks of layer 1 (d_model) and layer 2 (d_ff)
    int n_split, kb_per_split, split_major;
    int pair;                        // 1: every unit is run by a pair of CTAs, one feature tile each
    int small_rows;                  // hot experts with at most this many rows form class 2 (0: no such class)
    int seg1, seg2, seg3, total_units;   // list = [hot L1 | hot L2 | cold L1 | cold L2 (split)]

    __device__ __forceinline__ Unit decode(int u) const {
        Unit r;
        r.id = u;
        int v;
        if (u < seg1) { r.cold = 0; r.layer = 0; v = u; }
        else if (u < seg2) { r.cold = 0; r.layer = 1; v = u - seg1; }
        else if (u < seg3) { r.cold = 1; r.layer = 0; v = u - seg2; }
        else { r.cold = 1; r.layer = 1; v = u - seg3; }
        r.split = 0;
        r.n_split = 1;
        const int sgm = r.cold * 2 + r.layer;
        const int lo_entry = r.cold ? n_hot : 0;
        const int tt_base = tt_prefix[lo_entry];
        int lo, local;
        if (r.cold == 1 && r.layer && n_split > 1 && split_major) {
            // K-split segment, split index slowest over the whole segment: every expert's sub-units 0,
            // then 1, ..., and the finishing sub-units (S-1) at the very end of the list, where they
            // find their partial tiles long done and make a short tail.
            r.n_split = n_split;
            const int per_split = (total_units - seg3) / n_split;
            r.split = v / per_split;
            v -= r.split * per_split;
            const int ntl = upt[3];
            lo = lo_entry;
            int hi = n_all - 1;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if ((tt_prefix[mid] - tt_base) * ntl <= v) lo = mid; else hi = mid - 1;
            }
            local = v - (tt_prefix[lo] - tt_base) * ntl;
        } else if (r.cold == 1 && r.layer && n_split > 1) {
            // K-split segment, in slots: slot j holds the partial sub-units (splits 0..S-2, split
            // index slowest) of cold expert j followed by the finishing sub-units (split S-1) of
            // expert j-1.  A finisher is thus taken a good fraction of a scheduling round after the
            // partial tiles it adds (it does not wait for them) yet soon enough to find them in L2.
            r.n_split = n_split;
            const int n = n_all - n_hot;
            const int pm = upt[3] * (n_split - 1), fm = upt[3];
            auto before = [&](int j) {
                return pm * (tt_prefix[lo_entry + min(j, n)] - tt_base) + fm * (tt_prefix[lo_entry + max(j - 1, 0)] - tt_base);
            };
            int a = 0, b = n;                              // largest slot with before(slot) <= v
            while (a < b) {
                const int mid = (a + b + 1) >> 1;
                if (before(mid) <= v) a = mid; else b = mid - 1;
            }
            local = v - before(a);
            const int partial_units = a < n ? pm * tt[lo_entry + a] : 0;
            if (local < partial_units) {
                lo = lo_entry + a;
                const int per_split = tt[lo] * upt[3];
                r.split = local / per_split;
                local -= r.split * per_split;
            } else {
                lo = lo_entry + a - 1;
                local -= partial_units;
                r.split = n_split - 1;
            }
        } else {
            const int ntl = upt[sgm];
            lo = lo_entry;
            int hi = (r.cold ? n_all : n_hot) - 1;      // largest entry with block start <= v
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if ((tt_prefix[mid] - tt_base) * ntl <= v) lo = mid; else hi = mid - 1;
            }
            local = v - (tt_prefix[lo] - tt_base) * ntl;
        }
        const int tok = local % tt[lo];
        const int ntile = local / tt[lo];
        r.e = e[lo];
        r.n0 = ntile * kTileRows * tpu[sgm];
        r.tiles = min(tpu[sgm], (r.layer ? nt2 : nt1) - tpu[sgm] * ntile);
        if (!r.cold && m[lo] <= small_rows) r.cold = 2;
        r.wide = !pair && r.cold == 0 && tpu[sgm] == 2;
        const int r_in_e = tok * per[lo];
        r.rows = min(per[lo], m[lo] - r_in_e);
        r.nt = (r.rows + 15) & ~15;
        r.row0 = off[lo] + r_in_e;
        r.ready_idx = tt_prefix[lo] + tok;
        r.tile_idx = (tt_prefix[lo] - tt_base + tok) * upt[3] + ntile;
        const int kb_all = r.layer ? kblocks2 : kblocks1;
        r.kb0 = r.n_split > 1 ? r.split * kb_per_split : 0;
        r.kb1 = r.n_split > 1 ? min(kb_all, r.kb0 + kb_per_split) : kb_all;
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

// Tensor maps, all 64 columns (128 bytes) wide with the 128-byte swizzle.  Weights: boxes of 128
// and 256 rows (one or two feature tiles per copy).  Token rows (x_perm for layer 1, hidden
// activations for layer 2): boxes of 16, 64 and 256 rows, so that a token tile of any multiple
// of 16 rows is covered by a few large copies (sixteen 2 KB copies per 32 KB token tile made
// the TMA issue rate, not bandwidth, the limit of the hot class).
struct FfnMaps {
    CUtensorMap w[2][2];      // [layer][0: 128 rows, 1: 256 rows]
    CUtensorMap in[2][3];     // [layer][0: 16 rows, 1: 64 rows, 2: 256 rows]
};

template <int kAct, bool kPair>
__global__ void __launch_bounds__(kThreads, 1) expert_ffn_kernel(const __grid_constant__ FfnMaps M, const FfnParams P) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kTileBytes);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* unit_queue = reinterpret_cast<int*>(tmem_slot + 16);      // [kQueue] decoded units, 16 ints each
    int* tab = unit_queue + kQueue * 16;
    __nv_bfloat16* stg = reinterpret_cast<__nv_bfloat16*>(                     // 2 sets x 2 x [16 tokens][128 features]
        (reinterpret_cast<uintptr_t>(tab + kTableInts) + 15) & ~uintptr_t(15));
    UnitTable ut;
    ut.tt_prefix = tab;
    ut.e = tab + (kMaxExperts + 1);
    ut.off = ut.e + (kMaxExperts + 1);
    ut.m = ut.off + (kMaxExperts + 1);
    ut.tt = ut.m + (kMaxExperts + 1);
    ut.per = ut.tt + (kMaxExperts + 1);

    // barrier addresses
    const uint32_t bar0 = smem_u32(bars);
    constexpr int kRingBars = 2 * kMaxStagesA + 2 * kMaxStagesB;
    auto full_a = [&](int s) { return bar0 + 8u * s; };
    auto empty_a = [&](int s) { return bar0 + 8u * (kMaxStagesA + s); };
    auto full_b = [&](int s) { return bar0 + 8u * (2 * kMaxStagesA + s); };
    auto empty_b = [&](int s) { return bar0 + 8u * (2 * kMaxStagesA + kMaxStagesB + s); };
    auto acc_full = [&](int b) { return bar0 + 8u * (kRingBars + b); };
    auto acc_empty = [&](int b) { return bar0 + 8u * (kRingBars + 2 + b); };
    auto rows_stored = [&](int b) { return bar0 + 8u * (kRingBars + 4 + b); };
    auto q_full = [&](int s) { return bar0 + 8u * (kRingBars + 6 + s); };
    auto q_empty = [&](int s) { return bar0 + 8u * (kRingBars + 6 + kQueue + s); };
    auto mail_bar = [&](int s) { return bar0 + 8u * (kRingBars + 6 + 2 * kQueue + s); };
    const uint32_t way_out_bar = bar0 + 8u * (kRingBars + 6 + 2 * kQueue + kMailSlots);
    // Waits on another unit's results (hidden rows, partial tiles) give up after wait_ns; waits on the
    // CTA's own barriers, which can only be waiting for one of those, after twice as long, so that the
    // wait that names the cause is the one that reports.
    const uint64_t kDepWaitNs = P.wait_ns, kWaitLimitNs = 2 * P.wait_ns;
    volatile int* mail = reinterpret_cast<volatile int*>(tmem_slot + 4);   // [kMailSlots]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // K blocks per ring stage.  The MMA issuer spends some 400 cycles per stage on barrier probes
    // and commits, and the tensor core's queue hides only about as much: a stage must carry at
    // least eight MMAs to keep the tensor core busy.  Single CTAs issue 8 per K block (two feature
    // tiles), pairs 4 (one 256-row MMA per 16 columns of K), so pairs stage two K blocks at a time.
    constexpr int kKps = kPair ? 2 : 1;

    // ---- set-up that touches nothing another kernel produced: runs while the preceding
    // kernel of the stream is still finishing --------------------------------------------
    pdl_launch_dependents();
    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kMaxStagesA; ++s) {
            mbar_init(full_a(s), 1);    // weight producer's expect_tx arrival
            mbar_init(empty_a(s), 1);   // one tcgen05.commit
        }
        for (int s = 0; s < kMaxStagesB; ++s) {
            mbar_init(full_b(s), 1);    // token-tile producer's expect_tx arrival
            mbar_init(empty_b(s), 1);   // one tcgen05.commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full(b), 1);      // one commit
            mbar_init(acc_empty(b), kPair ? 18 : 9);   // 8 epilogue warps + the publisher (keeps it at most one use behind), of each CTA
            mbar_init(rows_stored(b), 8);   // 8 epilogue warps
        }
        for (int s = 0; s < kQueue; ++s) {
            mbar_init(q_full(s), 1);        // producer
            mbar_init(q_empty(s), 11);      // MMA issuer, 8 epilogue warps, publisher, token-tile producer
        }
        for (int s = 0; s < kMailSlots; ++s) mbar_init(mail_bar(s), 1);   // the pair leader's scheduler
        mbar_init(way_out_bar, 1);                                        // one commit, only after a wait gave up
        fence_barrier_init();
        for (int l = 0; l < 2; ++l) {
            prefetch_tensormap(&M.w[l][0]);
            prefetch_tensormap(&M.w[l][1]);
            for (int i = 0; i < 3; ++i) prefetch_tensormap(&M.in[l][i]);
        }
    } else if (warp == 1) {
        if (kPair) {
            tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(tmem_slot), kTmemCols);
            tmem_relinquish();
        }
    }
    pdl_wait();

    // Every unit, the first included, comes from the device-wide counter: a unit is only ever held
    // by a CTA that is running, so a launch whose CTAs are not all resident at once (another
    // kernel holding some SMs) still cannot wait on a unit that nobody is working on.  The draw is
    // issued here and its answer used after the unit table is built, which hides the round trip.
    int first_draw = 0;
    if (warp == 0 && lane == 0 && (!kPair || cluster_ctarank() == 0)) first_draw = atomicAdd(P.next_unit, 1);

    // ---- unit table from the router's outputs -----------------------------------------------
    // Thread e reads expert e's class, count and offset (independent loads: one round trip to
    // memory instead of the three that following n_hot_cold -> id lists -> counts would take) and
    // the entries are compacted in expert order, which is the order of the router's id lists.
    // Hot experts with more than kSmallHotRows rows come first, then the other hot ones, then the cold.
    // The split is made only where hot units carry two feature tiles (wide models): there a token
    // tile of 128 rows instead of 256 leaves room for a fourth 32 KB weight stage, and weight bytes
    // in flight are what bounds a unit with few rows.  With one-tile units the ring is already six
    // stages deep and regrouping the list measured slightly slower, so the list keeps expert order.
    const int small_rows = (P.pair_mask & 1) ? kSmallHotRows : 0;
    ut.small_rows = small_rows;
    __shared__ int s_warp_big[kThreads / 32], s_warp_small[kThreads / 32], s_warp_cold[kThreads / 32], s_n_hot, s_n_all;
    {
        const int e = tid;
        const int k = e < P.E ? P.cls[e] : 0;
        const int m = e < P.E ? P.counts[e] : 0;
        const int off = e < P.E ? P.offsets[e] : 0;
        const bool small = k == 2 && m <= small_rows;
        const unsigned big_mask = __ballot_sync(0xffffffffu, k == 2 && !small);
        const unsigned small_mask = __ballot_sync(0xffffffffu, small);
        const unsigned cold_mask = __ballot_sync(0xffffffffu, k == 1);
        if (lane == 0) {
            s_warp_big[warp] = __popc(big_mask);
            s_warp_small[warp] = __popc(small_mask);
            s_warp_cold[warp] = __popc(cold_mask);
        }
        __syncthreads();
        int big_before = 0, small_before = 0, cold_before = 0, n_big = 0, n_small = 0, n_cold = 0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) {
            if (w < warp) { big_before += s_warp_big[w]; small_before += s_warp_small[w]; cold_before += s_warp_cold[w]; }
            n_big += s_warp_big[w];
            n_small += s_warp_small[w];
            n_cold += s_warp_cold[w];
        }
        const int n_hot = n_big + n_small;
        if (tid == 0) { s_n_hot = n_hot; s_n_all = n_hot + n_cold; }
        if (k != 0) {
            const bool cold = k == 1;
            const unsigned lt = (1u << lane) - 1u;
            const int i = cold ? n_hot + cold_before + __popc(cold_mask & lt)
                               : (small ? n_big + small_before + __popc(small_mask & lt) : big_before + __popc(big_mask & lt));
            const int tile = cold ? P.cold_tile : kHotTokTile;
            const int tt = max(1, (m + tile - 1) / tile);
            ut.e[i] = e;
            ut.off[i] = off;
            ut.m[i] = m;
            ut.tt[i] = tt;
            ut.per[i] = ((m + tt - 1) / tt + 15) & ~15;
            ut.tt_prefix[i + 1] = tt;
        }
    }
    if (tid == 0) ut.tt_prefix[0] = 0;
    __syncthreads();
    ut.n_hot = s_n_hot;
    ut.n_all = s_n_all;
    ut.nt1 = (P.d_ff + kTileRows - 1) / kTileRows;
    ut.nt2 = (P.d_model + kTileRows - 1) / kTileRows;
#pragma unroll
    for (int g = 0; g < 6; ++g) {
        ut.tpu[g] = ((P.pair_mask >> (g & 3)) & 1) + 1;     // classes 0 and 2 are both the hot class
        ut.upt[g] = (((g & 1) ? ut.nt2 : ut.nt1) + ut.tpu[g] - 1) / ut.tpu[g];
    }
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
    }
    tc_fence_before_sync();
    __syncthreads();
    if (kPair) cluster_sync_all();   // the other CTA's barriers and tensor memory exist from here on
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // CTA pairs: rank within the pair, and the leader's copy of the barrier array (the full and
    // accumulator-free barriers that the MMA issuer waits on live in the leader only).
    const uint32_t rank = kPair ? cluster_ctarank() : 0u;
    const uint32_t bar0_leader = kPair ? map_to_cta(bar0, 0) : bar0;
    const int tt_all = ut.tt_prefix[ut.n_all];
    const int tt_hot = ut.tt_prefix[ut.n_hot];
    ut.kblocks1 = P.d_model / kBlockK;
    ut.kblocks2 = P.d_ff / kBlockK;
    ut.n_split = P.n_split;
    ut.split_major = P.split_major;
    ut.pair = kPair;
    ut.kb_per_split = (ut.kblocks2 + P.n_split - 1) / P.n_split;
    ut.seg1 = tt_hot * ut.upt[0];
    ut.seg2 = ut.seg1 + tt_hot * ut.upt[1];
    ut.seg3 = ut.seg2 + (tt_all - tt_hot) * ut.upt[2];
    ut.total_units = ut.seg3 + (tt_all - tt_hot) * ut.upt[3] * P.n_split;
    const uint32_t tiles_u32 = smem_u32(smem);
    // Ring geometry of a segment.  Weight tiles come from DRAM (long latency) and token tiles from
    // L2 (short latency, re-read by every feature tile), so they get separate rings: a few
    // token-tile stages fetched just in time, and all remaining shared memory as weight stages
    // in flight.  (With one combined ring the hot class had 48 KB of weights in flight per SM
    // and ran at the latency limit, 77 GB/s of fill per SM.)
    struct Geom { int a_bytes, b_bytes, na, nb, b_base; };
    auto geom_of = [&](int g) {
        Geom r;
        r.a_bytes = kPair ? kKps * kABytes : ut.tpu[g] * kABytes;                        // per CTA
        const int cl = g >> 1;                       // 0 hot, 1 cold, 2 hot with few rows
        r.b_bytes = (cl == 1 ? P.cold_tile : (cl == 2 ? kSmallHotRows : kHotTokTile)) * (kPair ? kKps * 64 : 128);   // a pair holds half the tokens each
        r.nb = cl == 0 ? 3 : 4;
        r.na = min(kMaxStagesA, (kTileBytes - r.nb * r.b_bytes) / r.a_bytes);
        r.b_base = r.na * r.a_bytes;
        return r;
    };
    auto same_geom = [](const Geom& x, const Geom& y) {
        return x.a_bytes == y.a_bytes && x.b_bytes == y.b_bytes && x.na == y.na && x.nb == y.nb;
    };

    // The producer decodes every unit once, one unit ahead of its loads, and hands the decoded
    // record to the other roles through a small shared-memory queue (decoding costs about half
    // a microsecond of dependent shared-memory loads and divisions: too much to repeat in every
    // role at the start of every 6 us unit).  id = -1 marks the end of the list or a wait that
    // gave up.  `whole_warp`: all 32 lanes call (epilogue warps); otherwise a single lane calls.
    auto pop_unit = [&](int it, bool whole_warp) -> Unit {
        const int slot = it % kQueue;
        Unit un;
        if (!mbar_wait(q_full(slot), (it / kQueue) & 1, abort_flag, kWaitLimitNs)) {
            un.id = -1;
            return un;
        }
        un = *reinterpret_cast<const Unit*>(unit_queue + slot * 16);
        if (whole_warp) __syncwarp();
        if (lane == 0) mbar_arrive(q_empty(slot));
        return un;
    };

    // Accumulator buffers.  A narrow unit (cold, or hot with one feature tile) uses one of two
    // 256-column buffers in turn (its tiles at +0 and +128); a wide unit (hot, two tiles of up
    // to 256 tokens) fills all 512 columns (tiles at 0 and 256) and is tracked as buffer 0.
    // The narrow unit that follows a wide one starts again at buffer 0, so waiting for that
    // buffer also waits for the wide unit's drain; a wide unit that follows narrow ones
    // additionally waits for buffer 1 (see the MMA issuer).  Every role walks the same
    // sequence and keeps the same counts.
    struct AccCursor {
        int uses0 = 0, uses1 = 0;
        int seq = 0;
        int b = 0;
        uint32_t parity = 0;        // parity of this use of buffer b (full: wait parity, empty: wait parity ^ 1)
        uint32_t other_parity = 0;  // parity that tells buffer 1's latest use has been drained (wide units)
        __device__ void next(const Unit& un) {
            b = un.wide ? 0 : (seq++ & 1);
            if (un.wide) seq = 0;
            other_parity = (uses1 & 1) ^ 1;
            if (b == 0) { parity = uses0 & 1; ++uses0; } else { parity = uses1 & 1; ++uses1; }
        }
    };
    auto acc_col = [](const Unit& un, int b, int t) { return un.wide ? t * 256 : b * 256 + t * 128; };

    if (warp == 0) {
        // ---- scheduler + TMA producer ------------------------------------------------------
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first();   // weights are read once
            int stage = 0, cls = -1;
            Geom gm = {};
            uint32_t fill_bits = 0;     // bit s: parity of the number of fills of stage s
            uint32_t filled = 0;        // bit s: stage s has been filled at least once
            bool ok = true;
            // Publishes unit number `j` of this CTA (or the end marker) to the other roles.
            auto push_unit = [&](int j, const Unit& un) -> bool {
                const int slot = j % kQueue;
                if (!mbar_wait(q_empty(slot), ((j / kQueue) & 1) ^ 1, abort_flag, kWaitLimitNs)) {
                    report_timeout(P.status, abort_flag, kSiteQueue);
                    return false;
                }
                *reinterpret_cast<Unit*>(unit_queue + slot * 16) = un;
                mbar_arrive(q_full(slot));          // release: the record is visible to whoever acquires
                return true;
            };
            // In a CTA pair the
            // leader draws from the counter and posts the index into the other CTA's mailbox (a
            // remote store released by a remote mbarrier arrival).  The other CTA's loads gate the
            // leader's MMAs, so it is never more than five draws behind and eight slots suffice.
            int draws = 0;
            auto draw = [&]() -> int {
                if (draws == 0) return first_draw;      // drawn before the unit table was built
                return atomicAdd(P.next_unit, 1);
            };
            auto take_next = [&]() -> int {
                if (!kPair) {
                    const int idx = draw();
                    ++draws;
                    return idx;
                }
                const int slot = draws % kMailSlots;
                const uint32_t parity = (draws / kMailSlots) & 1;
                if (rank == 0) {
                    const int idx = draw();
                    ++draws;
                    st_cluster_u32(map_to_cta(smem_u32(const_cast<int*>(mail) + slot), 1), static_cast<uint32_t>(idx));
                    mbar_arrive_cluster(map_to_cta(mail_bar(slot), 1));
                    return idx;
                }
                ++draws;
                if (!mbar_wait_cluster(mail_bar(slot), parity, abort_flag, kWaitLimitNs)) {
                    report_timeout(P.status, abort_flag, kSiteQueue);
                    return 0x7fffffff;
                }
                return mail[slot];
            };
            // Diagnostics build: a decoded unit whose rows or features fall outside the problem is recorded
            // and ends this CTA's list (nothing of it is loaded or stored).
            auto checked = [&](Unit un) -> Unit {
                [[maybe_unused]] const int N = un.layer ? P.d_model : P.d_ff;
                if (!MONDE_IN_RANGE(un.row0 >= 0 && un.rows > 0 && un.row0 + un.rows <= P.A, P.diag, 4, un.row0) ||
                    !MONDE_IN_RANGE(un.e >= 0 && un.e < P.E && un.n0 >= 0 && un.n0 < N && un.kb0 >= 0 && un.kb0 < un.kb1,
                                    P.diag, 5, un.n0)) {
                    if (atomicCAS(P.status, 0, MONDE_ERR_BOUNDS) == 0) P.status[1] = un.id;
                    un.id = -1;
                }
                return un;
            };
            Unit cur, nxt;
            const int u = take_next();
            cur.id = -1;
            if (u < ut.total_units) cur = checked(ut.decode(u));
            ok = push_unit(0, cur);
            int u_ahead = cur.id >= 0 ? take_next() : 0;   // used a few K blocks later
            for (int it = 0; ok && cur.id >= 0; ++it) {
                const Unit un = cur;
                trace_mark(P, it, 0, static_cast<unsigned long long>(un.id));
                if (un.cold * 2 + un.layer != cls) {
                    const Geom g2 = geom_of(un.cold * 2 + un.layer);
                    if (cls < 0 || !same_geom(g2, gm)) {
                        // geometry switch: every stage filled so far must have been consumed
                        for (int s = 0; ok && cls >= 0 && s < gm.na; ++s)
                            if (!mbar_wait(empty_a(s), ((fill_bits >> s) & 1u) ^ 1u, abort_flag, kWaitLimitNs)) {
                                report_timeout(P.status, abort_flag, kSiteDrain);
                                ok = false;
                            }
                        if (!ok) break;
                        gm = g2;
                        stage = 0;
                    }
                    cls = un.cold * 2 + un.layer;
                }
                const CUtensorMap* mw = &M.w[un.layer][kPair ? 0 : un.tiles - 1];   // single CTA: both feature tiles in one copy
                const int N = un.layer ? P.d_model : P.d_ff;
                // loop state in registers (see the MMA issuer)
                const int kb0 = un.kb0, kb1 = un.kb1, a_bytes = gm.a_bytes, na = gm.na;
                const int w_row = un.e * N + un.n0 + (kPair ? static_cast<int>(rank) * kTileRows : 0);
                const uint32_t tx_bytes = un.tiles * kABytes;
                const bool trace_on = P.trace != nullptr;
                bool next_ready = false;
                for (int kb = kb0; kb < kb1; kb += kKps) {
                    if (!next_ready && (kb1 - kb <= kClaimAhead || kb + kKps >= kb1)) {
                        // take, decode and publish the next unit while this one's last loads are in flight
                        // (not earlier: a unit claimed at the start of a long one would sit unworked for
                        // the whole of it while other SMs run out of units of its kind)
                        nxt.id = -1;
                        if (u_ahead < ut.total_units) {
                            nxt = checked(ut.decode(u_ahead));
                            u_ahead = take_next();
                        }
                        if (!push_unit(it + 1, nxt)) { ok = false; break; }
                        next_ready = true;
                    }
                    if (!mbar_wait(empty_a(stage), ((fill_bits >> stage) & 1u) ^ 1u, abort_flag, kWaitLimitNs)) {
                        report_timeout(P.status, abort_flag, kSiteProducerEmpty);
                        ok = false;
                        break;
                    }
                    if (trace_on && kb == kb0) trace_time(P, it, 1);
                    const uint32_t a_dst = tiles_u32 + stage * a_bytes;
                    if (kPair) {
                        // each CTA streams its own feature tile; the leader's barrier counts both
                        const int nk = min(kKps, kb1 - kb);
                        if (rank == 0) mbar_arrive_expect_tx(full_a(stage), 2 * nk * kABytes);
                        for (int j = 0; j < nk; ++j)
                            tma_load_2d_pair(a_dst + j * kABytes, mw, bar0_leader + 8u * stage, (kb + j) * kBlockK, w_row, pol_w);
                    } else {
                        const uint32_t full = full_a(stage);
                        mbar_arrive_expect_tx(full, tx_bytes);
                        tma_load_2d(a_dst, mw, full, kb * kBlockK, w_row, pol_w);
                    }
                    fill_bits ^= 1u << stage;
                    filled |= 1u << stage;
                    if (++stage == na) stage = 0;
                }
                trace_time(P, it, 2);
                cur = nxt;
            }
            // A CTA must not exit while bulk copies into its shared memory are outstanding.  After a
            // normal run every fill has been consumed (the MMA issuer waited for it) and these probes
            // answer at once; after a wait gave up, the last fills may still be in flight: wait for
            // them, bounded by time alone.  (Pairs: the leader's barriers count both CTAs' copies and
            // the cluster barrier in the teardown holds the other CTA until the leader is through.)
            if (!kPair || rank == 0)
                for (int s = 0; s < kMaxStagesA; ++s)
                    if ((filled >> s) & 1u) mbar_wait_deadline(full_a(s), ((fill_bits >> s) & 1u) ^ 1u, kDrainLimitNs);
        }
    } else if (warp == 7) {
        // ---- token-tile producer (operand B: rows of x_perm or of the hidden activations) -------
        if (lane == 0) {
            const uint64_t pol_x = policy_evict_last();    // token tiles are re-read by every feature tile
            int stage = 0, cls = -1;
            Geom gm = {};
            uint32_t fill_bits = 0, filled = 0;
            bool ok = true;
            for (int it = 0; ok; ++it) {
                const Unit un = pop_unit(it, false);
                if (un.id < 0) break;
                if (un.cold * 2 + un.layer != cls) {
                    const Geom g2 = geom_of(un.cold * 2 + un.layer);
                    if (cls < 0 || !same_geom(g2, gm)) {
                        for (int s = 0; ok && cls >= 0 && s < gm.nb; ++s)
                            if (!mbar_wait(empty_b(s), ((fill_bits >> s) & 1u) ^ 1u, abort_flag, kWaitLimitNs)) {
                                report_timeout(P.status, abort_flag, kSiteDrain);
                                ok = false;
                            }
                        if (!ok) break;
                        gm = g2;
                        stage = 0;
                    }
                    cls = un.cold * 2 + un.layer;
                }
                const CUtensorMap* mi = M.in[un.layer];
                if (un.layer == 1) {
                    // the hidden rows of this token tile must be complete (its weights already stream)
                    const int32_t* flag = P.ready + un.ready_idx;
                    const int ready_target = ut.upt[un.cold * 2] * (kPair ? 2 : 1);   // first-layer units per token tile (x CTAs)
                    if (ld_acquire(flag) < ready_target) {
                        const uint64_t t0 = global_timer_ns();
                        while (ld_acquire(flag) < ready_target) {
                            if (*abort_flag != 0 || global_timer_ns() - t0 > kDepWaitNs) {
                                report_timeout(P.status, abort_flag, kSiteHiddenReady);
                                ok = false;
                                break;
                            }
                        }
                        if (!ok) break;
                    }
                    fence_proxy_async_all();
                }
                // loop state in registers (see the MMA issuer)
                const int kb0 = un.kb0, kb1 = un.kb1, nt = un.nt, row0 = un.row0, b_bytes = gm.b_bytes, nb = gm.nb;
                const uint32_t b_ring = tiles_u32 + gm.b_base;
                for (int kb = kb0; kb < kb1; kb += kKps) {
                    if (!mbar_wait(empty_b(stage), ((fill_bits >> stage) & 1u) ^ 1u, abort_flag, kWaitLimitNs)) {
                        report_timeout(P.status, abort_flag, kSiteProducerEmpty);
                        ok = false;
                        break;
                    }
                    const uint32_t b_dst = b_ring + stage * b_bytes;
                    if (kPair) {
                        // this CTA's half of the token rows, in boxes of 128, 32 and 8 rows
                        const int half = nt >> 1, r0 = row0 + static_cast<int>(rank) * half;
                        const uint32_t full = bar0_leader + 8u * (2 * kMaxStagesA + stage);
                        const int nk = min(kKps, kb1 - kb);
                        if (rank == 0) mbar_arrive_expect_tx(full_b(stage), nk * nt * 128);
                        for (int jk = 0; jk < nk; ++jk) {
                            const uint32_t dst = b_dst + jk * (b_bytes / kKps);
                            const int x = (kb + jk) * kBlockK;
                            int j = 0;
                            for (; half - j >= 128; j += 128) tma_load_2d_pair(dst + j * 128, mi + 2, full, x, r0 + j, pol_x);
                            for (; half - j >= 32; j += 32) tma_load_2d_pair(dst + j * 128, mi + 1, full, x, r0 + j, pol_x);
                            for (; half - j >= 8; j += 8) tma_load_2d_pair(dst + j * 128, mi, full, x, r0 + j, pol_x);
                        }
                    } else {
                        const uint32_t full = full_b(stage);
                        mbar_arrive_expect_tx(full, nt * 128);
                        int j = 0;
                        for (; nt - j >= 256; j += 256)
                            tma_load_2d(b_dst + j * 128, mi + 2, full, kb * kBlockK, row0 + j, pol_x);
                        for (; nt - j >= 64; j += 64)
                            tma_load_2d(b_dst + j * 128, mi + 1, full, kb * kBlockK, row0 + j, pol_x);
                        for (; nt - j >= 16; j += 16)
                            tma_load_2d(b_dst + j * 128, mi, full, kb * kBlockK, row0 + j, pol_x);
                    }
                    fill_bits ^= 1u << stage;
                    filled |= 1u << stage;
                    if (++stage == nb) stage = 0;
                }
            }
            // copies in flight into this CTA's shared memory must land before it exits (see the weight producer)
            if (!kPair || rank == 0)
                for (int s = 0; s < kMaxStagesB; ++s)
                    if ((filled >> s) & 1u) mbar_wait_deadline(full_b(s), ((fill_bits >> s) & 1u) ^ 1u, kDrainLimitNs);
        }
    } else if (warp == 1) {
        // ---- MMA issuer --------------------------------------------------------------
        if (lane == 0) {
            int sa = 0, sb = 0, cls = -1;
            Geom gm = {};
            uint32_t use_a = 0, use_b = 0;   // bit s: parity of the number of uses of stage s of each ring
            bool ok = true;
            AccCursor acc;
            for (int it = 0; ok; ++it) {
                const Unit un = pop_unit(it, false);
                if (un.id < 0) break;
                if (kPair && rank != 0) continue;    // the leader issues for both CTAs
                if (un.cold * 2 + un.layer != cls) {
                    const Geom g2 = geom_of(un.cold * 2 + un.layer);
                    if (cls < 0 || !same_geom(g2, gm)) {
                        gm = g2;
                        sa = 0;
                        sb = 0;
                    }
                    cls = un.cold * 2 + un.layer;
                }
                acc.next(un);
                const int b = acc.b;
                if (!mbar_wait(acc_empty(b), acc.parity ^ 1u, abort_flag, kWaitLimitNs) ||
                    (un.wide && !mbar_wait(acc_empty(1), acc.other_parity, abort_flag, kWaitLimitNs))) {
                    report_timeout(P.status, abort_flag, kSiteMmaTmemEmpty);
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t idesc = kPair ? idesc_bf16_m256(un.nt) : idesc_bf16_m128(un.nt);
                // Everything the K loop needs sits in registers: this thread's instruction stream is
                // what feeds the tensor core, and a reload after every inline-assembly statement
                // (they act as compiler barriers) showed up as hundreds of cycles per K block.
                const int kb0 = un.kb0, kb1 = un.kb1, tiles = un.tiles;
                const int a_bytes = gm.a_bytes, b_bytes = gm.b_bytes, na = gm.na, nb = gm.nb;
                const uint32_t a_ring = tiles_u32, b_ring = tiles_u32 + gm.b_base;
                const uint32_t acc0 = tmem_base + (kPair ? b * 256 : acc_col(un, b, 0));
                const uint32_t acc1 = tmem_base + (kPair ? b * 256 : acc_col(un, b, 1));
                const bool trace_on = P.trace != nullptr;
                bool stage_ready = false;       // the next K block's barriers were probed during this one's MMAs
                unsigned long long waited = 0;   // diagnostic timeline: time spent waiting for operands
                for (int kb = kb0; kb < kb1; kb += kKps) {
                    const unsigned long long w0 = trace_on && !stage_ready ? global_timer_ns() : 0;
                    if (!stage_ready &&
                        (!mbar_wait(full_a(sa), (use_a >> sa) & 1u, abort_flag, kWaitLimitNs) ||
                         !mbar_wait(full_b(sb), (use_b >> sb) & 1u, abort_flag, kWaitLimitNs))) {
                        report_timeout(P.status, abort_flag, kSiteMmaFull);
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    if (trace_on && !stage_ready) waited += global_timer_ns() - w0;
                    if (trace_on && kb == kb0) trace_time(P, it, 3);
                    const uint32_t a_addr = a_ring + sa * a_bytes;
                    const uint32_t b_addr = b_ring + sb * b_bytes;
                    const uint32_t later = kb != kb0;      // 0 for the K block that initialises the accumulator
                    if (kPair) {
                        // 256-row MMAs: this CTA's feature tile and the other CTA's, each against
                        // all token rows (half of them staged in either CTA); a stage holds two K blocks
                        const int nk = min(kKps, kb1 - kb);
                        for (int j = 0; j < nk; ++j) {
                            const uint64_t a_desc = smem_desc_sw128(a_addr + j * kABytes);
                            const uint64_t bj_desc = smem_desc_sw128(b_addr + j * (b_bytes / kKps));
#pragma unroll
                            for (int k4 = 0; k4 < kBlockK / 16; ++k4)
                                umma_bf16_pair(acc0, a_desc + 2 * k4, bj_desc + 2 * k4, idesc, later | (j != 0) | (k4 != 0));
                        }
                        umma_commit_pair(empty_a(sa));   // frees the stage in both CTAs
                        umma_commit_pair(empty_b(sb));
                    } else {
                        const uint64_t b_desc = smem_desc_sw128(b_addr);
                        const uint64_t a_desc = smem_desc_sw128(a_addr);
                        // rings have at least three stages, so the next stage is not this one and its use
                        // bit is still that of its next fill; past the unit's last K block the answer is unused
                        const int sa_next = sa + 1 == na ? 0 : sa + 1, sb_next = sb + 1 == nb ? 0 : sb + 1;
                        stage_ready = umma_bf16_x4_probe(acc0, a_desc, b_desc, idesc, later, full_a(sa_next),
                                                         (use_a >> sa_next) & 1u, full_b(sb_next), (use_b >> sb_next) & 1u) &&
                                      kb + 1 < kb1;
                        if (tiles == 2) {                  // the second feature tile shares the token tile
                            const uint64_t a1_desc = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
                            for (int k4 = 0; k4 < kBlockK / 16; ++k4)
                                umma_bf16(acc1, a1_desc + 2 * k4, b_desc + 2 * k4, idesc, later | (k4 != 0));
                        }
                        umma_commit(empty_a(sa));   // both stages reusable once these MMAs finish
                        umma_commit(empty_b(sb));
                    }
                    use_a ^= 1u << sa;
                    use_b ^= 1u << sb;
                    if (++sa == na) sa = 0;
                    if (++sb == nb) sb = 0;
                }
                if (ok) {                           // accumulator complete
                    if (kPair) umma_commit_pair(acc_full(b)); else umma_commit(acc_full(b));
                }
                trace_time(P, it, 4);
                trace_mark(P, it, 7, waited);
            }
            // Leaving because a wait gave up (here or in another role): MMAs issued so far may still be
            // reading shared memory and writing tensor memory.  One more commit on a barrier of its own
            // tells when they are done; the teardown frees tensor memory only after that.
            if ((!ok || *abort_flag != 0) && (!kPair || rank == 0)) {
                if (kPair) umma_commit_pair(way_out_bar); else umma_commit(way_out_bar);
                mbar_wait_deadline(way_out_bar, 0, kDrainLimitNs);
            }
        }
    } else if (warp < 6 || warp >= 8) {
        // ---- epilogue: TMEM -> registers -> bias, activation -> shared -> global -------------
        // Two sets of four warps (2-5 and 8-11): a warp may only read the TMEM lanes of quarter warp % 4,
        // so each set covers all 128 features; set s drains the 16-token groups of parity s.  One warp per
        // scheduler did not hide the latencies of its own 110 instructions per group; two interleave.
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int set = warp >= 8;
        const int bar_id = 1 + set;             // named barrier of the set
        __nv_bfloat16* const stg_set = stg + set * (2 * 16 * kTileRows);
        AccCursor acc;
        for (int it = 0;; ++it) {
            const Unit un = pop_unit(it, true);
            bool got = un.id >= 0;
            if (got) acc.next(un);
            const int b = acc.b;
            if (got) {
                got = mbar_wait(acc_full(b), acc.parity, abort_flag, kWaitLimitNs);
                if (!got) report_timeout(P.status, abort_flag, kSiteEpilogueTmemFull);
            }
            // the four epilogue warps share a named barrier below: leave together or not at all
            uint32_t all_got;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.u32 q, %1, 0;\n\t"
                "bar.red.and.pred p, %2, 128, q;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(all_got) : "r"(static_cast<uint32_t>(got)), "r"(bar_id) : "memory");
            if (!all_got) break;
            tc_fence_after_sync();
            if (warp == 2 && lane == 0) trace_time(P, it, 5);
            const int N = un.layer ? P.d_model : P.d_ff;
            const __nv_bfloat16* bias = un.layer ? P.b2 : P.b1;
            // unit fields used per token group, in registers (see the MMA issuer)
            const int u_rows = un.rows, u_row0 = un.row0, u_nt = un.nt, u_split = un.split, u_nsplit = un.n_split;
            const bool is_partial = u_split + 1 < u_nsplit;
            if (u_nsplit > 1 && !is_partial) {
                // finishing sub-unit: the partial tiles were taken from the list before this one
                if (lane == 0) {
                    const int32_t* flag = P.part_done + un.tile_idx;
                    const uint64_t t0 = global_timer_ns();
                    while (ld_acquire(flag) < (u_nsplit - 1) * (kPair ? 2 : 1)) {
                        if (*abort_flag != 0 || global_timer_ns() - t0 > kDepWaitNs) {
                            report_timeout(P.status, abort_flag, kSitePartials);
                            break;   // the sums below are wrong but every access stays in bounds
                        }
                    }
                }
                __syncwarp();
            }
            int grp = 0;       // running 16-token group count: alternates the two staging buffers
#pragma unroll 1
            for (int ft = kPair ? static_cast<int>(rank) : 0; ft < (kPair ? static_cast<int>(rank) + 1 : un.tiles); ++ft) {
            const int n0 = un.n0 + ft * kTileRows;
            const int n = n0 + q * 32 + lane;
            const float bias_v = (bias != nullptr && n < N) ? __bfloat162float(bias[static_cast<int64_t>(un.e) * N + n]) : 0.0f;
            const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + (kPair ? b * 256 : acc_col(un, b, ft));
            __nv_bfloat16* out = un.layer ? P.y : P.h;
            const int et = set ? tid - 256 : tid - 64;   // 0..127 within the set
            const int rd_row = et >> 4, rd_col = (et & 15) * 8;
            const bool col_ok = n0 + rd_col < N;     // N is a multiple of 64: 8-wide groups are all in or all out
            // Each group of 16 tokens is transposed through shared memory so that global stores are
            // 16-byte pieces of 256-byte contiguous row segments.  The code is kept small on purpose:
            // a widely unrolled epilogue with an inlined library erf per element overflowed the
            // instruction cache and ran 20x slower.
            // K-split tiles: fp32 partials live as [split][token][feature] so that a warp touches
            // 128 contiguous bytes per token.
            const int cold_tile = P.cold_tile;
            float* part = P.partials + static_cast<size_t>(un.tile_idx * kTilesPerUnit + ft) * (u_nsplit - 1) *
                                           (cold_tile * kTileRows) + q * 32 + lane;
            // One group = 16 tokens.  mode: 0 first layer (activation), 1 second layer, 2 second
            // layer finishing a K-split tile (adds the partial tiles), 3 partial tile (fp32 store).
            const int mode = un.layer == 0 ? 0 : (u_nsplit == 1 ? 1 : (is_partial ? 3 : 2));
            const bool fused = P.fuse_out != nullptr && (mode == 1 || mode == 2);
            auto drain16 = [&](const uint32_t (&v)[16], int c0) {
                if (mode == 3) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        part[(u_split * cold_tile + c0 + j) * kTileRows] = __uint_as_float(v[j]);
                    return;
                }
                // fused combine: the token and gate weight of the two rows this thread stores are
                // fetched now and used after the transpose
                int f_tok[2] = {0, 0};
                float f_w[2] = {0.0f, 0.0f};
                if (fused) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int r = rd_row + half * 8;
                        if (c0 + r < u_rows) {
                            f_tok[half] = __ldg(P.fuse_perm + u_row0 + c0 + r);     // assignment id (top-1: = token id)
                            if (P.fuse_w != nullptr) f_w[half] = __ldg(P.fuse_w + f_tok[half]);
                        }
                    }
                }
                __nv_bfloat16* sb = stg_set + (grp & 1) * (16 * kTileRows) + q * 32 + lane;
                if (mode == 0) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        sb[j * kTileRows] = __float2bfloat16_rn(activate<kAct>(__uint_as_float(v[j]) + bias_v));
                } else if (mode == 1) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        sb[j * kTileRows] = __float2bfloat16_rn(__uint_as_float(v[j]) + bias_v);
                } else {
                    // all partial tiles are requested before any is used: one trip to L2 per group
                    // instead of one per split; summed in a fixed order: split 0, 1, 2, own
                    const float* ps = part + c0 * kTileRows;
                    const int stride = cold_tile * kTileRows;
                    float p0[16], p1[16], p2[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        p0[j] = __ldcg(ps + j * kTileRows);
                        p1[j] = u_nsplit > 2 ? __ldcg(ps + stride + j * kTileRows) : 0.0f;
                        p2[j] = u_nsplit > 3 ? __ldcg(ps + 2 * stride + j * kTileRows) : 0.0f;
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        sb[j * kTileRows] = __float2bfloat16_rn(((p0[j] + p1[j]) + p2[j]) + __uint_as_float(v[j]) + bias_v);
                }
                asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
                const __nv_bfloat16* rb = stg_set + (grp & 1) * (16 * kTileRows);
                ++grp;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = rd_row + half * 8;
                    if (col_ok && c0 + r < u_rows) {
                        const uint4 val = *reinterpret_cast<const uint4*>(rb + r * kTileRows + rd_col);
                        if (fused) {
                            // out[token] = gate weight x the bf16-rounded expert output, rounded once more:
                            // the bytes monde_combine would produce from y_perm
                            const uint32_t w4[4] = {val.x, val.y, val.z, val.w};
                            uint32_t o4[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float lo = __uint_as_float(w4[i] << 16), hi = __uint_as_float(w4[i] & 0xFFFF0000u);
                                const __nv_bfloat162 pr = __floats2bfloat162_rn(fmaf(f_w[half], lo, 0.0f), fmaf(f_w[half], hi, 0.0f));
                                o4[i] = P.fuse_w != nullptr ? *reinterpret_cast<const uint32_t*>(&pr) : w4[i];   // staging rows keep y as it is
                            }
                            *reinterpret_cast<uint4*>(P.fuse_out + static_cast<int64_t>(f_tok[half]) * N + n0 + rd_col) =
                                make_uint4(o4[0], o4[1], o4[2], o4[3]);
                        } else {
                            *reinterpret_cast<uint4*>(out + static_cast<int64_t>(u_row0 + c0 + r) * N + n0 + rd_col) = val;
                        }
                    }
                }
            };
            // Two 16-column loads in flight, ping-pong; the loop is kept rolled so that the whole
            // epilogue stays a few KB of code.
            uint32_t va[16], vb[16];
            int c0 = 16 * set;
            if (c0 < u_nt) tmem_ld_16(t_addr + c0, va);
#pragma unroll 1
            for (; c0 < u_nt; c0 += 64) {
                tmem_ld_wait();
                if (c0 + 32 < u_nt) tmem_ld_16(t_addr + c0 + 32, vb);
                drain16(va, c0);
                if (c0 + 32 < u_nt) {
                    tmem_ld_wait();
                    if (c0 + 64 < u_nt) tmem_ld_16(t_addr + c0 + 64, va);
                    drain16(vb, c0 + 32);
                }
            }
            }   // feature tiles of the unit
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (kPair) mbar_arrive_cluster(bar0_leader + 8u * (kRingBars + 2 + b));   // the leader's MMA issuer waits
                else mbar_arrive(acc_empty(b));     // accumulator buffer free
                mbar_arrive(rows_stored(b));   // rows stored (release, CTA scope)
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
            AccCursor acc;
            for (int it = 0;; ++it) {
                const Unit un = pop_unit(it, false);
                if (un.id < 0) break;
                acc.next(un);
                if (!mbar_wait(rows_stored(acc.b), acc.parity, abort_flag, kWaitLimitNs))
                    break;   // the role that stalled has already reported
                // Only now may this accumulator buffer be reused: the epilogue cannot signal "rows
                // stored" for the buffer's next use before this thread has seen the current one
                // (a waiter that falls two phases behind an mbarrier would wait on the wrong phase).
                if (kPair) mbar_arrive_cluster(bar0_leader + 8u * (kRingBars + 2 + acc.b));
                else mbar_arrive(acc_empty(acc.b));
                if (un.layer == 0) {
                    if (P.hold_ready) continue;     // diagnostic: the rows are never announced
                    __threadfence();
                    fence_proxy_async_all();
                    atomicAdd(P.ready + un.ready_idx, 1);
                } else if (un.split + 1 < un.n_split) {
                    __threadfence();
                    atomicAdd(P.part_done + un.tile_idx, 1);
                }
            }
        }
    }

    // ---- teardown --------------------------------------------------------------------
    if (kPair && *abort_flag != 0) {
        // A pair that gives up: the other CTA's copies into its own shared memory are counted on the
        // leader's barriers, which the leader may not have armed for the last of them; allow them the
        // time any copy needs to land before either CTA leaves.
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 50000ull) { }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (kPair) cluster_sync_all();   // neither CTA leaves while the other may still signal its barriers
    if (warp == 1) {
        tc_fence_after_sync();
        if (kPair) tmem_dealloc_pair(tmem_base, kTmemCols); else tmem_dealloc(tmem_base, kTmemCols);
    }
    // The last CTA to finish leaves the counters at zero for the next call.
    if (warp == 2) {
        int last = 0;
        if (lane == 0) {
            __threadfence();
            last = atomicAdd(P.ticket, 1) == static_cast<int>(gridDim.x) - 1;
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            for (int i = lane; i < tt_all; i += 32) P.ready[i] = 0;
            if (P.n_split > 1)
                for (int i = lane; i < (tt_all - tt_hot) * ut.upt[3]; i += 32) P.part_done[i] = 0;
            if (lane == 0) {
                *P.next_unit = 0;
                *P.ticket = 0;
            }
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

// Opt-in to the kernel's dynamic shared memory; a per-device attribute (see per_device_once).
cudaError_t ffn_kernel_attributes() {
    const void* kernels[4] = {
        reinterpret_cast<const void*>(expert_ffn_kernel<MONDE_ACT_RELU, false>),
        reinterpret_cast<const void*>(expert_ffn_kernel<MONDE_ACT_GELU_ERF, false>),
        reinterpret_cast<const void*>(expert_ffn_kernel<MONDE_ACT_RELU, true>),
        reinterpret_cast<const void*>(expert_ffn_kernel<MONDE_ACT_GELU_ERF, true>)};
    for (int i = 0; i < 4; ++i) {
        const cudaError_t e = cudaFuncSetAttribute(kernels[i], cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// The ten tensor maps of a call depend only on addresses and shapes, never on memory contents, and a
// layer is called again and again with the same buffers: the last few sets are kept (per process,
// under a mutex) so that a repeated call skips ten driver calls on its host path.
struct MapKey {
    int dev;
    const void *W1, *W2, *x, *h;
    uint64_t A;
    int E, d_model, d_ff, pair;
    bool operator==(const MapKey& o) const {
        return dev == o.dev && W1 == o.W1 && W2 == o.W2 && x == o.x && h == o.h && A == o.A && E == o.E &&
               d_model == o.d_model && d_ff == o.d_ff && pair == o.pair;
    }
};
constexpr int kMapCacheSlots = 16;
std::mutex g_map_mutex;
MapKey g_map_keys[kMapCacheSlots];
FfnMaps g_map_vals[kMapCacheSlots];
bool g_map_used[kMapCacheSlots] = {};
int g_map_next = 0;

bool ffn_maps(const MapKey& k, FfnMaps* out) {
    std::lock_guard<std::mutex> lock(g_map_mutex);
    for (int i = 0; i < kMapCacheSlots; ++i)
        if (g_map_used[i] && g_map_keys[i] == k) { *out = g_map_vals[i]; return true; }
    FfnMaps M;
    const uint32_t in_box_single[3] = {16, 64, 256}, in_box_pair[3] = {8, 32, 128};
    const uint32_t* in_box = k.pair ? in_box_pair : in_box_single;
    for (int i = 0; i < 2; ++i) {
        if (!make_map(&M.w[0][i], k.W1, static_cast<uint64_t>(k.E) * k.d_ff, k.d_model, kTileRows << i)) return false;
        if (!make_map(&M.w[1][i], k.W2, static_cast<uint64_t>(k.E) * k.d_model, k.d_ff, kTileRows << i)) return false;
    }
    for (int i = 0; i < 3; ++i) {
        if (!make_map(&M.in[0][i], k.x, k.A, k.d_model, in_box[i])) return false;
        if (!make_map(&M.in[1][i], k.h, k.A, k.d_ff, in_box[i])) return false;
    }
    const int slot = g_map_next;
    g_map_next = (g_map_next + 1) % kMapCacheSlots;
    g_map_keys[slot] = k;
    g_map_vals[slot] = M;
    g_map_used[slot] = true;
    *out = M;
    return true;
}

}  // namespace

int launch_ffn_bf16(const monde_problem& p, const void* x_perm, const void* W1, const void* b1,
                    const void* W2, const void* b2, const int32_t* counts, const int32_t* offsets,
                    const uint8_t* cls, void* y_perm, void* ws, cudaStream_t s, const int32_t* fuse_perm,
                    const float* fuse_w, void* fuse_out) {
    if (per_device_once(kSetupFfn, ffn_kernel_attributes) != cudaSuccess) return MONDE_ERR_CUDA;
    const DiagState diag = diag_state();
    char* base = static_cast<char*>(ws);
    const uint64_t A = static_cast<uint64_t>(p.T) * p.top_k;
    FfnParams P;
    P.E = p.E;
    P.d_model = p.d_model;
    P.d_ff = p.d_ff;
    P.act = p.act;
    P.b1 = static_cast<const __nv_bfloat16*>(b1);
    P.b2 = static_cast<const __nv_bfloat16*>(b2);
    P.h = reinterpret_cast<__nv_bfloat16*>(base + WsLayout::kHidden);
    P.y = static_cast<__nv_bfloat16*>(y_perm);
    P.cls = cls;
    P.counts = counts;
    P.offsets = offsets;
    P.status = reinterpret_cast<int32_t*>(base + WsLayout::kStatus);
    P.ticket = reinterpret_cast<int32_t*>(base + WsLayout::kCounters);
    P.next_unit = P.ticket + 1;
    P.cold_tile = cold_token_tile(p);
    // Cold units always pair feature tiles.  Hot units pair them when d_model >= 1536: the K loop of
    // the first layer is then long enough to pay for the exposed epilogue, and the second layer
    // has enough feature tiles left to keep every SM busy with half as many, twice as long units
    // (measured: pairing the hot class takes NLLB-sized layers from 1.53 to 1.39 ms and
    // Switch-Base-sized ones from 175 to 195 us).
    P.pair_mask = 0xC | (p.d_model >= 1536 ? 0x3 : 0);
    // CTA pairs (one 256-row MMA per pair of SMs, each CTA staging its own feature tile and half of
    // the token tile) give the hot class the halved token-tile traffic of two-tile units without
    // filling all of tensor memory, so the epilogue overlaps the next unit's MMAs.  Measured, the
    // two modes are within 3 % of each other on every workload tried (the feed from L2, about
    // 11 TB/s over all SMs, limits both), so single CTAs stay the default and pairs are opt-in
    // (monde_diag_set_ffn_cta_pairs).
    const bool pair = diag.ffn_pair > 0;
    if (pair) P.pair_mask = 0xF;
    const WsLayout L = ws_layout(p);
    P.n_split = L.n_split;
    // Finishing sub-units at the very end of the list give the shortest tail (Switch-Base-sized
    // layer: 152 -> 144 us) but their partial tiles must survive in L2 while the rest of the
    // cold second-layer weights stream through; with gigabytes of weights they do not (NLLB-sized
    // layer: 1.38 -> 1.41 ms), and the expert-by-expert order is used instead.
    P.split_major = 4.0 * p.E * p.d_model * static_cast<double>(p.d_ff) <= 1.0e9;
    P.part_done = reinterpret_cast<int32_t*>(base + L.part_done_off);
    P.partials = reinterpret_cast<float*>(base + L.partials_off);
    P.ready = reinterpret_cast<int32_t*>(base + WsLayout::kTiles);
    P.fuse_perm = fuse_perm;
    P.fuse_w = fuse_w;
    P.fuse_out = static_cast<__nv_bfloat16*>(fuse_out);
    P.diag = diag_record_ptr();
    P.A = static_cast<int>(A);
    P.trace = diag.trace;
    P.trace_slots = diag.trace_slots;
    P.hold_ready = diag.hold_hidden_ready;
    P.wait_ns = diag.wait_limit_ns;
    FfnMaps M;
    MapKey key;
    if (cudaGetDevice(&key.dev) != cudaSuccess) return MONDE_ERR_CUDA;
    key.W1 = W1; key.W2 = W2; key.x = x_perm; key.h = P.h; key.A = A;
    key.E = p.E; key.d_model = p.d_model; key.d_ff = p.d_ff; key.pair = pair;
    if (!ffn_maps(key, &M)) return MONDE_ERR_CUDA;
    cudaError_t err;
    const int sms = current_sm_count();
    const dim3 grid(pair ? sms & ~1 : sms);
    if (pair && p.act == MONDE_ACT_RELU)
        err = launch_pdl_cluster(expert_ffn_kernel<MONDE_ACT_RELU, true>, grid, dim3(kThreads), kSmemBytes, 2, s, M, P);
    else if (pair)
        err = launch_pdl_cluster(expert_ffn_kernel<MONDE_ACT_GELU_ERF, true>, grid, dim3(kThreads), kSmemBytes, 2, s, M, P);
    else if (p.act == MONDE_ACT_RELU)
        err = launch_pdl(expert_ffn_kernel<MONDE_ACT_RELU, false>, grid, dim3(kThreads), kSmemBytes, s, M, P);
    else
        err = launch_pdl(expert_ffn_kernel<MONDE_ACT_GELU_ERF, false>, grid, dim3(kThreads), kSmemBytes, s, M, P);
    if (err != cudaSuccess) return MONDE_ERR_CUDA;
    return launched();
}

}  // namespace monde

