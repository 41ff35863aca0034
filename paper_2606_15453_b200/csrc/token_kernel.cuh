// One decode step of a resident stack as a single persistent kernel.
//
// One 512-thread CTA per SM, launched cooperatively (all CTAs resident), walks the layers:
//   R   split-K router GEMV tasks dealt over all warps of the grid        -> grid barrier
//   T   every CTA sums the partial logits and runs softmax / top-K / grouping for the whole
//       batch itself (redundantly: cheaper than one CTA doing it while 147 wait, and the work
//       list then lives in shared memory); CTA 0 also writes the step's outputs
//   GU  gate/up projection over this CTA's share of the rows              -> grid barrier
//   D   down projection + fused weighted sum / residual                   -> grid barrier
// so a layer costs three grid barriers (about a microsecond each) instead of three kernel
// launches with their launch latency, ramp-up and drain.  The predictor (Algorithms 1-3) runs
// on one warp of the last CTA beside the GU phase of the same layer.
//
// Coherence: data that other SMs produce inside this launch is either read past L1
// (ld.global.cg: router partials, down-projection partials) or lives at an address that is
// unique to the layer (hidden state, activations), so a line can never be in an SM's L1 before
// its producer has written it and a grid barrier has been passed.
// Grid barrier: one monotonically increasing counter; every wait is bounded and a timeout
// raises an error word that makes all later barriers fall through, so the kernel always ends.
#pragma once
#include "device_utils.cuh"
#include "ffn.cuh"
#include "predictor.cuh"
#include "router.cuh"

namespace stmoe_dev {

constexpr int kBarrierSpinLimit = 1 << 22;


struct TokenArgs {
    int L, B, E, K, n_shared, H, I, S, mt, renorm;
    float eps, residual_scale;
    const float *h_in;              // [B][H]
    float *h_out;                   // [B][H]
    float *hbuf;                    // [L][B][H]   input of layers 1..L-1 lives in hbuf[l]
    const uint8_t *router;          // [L][E][H]
    const uint8_t *const *blob;     // [L][E+n_shared]
    float *rpart, *sspart;          // [L][C][B][E], [L][C][B]
    float *act, *part;              // [L][B*KS][I], [L][B*KS][S][H]
    unsigned *tile_done;            // [L][ceil(H/32)]
    int32_t *ids_all;               // [L][Bmax][K] library copy of the routing
    int Bmax;
    int32_t *ids_out;               // optional [L][B][K]
    float *w_out;                   // optional [L][B][K]
    uint32_t *flags_out;            // optional [L][B]
    int32_t *pred_ids;              // optional [L][B][max_pred]
    int32_t *n_pred;                // optional [L][B]
    int max_pred;
    PredState pst;
    int P, mode;
    unsigned *barrier;              // [1] zero at launch
    unsigned *err;                  // [1]
    // single-sequence schedule: resident images by address arithmetic, on-chip staging budgets
    const uint8_t *store;           // routed images [L][E], then shared images [L][n_shared]
    size_t img_bytes;
    long long stage_down_bytes;     // per entry and CTA: down-projection bytes staged ahead of the GU->D barrier
    long long stage_pred_bytes;     // per layer, whole GPU: gate/up bytes of predicted experts staged ahead (0: off)
    int stage_shared;               // stage the next layer's shared experts ahead of its router
};

// Algorithms 1-3 for one layer step on `nw` warps of one CTA (this is warp `wi` of them; all nw
// call together), same arithmetic and order as predictor_step_kernel.  The tables live in global
// memory, which only these warps touch during the launch.  Work is split so that no two warps
// ever need the same data: table rows (Algorithm 3) by row index, with each warp walking the
// batch in order, so a row sees its updates in the sequential order; predictions (Algorithm 2,
// Eq. 1) and their scoring by sequence.  Scores are kept in registers (lane f % 32 holds expert
// f), so the warps need no shared memory.  cur/prev: routing of this and the
// previous layer [B][K].
__device__ __forceinline__ void prefetch_l1(const void *p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

__device__ __forceinline__ void predictor_step_group(const TokenArgs &a, int layer, const int *cur, const int *prev,
                                                     int wi, int nw, int lane, int bar_id = 3)
{
    const int E = a.E, K = a.K, L = a.L, B = a.B;
    const PredState &st = a.pst;
    const long long t = *st.t;
    const bool runtime = t >= a.P;
    const bool last_profiling = (!runtime) && t == a.P - 1 && layer == L - 1;
    if (runtime && __isGlobal(st.cct_id)) {  // (a caller may keep the tables in shared memory: nothing to pull)
        // Every table row this step touches, pulled into L1 in one trip: the rows are then read
        // one after the other (Algorithm 3 is sequential per row), each of which would otherwise
        // be a trip to L2 of its own.  The tables are private to these warps' SM during the launch.
        for (int i = wi * kWarp + lane; i < B * K; i += nw * kWarp) {
            if (layer > 0) {
                prefetch_l1(st.cct_id + ((size_t)(layer - 1) * E + prev[i]) * K);
                prefetch_l1(st.cct_conf + ((size_t)(layer - 1) * E + prev[i]) * K);
            }
            if (layer < L - 1) {
                prefetch_l1(st.cct_id + ((size_t)layer * E + cur[i]) * K);
                prefetch_l1(st.cct_conf + ((size_t)layer * E + cur[i]) * K);
            }
        }
    }
    if (runtime) {
        for (int b = wi; b < B; b += nw) {
            const bool valid = st.pred_valid[b] != 0;
            int np = 0, nh = 0;
            if (valid) {
                if (lane < 8) np = __popc(st.pred_mask[b * 8 + lane]);
                if (lane < K) {
                    const int f = cur[b * K + lane];
                    nh = (st.pred_mask[b * 8 + (f >> 5)] >> (f & 31)) & 1u;
                }
            }
            np = __reduce_add_sync(kFull, np);
            nh = __reduce_add_sync(kFull, nh);
            if (lane == 0) {
                atomicAdd(&st.stats[0], 1ull);
                atomicAdd(&st.stats[1], (unsigned long long)K);
                atomicAdd(&st.stats[2], (unsigned long long)np);
                atomicAdd(&st.stats[3], (unsigned long long)nh);
            }
        }
        if (layer > 0) {
            uint8_t *gid = st.cct_id + (size_t)(layer - 1) * E * K;
            uint8_t *gcf = st.cct_conf + (size_t)(layer - 1) * E * K;
            uint32_t *co = st.live_counts ? st.Co + (size_t)(layer - 1) * E * E : nullptr;
            for (int b = 0; b < B; ++b)
                update_rows_grouped(gid, gcf, K, prev + b * K, cur + b * K, lane, [&](int e) { return e % nw == wi; },
                                    co, E);
        }
    } else if (layer > 0) {
        uint32_t *Co = st.Co + (size_t)(layer - 1) * E * E;
        for (int i = wi * kWarp + lane; i < B * K * K; i += nw * kWarp) {
            const int b = i / (K * K), r = i % (K * K);
            atomicAdd(&Co[(size_t)prev[b * K + r / K] * E + cur[b * K + r % K]], 1u);
        }
    }
    __syncwarp();

    const bool predict_now = runtime || last_profiling;
    const int next = (layer + 1) % L;
    const bool spatial = predict_now && (a.mode & 2) && layer < L - 1;
    const bool temporal = predict_now && (a.mode & 1);
    int32_t *pred_ids = a.pred_ids ? a.pred_ids + (size_t)layer * B * a.max_pred : nullptr;
    int32_t *n_pred = a.n_pred ? a.n_pred + (size_t)layer * B : nullptr;
    const uint8_t *cid = st.cct_id + (size_t)layer * E * K;
    const uint8_t *ccf = st.cct_conf + (size_t)layer * E * K;
    for (int b = wi; b < B; b += nw) {
        // Scores of the eight experts lane, lane+32, ... packed one byte each into two registers
        // (a score is at most 3K + 2 <= 98: K rows of confidence <= 3, plus the history bonus).
        unsigned lo = 0u, hi = 0u;
        // lane j adds `add` to the score of expert `id` (add = 0: nothing), for all lanes in turn
        auto scatter = [&](int id, int add, int n_lanes) {
            for (int j = 0; j < n_lanes; ++j) {
                const int idj = __shfl_sync(kFull, id, j), addj = __shfl_sync(kFull, add, j);
                const int slot = idj >> 5;
                const unsigned inc = (unsigned)addj << ((slot & 3) * 8);
                if (lane == (idj & 31)) {
                    if (slot < 4)
                        lo += inc;
                    else
                        hi += inc;
                }
            }
        };
        if (spatial) {
            // the K candidates of each of the K routed experts' rows, 32 (row, slot) pairs per trip
            for (int i0 = 0; i0 < K * K; i0 += kWarp) {
                const int i = i0 + lane;
                int id = 0, add = 0;
                if (i < K * K) {
                    const int e = cur[b * K + i / K];
                    id = cid[e * K + i % K], add = ccf[e * K + i % K];
                }
                scatter(id, add, min(kWarp, K * K - i0));
            }
        }
        if (temporal) {
            int id = 0, add = 0;
            if (lane < K) {
                const int hte = st.HT[((size_t)b * L + next) * K + lane];
                if (hte >= 0) id = hte, add = kThreshold;
            }
            scatter(id, add, K);
        }
        int count = 0;
#pragma unroll
        for (int w = 0; w < kMaxExperts / kWarp; ++w) {
            const int f = w * kWarp + lane;
            const int score = (int)(((w < 4 ? lo : hi) >> ((w & 3) * 8)) & 0xffu);
            const bool in = f < E && score >= st.threshold;
            const unsigned msk = __ballot_sync(kFull, in);
            if (lane == 0) st.pred_mask[b * 8 + w] = msk;
            if (in) {
                const int pos = count + __popc(msk & ((1u << lane) - 1u));
                if (pred_ids && pos < a.max_pred) pred_ids[(size_t)b * a.max_pred + pos] = f;
            }
            count += __popc(msk);
        }
        if (pred_ids)
            for (int i = count + lane; i < a.max_pred; i += kWarp) pred_ids[(size_t)b * a.max_pred + i] = -1;
        if (lane == 0) {
            st.pred_valid[b] = predict_now ? 1u : 0u;
            if (n_pred) n_pred[b] = count;
        }
        __syncwarp();
    }
    for (int i = wi * kWarp + lane; i < B * K; i += nw * kWarp) {
        const int b = i / K, k = i % K;
        st.HT[((size_t)b * L + layer) * K + k] = (int16_t)cur[b * K + k];
    }
    // every warp has read the step counter before one of them advances it
    if (nw > 1) asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(nw * kWarp) : "memory");
    if (wi == 0 && lane == 0 && layer == L - 1) *st.t = t + 1;
}

// Bounded grid barrier on a monotonically increasing counter.
__device__ __forceinline__ void grid_barrier(unsigned *counter, unsigned *err, unsigned &target, volatile int *s_dead,
                                             int spin_limit = kBarrierSpinLimit)
{
    target += gridDim.x;
    __syncthreads();
    if (threadIdx.x == 0 && !*s_dead) {
        // Release at GPU scope: the CTA barrier above orders every thread's writes before this
        // thread's arrival (cumulativity), so no separate fence is needed; the acquiring load below
        // and the CTA barrier after it do the same on the way out.
        asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(counter), "r"(1u) : "memory");
        // poll with relaxed loads (the error word only now and then), acquire once on the way out
        int spins = 0;
        for (;;) {
            unsigned seen;
            asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if (seen >= target) break;
            if (++spins > spin_limit || ((spins & 255) == 0 && *((volatile unsigned *)err))) {
                *err = 1u;
                *s_dead = 1;
                break;
            }
        }
        asm volatile("{.reg .u32 t;\n\tld.acquire.gpu.global.u32 t, [%0];}" ::"l"(counter) : "memory");
    }
    __syncthreads();
}

// Next layer's routing-independent and predicted weights, asked into L2 by a warp that has run
// out of rows in the current layer (or, for layer 0, at the start of the launch): this CTA's
// slices of the shared experts' three matrices, then of the first rows of the gate and up
// matrices of the experts in the prefetch set of Algorithm 2 for that layer (lowest ids first
// when the budget does not cover them all).  The set was written by the predictor warp at least
// one grid barrier ago and is not overwritten before the next layer's top-K, which needs the
// barrier this warp has yet to arrive at.
template <int DT>
__device__ __forceinline__ void stage_layer_ahead(const TokenArgs &a, int layer, const FfnArgs &fa,
                                                  const SliceTickets &tg, const SliceTickets &td, int w, int nw,
                                                  int lane)
{
    constexpr int BYTES = Fmt<DT>::kBytes;
    const uint8_t *routed0 = a.store + (size_t)layer * a.E * a.img_bytes;
    const uint8_t *shared0 = a.store + ((size_t)a.L * a.E + (size_t)layer * a.n_shared) * a.img_bytes;
    if (a.stage_shared) {
        SingleCtx cx{routed0, shared0, a.img_bytes, nullptr, nullptr, 0};  // K = 0: entry g is shared expert g
        for (int i = 0; i < a.n_shared; ++i) stage_gate_up_slice<DT>(fa, cx.image(i), tg, tg.len, w, nw, lane);
        stage_down_slices<DT>(fa, cx, td, 0, a.n_shared, a.stage_down_bytes, w, nw, lane);
    }
    if (a.stage_pred_bytes > 0 && __ldcg(a.pst.pred_valid) != 0u) {
        unsigned msk = lane < kMaxExperts / kWarp ? __ldcg(a.pst.pred_mask + lane) : 0u;
        const int n_pred = __reduce_add_sync(kFull, __popc(msk));
        if (n_pred > 0) {
            const long long per_row = 2ll * a.H * BYTES * gridDim.x;  // one gate + one up row in every CTA
            const int rows_all = (int)(a.stage_pred_bytes / per_row);  // rows the budget buys per CTA
            const int n_take = min(n_pred, max(rows_all, 1));
            const int rows = max(rows_all / n_take, 1);
            int taken = 0;
            for (int wd = 0; wd < kMaxExperts / kWarp && taken < n_take; ++wd) {
                unsigned m = __shfl_sync(kFull, msk, wd);
                while (m && taken < n_take) {
                    const int f = wd * kWarp + __ffs(m) - 1;
                    m &= m - 1;
                    stage_gate_up_slice<DT>(fa, routed0 + (size_t)f * a.img_bytes, tg, rows, w, nw, lane);
                    ++taken;
                }
            }
        }
    }
}

// One decode step for a single sequence (see "single-sequence schedule" in ffn.cuh).
template <int DT, int RDT>
__device__ __forceinline__ void decode_token_single(const TokenArgs &a, int *dyn, int *s_scan, float *s_inv, int *s_next,
                                                    int *s_dead)
{
    constexpr int NW = kFfnThreads / kWarp;
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
    const int L = a.L, E = a.E, K = a.K, H = a.H, I = a.I, S = a.S;
    const int KS = K + a.n_shared;
    const int C = router_chunks<RDT>(H, 1), tiles = (H + kTileRows - 1) / kTileRows;
    int *s_ids = dyn + 4 + 5 * KS;
    int *s_prev = s_ids + K;
    float *s_w = reinterpret_cast<float *>(s_prev + K);
    unsigned target = 0;
    const bool lead = blockIdx.x == 0;
    const bool pred_cta = blockIdx.x == gridDim.x - 1;
    SliceTickets tg, td;
    tg.init(I, KS, TileShape<DT>::RG1);
    td.init(S * H, KS, TileShape<DT>::RD1);
    FfnArgs fa;
    fa.inv_rms = s_inv, fa.H = H, fa.I = I, fa.E = E, fa.S = S, fa.w = s_w;
    fa.B = 1, fa.K = K, fa.n_shared = a.n_shared, fa.residual_scale = a.residual_scale;
    stage_layer_ahead<DT>(a, 0, fa, tg, td, warp, NW, lane);

    for (int l = 0; l < L; ++l) {
        const float *h = l == 0 ? a.h_in : a.hbuf + (size_t)l * H;
        float *h_next = l == L - 1 ? a.h_out : a.hbuf + (size_t)(l + 1) * H;
        if (threadIdx.x == 0) s_next[0] = 0, s_next[1] = 0;  // row tickets of the two phases (read after barriers)

        // ---- R: split-K router GEMV -------------------------------------------------------
        RouterArgs ra;
        ra.h = h, ra.W = a.router + (size_t)l * E * H * Fmt<RDT>::kBytes, ra.H = H, ra.eps = a.eps;
        ra.part = a.rpart + (size_t)l * C * E, ra.ss_part = a.sspart + (size_t)l * C;
        ra.arrivals = nullptr, ra.inv_rms = s_inv, ra.logits_out = nullptr;
        TopkArgs &tk = ra.tk;
        tk.logits = nullptr, tk.B = 1, tk.E = E, tk.K = K, tk.n_shared = a.n_shared, tk.mt = 1, tk.renorm = a.renorm;
        tk.ids = s_ids, tk.w = s_w;
        tk.ids_out = (lead && a.ids_out) ? a.ids_out + (size_t)l * K : nullptr;
        tk.w_out = (lead && a.w_out) ? a.w_out + (size_t)l * K : nullptr;
        tk.flags_out = (lead && a.flags_out) ? a.flags_out + l : nullptr;
        tk.near_tie_counter = lead ? a.pst.stats + 4 : nullptr;
        tk.wl.n_groups = nullptr;  // no work list: the entries are the K routed ids, then the shared experts
        router_tasks<RDT, false>(ra, warp * gridDim.x + blockIdx.x, NW * gridDim.x, lane);  // over the SMs first
        grid_barrier(a.barrier, a.err, target, s_dead);

        // ---- T: softmax / top-K, redundantly per CTA --------------------------------------
        router_finalize<RDT>(ra, s_ids, s_scan, NW);
        __syncthreads();
        if (lead && threadIdx.x < K) a.ids_all[(size_t)l * a.Bmax * K + threadIdx.x] = s_ids[threadIdx.x];

        // ---- GU (+ the predictor on one warp of the last CTA) -----------------------------
        SingleCtx cx;
        cx.routed0 = a.store + (size_t)l * E * a.img_bytes;
        cx.shared0 = a.store + ((size_t)L * E + (size_t)l * a.n_shared) * a.img_bytes;
        cx.img_bytes = a.img_bytes, cx.s_ids = s_ids, cx.s_inv = s_inv, cx.K = K;
        fa.h = h, fa.act = a.act + (size_t)l * KS * I, fa.part = a.part + (size_t)l * KS * S * H;
        fa.h_out = h_next, fa.tile_done = a.tile_done + (size_t)l * tiles;
        gate_up_single<DT>(
            fa, cx, tg, s_next,
            [&]() {
                if (pred_cta && warp == NW - 1) predictor_step_group(a, l, s_ids, s_prev, 0, 1, lane);
            },
            [&]() { stage_down_slices<DT>(fa, cx, td, 0, K, a.stage_down_bytes, warp, NW, lane); });
        grid_barrier(a.barrier, a.err, target, s_dead);

        // ---- D ---------------------------------------------------------------------------
        down_single<DT>(fa, cx, td, s_next + 1, KS, [&]() {
            if (l + 1 < L) stage_layer_ahead<DT>(a, l + 1, fa, tg, td, warp, NW, lane);
        });
        if (threadIdx.x < K) s_prev[threadIdx.x] = s_ids[threadIdx.x];
        grid_barrier(a.barrier, a.err, target, s_dead);
    }
}

template <int DT, int RDT, int MTMAX>
__global__ void __launch_bounds__(kFfnThreads, 1) decode_token_kernel(TokenArgs a)
{
    constexpr int NW = kFfnThreads / kWarp;
    extern __shared__ __align__(16) int dyn[];  // work list | ids | prev ids | gate weights
    __shared__ int s_scan[2 * (kMaxExperts + 1)];
    __shared__ float s_inv[kMaxBatch];
    __shared__ int s_next[3], s_dead;
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
    const int L = a.L, B = a.B, E = a.E, K = a.K, H = a.H, I = a.I, S = a.S;
    const int KS = K + a.n_shared, pairs = B * KS;
    const int C = router_chunks<RDT>(H, B), tiles = (H + kTileRows - 1) / kTileRows;

    WorkList wl;
    wl.n_groups = dyn, wl.g_expert = dyn + 4, wl.g_start = dyn + 4 + pairs, wl.g_count = dyn + 4 + 2 * pairs;
    wl.pair_token = dyn + 4 + 3 * pairs, wl.pair_slot = dyn + 4 + 4 * pairs;
    int *s_ids = dyn + 4 + 5 * pairs;
    int *s_prev = s_ids + B * K;
    float *s_w = reinterpret_cast<float *>(s_prev + B * K);
    if (threadIdx.x == 0) s_dead = 0;
    unsigned target = 0;
    const bool lead = blockIdx.x == 0;
    const bool pred_cta = blockIdx.x == gridDim.x - 1;

    if constexpr (MTMAX == 1) {
        decode_token_single<DT, RDT>(a, dyn, s_scan, s_inv, s_next, &s_dead);
    } else
    for (int l = 0; l < L; ++l) {
        const float *h = l == 0 ? a.h_in : a.hbuf + (size_t)l * B * H;
        float *h_next = l == L - 1 ? a.h_out : a.hbuf + (size_t)(l + 1) * B * H;

        // ---- R: split-K router GEMV -------------------------------------------------------
        RouterArgs ra;
        ra.h = h, ra.W = a.router + (size_t)l * E * H * Fmt<RDT>::kBytes, ra.H = H, ra.eps = a.eps;
        ra.part = a.rpart + (size_t)l * C * B * E, ra.ss_part = a.sspart + (size_t)l * C * B;
        ra.arrivals = nullptr, ra.inv_rms = s_inv, ra.logits_out = nullptr;
        TopkArgs &tk = ra.tk;
        tk.logits = nullptr, tk.B = B, tk.E = E, tk.K = K, tk.n_shared = a.n_shared, tk.mt = a.mt, tk.renorm = a.renorm;
        tk.ids = s_ids, tk.w = s_w;
        tk.ids_out = (lead && a.ids_out) ? a.ids_out + (size_t)l * B * K : nullptr;
        tk.w_out = (lead && a.w_out) ? a.w_out + (size_t)l * B * K : nullptr;
        tk.flags_out = (lead && a.flags_out) ? a.flags_out + (size_t)l * B : nullptr;
        tk.near_tie_counter = lead ? a.pst.stats + 4 : nullptr;
        tk.wl = wl;
        router_tasks<RDT, false>(ra, warp * gridDim.x + blockIdx.x, NW * gridDim.x, lane);  // over the SMs first
        grid_barrier(a.barrier, a.err, target, &s_dead);

        // ---- T: softmax / top-K / grouping, redundantly per CTA ---------------------------
        router_finalize<RDT>(ra, s_ids, s_scan, NW);
        __syncthreads();
        if (lead)
            for (int i = threadIdx.x; i < B * K; i += blockDim.x)
                a.ids_all[(size_t)l * a.Bmax * K + i] = s_ids[i];

        // ---- GU (+ the predictor on one warp of the last CTA) -----------------------------
        FfnArgs fa;
        fa.h = h, fa.inv_rms = s_inv, fa.wl = wl, fa.blob = a.blob + (size_t)l * (E + a.n_shared);
        fa.act = a.act + (size_t)l * pairs * I, fa.part = a.part + (size_t)l * pairs * S * H;
        fa.H = H, fa.I = I, fa.E = E, fa.S = S;
        fa.w = s_w, fa.h_out = h_next, fa.tile_done = a.tile_done + (size_t)l * tiles;
        fa.B = B, fa.K = K, fa.n_shared = a.n_shared, fa.residual_scale = a.residual_scale;
        gate_up_phase<DT, MTMAX>(fa, s_next, [&]() {
            if (pred_cta && warp == NW - 1) predictor_step_group(a, l, s_ids, s_prev, 0, 1, lane);
        });
        grid_barrier(a.barrier, a.err, target, &s_dead);

        // ---- D ---------------------------------------------------------------------------
        down_phase<DT, MTMAX, false>(fa, s_next);
        for (int i = threadIdx.x; i < B * K; i += blockDim.x) s_prev[i] = s_ids[i];
        grid_barrier(a.barrier, a.err, target, &s_dead);
    }
}

}  // namespace stmoe_dev
