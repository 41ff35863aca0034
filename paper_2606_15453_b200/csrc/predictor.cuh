// Spatio-temporal expert predictor: co-activation counting and CCT construction
// (Algorithm 1), prediction (Algorithm 2 with the score combination of Eq. 1), verification
// and table update (Algorithm 3), history-table overwrite.  Integer only.  The CCT of the
// layer pair being updated is staged in shared memory; rows are handled one warp each with
// lane = candidate slot, membership tests by ballot and replacement targets by find-nth-set.
#pragma once
#include "device_utils.cuh"
#include "router.cuh"

namespace stmoe_dev {

constexpr int kConfInit = 2;   // binary 10
constexpr int kConfMax = 3;    // binary 11
constexpr int kThreshold = 2;  // history bonus of Eq. 1 and the paper's set threshold: binary 10

struct PredState {
    uint32_t *Co;        // [L-1][E][E]
    uint8_t *cct_id;     // [L-1][E][K]
    uint8_t *cct_conf;   // [L-1][E][K]
    int16_t *HT;         // [Bmax][L][K]
    long long *t;        // [0] decode steps completed
    uint32_t *pred_mask; // [Bmax][8] set predicted for the layer that runs next
    uint32_t *pred_valid;// [Bmax]
    unsigned long long *stats;  // [0] steps [1] routed [2] predicted [3] hits [4] near ties
    int threshold;       // an expert is predicted when its score reaches this (Section 4.2: binary 10)
    int live_counts;     // Algorithm 3's new candidate: 0 lowest routed id, 1 largest count in a Co row
                         // that keeps counting at run time
};

struct PredArgs {
    PredState st;
    int L, E, K, P, mode, layer, B;
    const int32_t *cur;   // [B][K] routing of this layer (ascending)
    const int32_t *prev;  // [B][K] routing of layer-1 (unused for layer 0)
    int32_t *pred_ids;    // optional [B][max_pred]
    int32_t *n_pred;      // optional [B]
    int max_pred;
    int32_t *queue;       // optional: [0] n, [1..E] ids, [1+E..2E] scores (priority order)
    // optional, with queue: host memory mapped into the device's address space that the host polls
    // instead of copying: [0] <- host_seq last, [1..1+Bmax*K) this layer's routing, then the queue
    int32_t *host_out;
    int32_t host_seq, host_queue_off;
};

// Which routed expert a replacing slot takes (Algorithm 3 leaves it open).  Every lane of a group
// of `width` lanes calls this; lane k < K of the group carries routed expert k.  avail: the group's
// routed experts the row does not hold; nth (1-based): this lane is the nth replacing slot of its
// row in slot order.  The nth replacing slot takes the nth candidate, exactly as a slot-by-slot
// scan that re-reads the row would: candidates in ascending id or, with by_count (cnt = this
// lane's expert's count in the row), by (count descending, id ascending).  Returns the group lane that carries the
// chosen expert, or 0xffffffff when there are fewer candidates than replacing slots.
__device__ __forceinline__ unsigned replacement_source(unsigned avail, int nth, bool by_count, unsigned cnt, int K,
                                                       int gl, int width)
{
    if (!by_count) return __fns(avail, 0, nth);
    int rank = 0;
    for (int k = 0; k < K; ++k) {
        const unsigned ck = __shfl_sync(kFull, cnt, k, width);
        rank += ((avail >> k) & 1u) && (ck > cnt || (ck == cnt && k < gl));
    }
    unsigned pos = 0xffffffffu;
    for (int k = 0; k < K; ++k) {
        const int rk = __shfl_sync(kFull, rank, k, width);
        if (((avail >> k) & 1u) && rk == nth - 1) pos = (unsigned)k;
    }
    return pos;
}

// Algorithm 3 for one row, executed by one warp: lane c < K owns candidate slot c.  co_row: the
// row of the pair's co-activation counts when counting goes on at run time (this step's K pairs
// of the row are counted here, before the update), else nullptr.
__device__ __forceinline__ void update_row(uint8_t *ids, uint8_t *conf, int K, const int32_t *F,
                                           int lane, uint32_t *co_row = nullptr)
{
    const bool act = lane < K;
    int id = act ? ids[lane] : -1, cf = act ? conf[lane] : 0;
    const int myf = act ? F[lane] : -2;  // lane k also carries routed expert k (ascending)
    unsigned cnt = 0;
    if (co_row && act) cnt = co_row[myf] + 1u, co_row[myf] = cnt;
    bool hit = false, held = false;
    for (int k = 0; k < K; ++k) {
        hit |= (id == __shfl_sync(kFull, myf, k));
        held |= (myf == __shfl_sync(kFull, id, k));
    }
    const bool replace = act && !hit && cf == 0;
    if (act) {
        if (hit)
            cf = min(cf + 1, kConfMax);
        else if (cf > 0)
            cf -= 1;
    }
    const unsigned rep = __ballot_sync(kFull, replace);
    if (rep) {
        // routed experts the row does not hold; the n-th replacing slot (in slot order) takes
        // the n-th of them, exactly as a slot-by-slot scan would.
        const unsigned avail = __ballot_sync(kFull, act && !held);
        const int nth = __popc(rep & ((1u << lane) - 1u)) + 1;
        const unsigned pos = replacement_source(avail, nth, co_row != nullptr, cnt, K, lane, kWarp);
        const int g = __shfl_sync(kFull, myf, pos & 31u);
        if (replace && pos != 0xffffffffu) id = g, cf = kConfInit;
    }
    if (act) ids[lane] = (uint8_t)id, conf[lane] = (uint8_t)cf;
}

// Algorithm 3 for the rows of one sequence's previous-layer experts, several rows at a time: the
// warp is cut into groups of G lanes (G = the power of two >= K) and each group updates one row
// exactly as update_row does.  The rows of one sequence are distinct, so they do not depend on
// one another.  take(k) says whether row prev[k] belongs to this warp.  co: the pair's [E][E]
// counts when counting goes on at run time, else nullptr.
template <typename Take>
__device__ __forceinline__ void update_rows_grouped(uint8_t *gid, uint8_t *gcf, int K, const int32_t *prev,
                                                    const int32_t *F, int lane, Take take, uint32_t *co = nullptr,
                                                    int E = 0)
{
    int G = 1;
    while (G < K) G <<= 1;
    const int per = kWarp / G, sub = lane / G, sl = lane % G;
    const unsigned gmask = G == kWarp ? kFull : ((1u << G) - 1u);
    const unsigned mine = __ballot_sync(kFull, lane < K && take(prev[lane]));
    const int nrows = __popc(mine);
    const int myf = sl < K ? F[sl] : -2;  // group lane k also carries routed expert k (ascending)
    for (int r0 = 0; r0 < nrows; r0 += per) {
        const int r = r0 + sub;
        const bool row_ok = r < nrows;
        const int e = row_ok ? prev[__fns(mine, 0, r + 1)] : 0;
        uint8_t *ids = gid + (size_t)e * K, *conf = gcf + (size_t)e * K;
        const bool act = row_ok && sl < K;
        int id = act ? ids[sl] : -1, cf = act ? conf[sl] : 0;
        unsigned cnt = 0;
        if (co && act) {
            uint32_t *c = co + (size_t)e * E + myf;
            cnt = *c + 1u, *c = cnt;
        }
        bool hit = false, held = false;
        for (int k = 0; k < K; ++k) {
            hit |= (id == __shfl_sync(kFull, myf, k, G));
            held |= (myf == __shfl_sync(kFull, id, k, G));
        }
        const bool replace = act && !hit && cf == 0;
        if (act) {
            if (hit)
                cf = min(cf + 1, kConfMax);
            else if (cf > 0)
                cf -= 1;
        }
        const unsigned rep_all = __ballot_sync(kFull, replace);
        if (rep_all) {  // rare; the whole warp takes the branch
            const unsigned rep = (rep_all >> (sub * G)) & gmask;
            const unsigned avail = (__ballot_sync(kFull, act && !held) >> (sub * G)) & gmask;
            // routed experts the row does not hold; the n-th replacing slot (in slot order) takes
            // the n-th of them
            const int nth = __popc(rep & ((1u << sl) - 1u)) + 1;
            unsigned pos = replacement_source(avail, nth, co != nullptr, cnt, K, sl, G);
            if (!replace) pos = 0u;
            const int g = __shfl_sync(kFull, myf, pos & (unsigned)(G - 1), G);
            if (replace && pos != 0xffffffffu) id = g, cf = kConfInit;
        }
        if (act) ids[sl] = (uint8_t)id, conf[sl] = (uint8_t)cf;
        __syncwarp();
    }
}

__global__ void __launch_bounds__(256) predictor_step_kernel(PredArgs a)
{
    constexpr int NW = 8;
    __shared__ uint8_t s_id[kMaxExperts * kMaxTopK], s_cf[kMaxExperts * kMaxTopK];
    __shared__ int s_score[NW][kMaxExperts];
    __shared__ int s_total[kMaxExperts];
    __shared__ int s_nq;
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
    const int E = a.E, K = a.K, L = a.L, layer = a.layer, B = a.B;
    const long long t = *a.st.t;
    const bool runtime = t >= a.P;
    const bool last_profiling = (!runtime) && t == a.P - 1 && layer == L - 1;

    if (runtime) {
        // V: score the earlier prediction for this layer against the routing
        for (int b = warp; b < B; b += NW) {
            const bool valid = a.st.pred_valid[b] != 0;
            int np = 0, nh = 0;
            if (valid) {
                if (lane < 8) np = __popc(a.st.pred_mask[b * 8 + lane]);
                if (lane < K) {
                    const int f = a.cur[b * K + lane];
                    nh = (a.st.pred_mask[b * 8 + (f >> 5)] >> (f & 31)) & 1u;
                }
            }
            np = __reduce_add_sync(kFull, np);
            nh = __reduce_add_sync(kFull, nh);
            if (lane == 0) {
                atomicAdd(&a.st.stats[0], 1ull);
                atomicAdd(&a.st.stats[1], (unsigned long long)K);
                atomicAdd(&a.st.stats[2], (unsigned long long)np);
                atomicAdd(&a.st.stats[3], (unsigned long long)nh);
            }
        }
        // Algorithm 3 on pair (layer-1, layer): sequences in index order, the K rows of one
        // sequence (distinct experts) in parallel, one warp per row.
        if (layer > 0) {
            uint8_t *gid = a.st.cct_id + (size_t)(layer - 1) * E * K;
            uint8_t *gcf = a.st.cct_conf + (size_t)(layer - 1) * E * K;
            for (int i = threadIdx.x; i < E * K; i += blockDim.x) s_id[i] = gid[i], s_cf[i] = gcf[i];
            __syncthreads();
            uint32_t *co = a.st.live_counts ? a.st.Co + (size_t)(layer - 1) * E * E : nullptr;
            for (int b = 0; b < B; ++b) {
                for (int k = warp; k < K; k += NW) {
                    const int e = a.prev[b * K + k];
                    update_row(s_id + e * K, s_cf + e * K, K, a.cur + b * K, lane, co ? co + (size_t)e * E : nullptr);
                }
                __syncthreads();
            }
            for (int i = threadIdx.x; i < E * K; i += blockDim.x) gid[i] = s_id[i], gcf[i] = s_cf[i];
        }
    } else if (layer > 0) {
        // Algorithm 1, counting: Co[e][f] += 1 for e routed at layer-1, f at layer
        uint32_t *Co = a.st.Co + (size_t)(layer - 1) * E * E;
        for (int i = threadIdx.x; i < B * K * K; i += blockDim.x) {
            const int b = i / (K * K), r = i % (K * K);
            atomicAdd(&Co[(size_t)a.prev[b * K + r / K] * E + a.cur[b * K + r % K]], 1u);
        }
    }

    // P: Algorithm 2 for layer+1 (after the last layer: layer 0 of the next decode step,
    // history table only).  The build of Algorithm 1 runs right after the last profiling
    // step, whose prediction is history-only and so does not depend on it.
    const bool predict_now = runtime || last_profiling;
    const int next = (layer + 1) % L;
    const bool spatial = predict_now && (a.mode & 2) && layer < L - 1;
    const bool temporal = predict_now && (a.mode & 1);
    for (int i = threadIdx.x; i < kMaxExperts; i += blockDim.x) s_total[i] = 0;
    __syncthreads();
    for (int b = warp; b < B; b += NW) {
        int *sc = s_score[warp];
        for (int f = lane; f < kMaxExperts; f += kWarp) sc[f] = 0;
        __syncwarp();
        if (spatial) {
            const uint8_t *cid = a.st.cct_id + (size_t)layer * E * K;
            const uint8_t *ccf = a.st.cct_conf + (size_t)layer * E * K;
            for (int k = 0; k < K; ++k) {
                const int e = a.cur[b * K + k];
                if (lane < K) sc[cid[e * K + lane]] += ccf[e * K + lane];  // ids of a row differ
                __syncwarp();
            }
        }
        if (temporal) {
            if (lane < K) {
                const int hte = a.st.HT[((size_t)b * L + next) * K + lane];
                if (hte >= 0) sc[hte] += kThreshold;  // Eq. 1: CCT(e) + HT(e), HT(e) = binary 10
            }
            __syncwarp();
        }
        int count = 0;
        for (int w = 0; w < kMaxExperts / kWarp; ++w) {
            const int f = w * kWarp + lane;
            const bool in = f < E && sc[f] >= a.st.threshold;
            const unsigned msk = __ballot_sync(kFull, in);
            if (lane == 0) a.st.pred_mask[b * 8 + w] = msk;
            if (in) {
                atomicAdd(&s_total[f], sc[f]);
                const int pos = count + __popc(msk & ((1u << lane) - 1u));
                if (a.pred_ids && pos < a.max_pred) a.pred_ids[(size_t)b * a.max_pred + pos] = f;
            }
            count += __popc(msk);
        }
        if (a.pred_ids)
            for (int i = count + lane; i < a.max_pred; i += kWarp) a.pred_ids[(size_t)b * a.max_pred + i] = -1;
        if (lane == 0) {
            a.st.pred_valid[b] = predict_now ? 1u : 0u;
            if (a.n_pred) a.n_pred[b] = count;
        }
    }
    __syncthreads();

    // prefetch queue: union of the batch, score summed over sequences, (score desc, id asc)
    if (a.queue) {
        if (threadIdx.x == 0) s_nq = 0;
        __syncthreads();
        const int f = threadIdx.x;
        const int mine = f < E ? s_total[f] : 0;
        if (mine > 0) {
            int rank = 0;
            for (int g = 0; g < E; ++g) {
                const int o = s_total[g];
                rank += (o > mine) || (o == mine && g < f);
            }
            a.queue[1 + rank] = f;
            a.queue[1 + E + rank] = mine;
            if (a.host_out) {
                a.host_out[a.host_queue_off + 1 + rank] = f;
                a.host_out[a.host_queue_off + 1 + E + rank] = mine;
            }
            atomicAdd(&s_nq, 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            a.queue[0] = s_nq;
            if (a.host_out) a.host_out[a.host_queue_off] = s_nq;
        }
    }
    if (a.queue && a.host_out) {
        // hand the routing and the queue to the host without a copy: every writer fences its stores
        // to system scope, the stamp goes last
        for (int i = threadIdx.x; i < B * K; i += blockDim.x) a.host_out[1 + i] = a.cur[i];
        __threadfence_system();
        __syncthreads();
        if (threadIdx.x == 0) *reinterpret_cast<volatile int32_t *>(a.host_out) = a.host_seq;
    }

    // HT[layer] <- routing; advance the step counter after the last layer
    for (int i = threadIdx.x; i < B * K; i += blockDim.x) {
        const int b = i / K, k = i % K;
        a.st.HT[((size_t)b * L + layer) * K + k] = (int16_t)a.cur[b * K + k];
    }
    if (threadIdx.x == 0 && layer == L - 1) *a.st.t = t + 1;
}

// Algorithm 1, construction: per row the K largest counts (ties: lower id), rank order, all
// confidences binary 10.  One warp per (pair, row).
__global__ void __launch_bounds__(256) cct_build_kernel(PredState st, int L, int E, int K)
{
    constexpr int VPL = kMaxExperts / kWarp;
    const int lane = threadIdx.x % kWarp;
    const int row = blockIdx.x * (blockDim.x / kWarp) + threadIdx.x / kWarp;
    if (row >= (L - 1) * E) return;
    const uint32_t *co = st.Co + (size_t)row * E;
    uint32_t cnt[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) cnt[v] = (v * kWarp + lane < E) ? co[v * kWarp + lane] : 0u;
    uint32_t taken = 0;
    for (int r = 0; r < K; ++r) {
        unsigned long long best = 0;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int f = v * kWarp + lane;
            if (f < E && !((taken >> v) & 1u)) {
                const unsigned long long key =
                    ((unsigned long long)cnt[v] << 32) | (uint32_t)(0xffffffffu - f) | (1ull << 63);
                best = key > best ? key : best;
            }
        }
        best = warp_max_u64(best);
        const int f = (int)(0xffffffffu - (uint32_t)best);
        if (f % kWarp == lane) taken |= 1u << (f / kWarp);
        if (lane == 0) {
            st.cct_id[(size_t)row * K + r] = (uint8_t)f;
            st.cct_conf[(size_t)row * K + r] = (uint8_t)kConfInit;
        }
    }
}

}  // namespace stmoe_dev
