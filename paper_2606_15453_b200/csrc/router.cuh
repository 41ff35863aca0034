// Gating network (Section 2): RMSNorm scale, router GEMV, softmax, top-K, and the grouping of
// a batch's routed (token, expert) pairs into per-expert work-list entries.
#pragma once
#include "device_utils.cuh"

namespace stmoe_dev {

constexpr int kRouterWarps = 8;
constexpr int kRouterTokTile = 8;
constexpr int kMaxBatch = 64;
constexpr int kMaxExperts = 256;
constexpr int kMaxTopK = 32;

// logits[b][j] = inv_rms[b] * sum_i W[j][i] h[b][i];  inv_rms[b] = 1/sqrt(mean(h_b^2)+eps).
// One warp per expert row; every CTA recomputes the B scale factors (h is tiny and L2-hot).
template <int DT>
__global__ void __launch_bounds__(kRouterWarps * kWarp)
router_logits_kernel(const float *__restrict__ h, const uint8_t *__restrict__ W, int B, int E, int H,
                     float eps, float *__restrict__ inv_rms, float *__restrict__ logits)
{
    constexpr int EPL = Fmt<DT>::kEpl;
    __shared__ float s_inv[kMaxBatch];
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;

    for (int b = warp; b < B; b += kRouterWarps) {
        float ss = 0.f;
        for (int i = lane * 4; i < H; i += kWarp * 4) {
            const float4 v = ld_f4(h + (size_t)b * H + i);
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        ss = warp_sum(ss);
        if (lane == 0) {
            const float inv = 1.0f / sqrtf(ss / (float)H + eps);
            s_inv[b] = inv;
            if (blockIdx.x == 0) inv_rms[b] = inv;
        }
    }
    __syncthreads();

    const int j = blockIdx.x * kRouterWarps + warp;
    if (j >= E) return;
    const uint8_t *row = W + (size_t)j * H * Fmt<DT>::kBytes;
    for (int b0 = 0; b0 < B; b0 += kRouterTokTile) {
        float acc[kRouterTokTile];
#pragma unroll
        for (int t = 0; t < kRouterTokTile; ++t) acc[t] = 0.f;
        for (int k = lane * EPL; k < H; k += kWarp * EPL) {
            float wf[EPL];
            Fmt<DT>::unpack(ld_stream16(row + (size_t)k * Fmt<DT>::kBytes), wf);
#pragma unroll
            for (int t = 0; t < kRouterTokTile; ++t) {
                if (b0 + t < B) {
                    const float *hp = h + (size_t)(b0 + t) * H + k;
#pragma unroll
                    for (int e = 0; e < EPL; e += 4) {
                        const float4 v = ld_f4(hp + e);
                        acc[t] = fmaf(wf[e], v.x, acc[t]);
                        acc[t] = fmaf(wf[e + 1], v.y, acc[t]);
                        acc[t] = fmaf(wf[e + 2], v.z, acc[t]);
                        acc[t] = fmaf(wf[e + 3], v.w, acc[t]);
                    }
                }
            }
        }
#pragma unroll
        for (int t = 0; t < kRouterTokTile; ++t) {
            const float s = warp_sum(acc[t]);
            if (lane == 0 && b0 + t < B) logits[(size_t)(b0 + t) * E + j] = s * s_inv[b0 + t];
        }
    }
}

// Work list of one layer step: entries of at most `mt` tokens that share one expert.
struct WorkList {
    int *n_groups;    // [1]
    int *g_expert;    // [max_groups] routed: expert id; shared: E + index
    int *g_start;     // [max_groups] first pair of the entry
    int *g_count;     // [max_groups] pairs in the entry (<= mt)
    int *pair_token;  // [B*(K+n_shared)] sequence index
    int *pair_slot;   // [B*(K+n_shared)] row of act/partial buffers: b*(K+n_shared)+k
};

struct TopkArgs {
    const float *logits;  // [B][E]
    int B, E, K, n_shared, mt, renorm;
    int32_t *ids;     // [B][K] ascending (library copy)
    float *w;         // [B][K]
    int32_t *ids_out; // optional caller copies
    float *w_out;
    uint32_t *flags_out;
    unsigned long long *near_tie_counter;  // optional
    WorkList wl;      // wl.n_groups == nullptr: no grouping
};

constexpr int kVplMax = kMaxExperts / kWarp;  // logits held per lane at the maximum expert count

// softmax + top-K for one sequence, by one warp.  Lane l holds the logits of experts
// l, l+32, ... in z[].  K rounds of warp arg-max (hardware redux on order-preserving 32-bit
// keys, then redux-min over the tied ids so the lower id wins), one more round for the
// K-th/(K+1)-th gap; ids are emitted in ascending order with w = softmax(z)[id].
template <int VPL>
__device__ __forceinline__ void route_token(const float (&z)[VPL], float *, int *s_ids_row, const TopkArgs &a,
                                            int b, int lane)
{
    constexpr int kVpl = VPL;  // logits per lane: experts lane, lane+32, ... (E <= 32*VPL)
    const int E = a.E, K = a.K;
    float m = -INFINITY;
    uint32_t key[kVpl];
#pragma unroll
    for (int v = 0; v < kVpl; ++v) {
        m = fmaxf(m, z[v]);
        key[v] = (v * kWarp + lane < E) ? float_key(z[v]) : 0u;  // 0 never wins: real keys are > 0
    }
    m = warp_max(m);
    float ex[kVpl], sum = 0.f;
#pragma unroll
    for (int v = 0; v < kVpl; ++v) {
        ex[v] = (v * kWarp + lane < E) ? expf(z[v] - m) : 0.f;
        sum += ex[v];
    }
    sum = warp_sum(sum);

    uint32_t taken = 0;  // bit v: my value v is selected
    float kth = 0.f, gap = INFINITY;
    for (int r = 0; r <= K && r < E; ++r) {
        uint32_t best = 0;
        int best_v = 0;
#pragma unroll
        for (int v = 0; v < kVpl; ++v)
            if (!((taken >> v) & 1u) && key[v] > best) best = key[v], best_v = v;  // first max = lowest id
        const uint32_t top = __reduce_max_sync(kFull, best);
        const uint32_t cand = (best == top && best != 0u) ? (uint32_t)(best_v * kWarp + lane) : 0xffffffffu;
        const int j = (int)__reduce_min_sync(kFull, cand);
        float zj = 0.f;
#pragma unroll
        for (int v = 0; v < kVpl; ++v)
            if (v == best_v) zj = z[v];
        zj = __shfl_sync(kFull, zj, j % kWarp);
        if (r < K) {
            if (j % kWarp == lane) taken |= 1u << (j / kWarp);
            kth = zj;
        } else {
            gap = kth - zj;
        }
    }

    float sel = 0.f;
#pragma unroll
    for (int v = 0; v < kVpl; ++v)
        if ((taken >> v) & 1u) sel += ex[v];
    sel = a.renorm ? warp_sum(sel) : sum;
    int base = 0;
#pragma unroll
    for (int v = 0; v < kVpl; ++v) {
        const unsigned msk = __ballot_sync(kFull, (taken >> v) & 1u);
        if ((taken >> v) & 1u) {
            const int pos = base + __popc(msk & ((1u << lane) - 1u));
            const int j = v * kWarp + lane;
            const float p = ex[v] / sel;
            a.ids[(size_t)b * K + pos] = j;
            a.w[(size_t)b * K + pos] = p;
            s_ids_row[pos] = j;
            if (a.ids_out) a.ids_out[(size_t)b * K + pos] = j;
            if (a.w_out) a.w_out[(size_t)b * K + pos] = p;
        }
        base += __popc(msk);
    }
    if (lane == 0) {
        const uint32_t f = gap < 1e-4f ? 1u : 0u;
        if (a.flags_out) a.flags_out[b] = f;
        if (f && a.near_tie_counter) atomicAdd(a.near_tie_counter, 1ull);
    }
    __syncwarp();
}

// Grouping of the batch's routed pairs by expert (256 threads, thread e owns expert e):
// entries of at most mt tokens in ascending expert order, then the shared experts.
// s_ids: [B*K] routed ids; s_scan: 2*(kMaxExperts+1) ints of scratch.
__device__ __forceinline__ void group_tokens(const int *s_ids, int *s_scan, int B, int E, int K, int n_shared,
                                             int mt, const WorkList &wl)
{
    if (B == 1) {  // one sequence: its K experts (already ascending), then the shared ones
        const int t = threadIdx.x;
        if (t < K + n_shared) {
            wl.g_expert[t] = t < K ? s_ids[t] : E + (t - K);
            wl.g_start[t] = t, wl.g_count[t] = 1;
            wl.pair_token[t] = 0, wl.pair_slot[t] = t;
        }
        if (t == 0) *wl.n_groups = K + n_shared;
        return;
    }
    // Thread e owns expert e for the counts and the entries; the pairs are placed by one thread
    // each: a 64-bit token mask per expert gives a pair's position inside its entry (tokens
    // ascending) without any thread walking the whole batch.
    __shared__ unsigned long long s_mask[kMaxExperts];
    int *s_g = s_scan, *s_p = s_scan + 8, *s_base = s_scan + 16;  // warp sums; first pair of each expert
    const int e = threadIdx.x, KS = K + n_shared, lane = e % kWarp, warp = e / kWarp;
    auto sync256 = []() { asm volatile("bar.sync 2, 256;" ::: "memory"); };
    s_mask[e] = 0ull;
    sync256();
    for (int i = e; i < B * K; i += 256) atomicOr(&s_mask[s_ids[i]], 1ull << (i / K));
    sync256();
    const int cnt = e < E ? __popcll(s_mask[e]) : 0;
    // exclusive scans of (entries, pairs) over the 256 experts
    int g_inc = (cnt + mt - 1) / mt, p_inc = cnt;
#pragma unroll
    for (int o = 1; o < kWarp; o <<= 1) {
        const int tg = __shfl_up_sync(kFull, g_inc, o), tp = __shfl_up_sync(kFull, p_inc, o);
        if (lane >= o) g_inc += tg, p_inc += tp;
    }
    if (lane == kWarp - 1) s_g[warp] = g_inc, s_p[warp] = p_inc;
    sync256();
    int g0 = g_inc - (cnt + mt - 1) / mt, p0 = p_inc - cnt, g_all = 0;
    for (int wi = 0; wi < kMaxExperts / kWarp; ++wi) {
        if (wi < warp) g0 += s_g[wi], p0 += s_p[wi];
        g_all += s_g[wi];
    }
    s_base[e] = p0;
    sync256();
    if (e < E && cnt > 0) {
        for (int t = 0, g = g0; t < cnt; t += mt, ++g) {
            wl.g_expert[g] = e;
            wl.g_start[g] = p0 + t;
            wl.g_count[g] = min(mt, cnt - t);
        }
    }
    for (int i = e; i < B * K; i += 256) {
        const int x = s_ids[i], b = i / K;
        const int p = s_base[x] + __popcll(s_mask[x] & ((1ull << b) - 1ull));
        wl.pair_token[p] = b;
        wl.pair_slot[p] = b * KS + i % K;
    }
    const int tiles = (B + mt - 1) / mt;
    for (int i = e; i < n_shared * tiles; i += 256) {
        const int sh = i / tiles, t = i % tiles;
        const int g = g_all + i;
        wl.g_expert[g] = E + sh;
        wl.g_start[g] = B * K + sh * B + t * mt;
        wl.g_count[g] = min(mt, B - t * mt);
    }
    for (int i = e; i < n_shared * B; i += 256) {
        const int sh = i / B, b = i % B;
        wl.pair_token[B * K + i] = b;
        wl.pair_slot[B * K + i] = b * KS + K + sh;
    }
    if (threadIdx.x == 0) *wl.n_groups = g_all + n_shared * tiles;
}

// Stand-alone softmax/top-K/grouping over ready logits.  One CTA, one warp per sequence.
__global__ void __launch_bounds__(256) topk_group_kernel(TopkArgs a)
{
    constexpr int NW = 8;
    __shared__ int s_ids[kMaxBatch * kMaxTopK];
    __shared__ int s_scan[2 * (kMaxExperts + 1)];
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
    for (int b = warp; b < a.B; b += NW) {
        float z[kVplMax];
#pragma unroll
        for (int v = 0; v < kVplMax; ++v) {
            const int j = v * kWarp + lane;
            z[v] = j < a.E ? a.logits[(size_t)b * a.E + j] : -INFINITY;
        }
        route_token<kVplMax>(z, nullptr, s_ids + b * a.K, a, b, lane);
    }
    if (a.wl.n_groups == nullptr) return;
    __syncthreads();
    group_tokens(s_ids, s_scan, a.B, a.E, a.K, a.n_shared, a.mt, a.wl);
}

// ---- the whole gating network in one launch -------------------------------------------------
// Split-K router GEMV over many CTAs (one warp per (expert row, column chunk), all of its
// loads issued up front), partial logits and partial sums of squares to global memory; the
// CTA that arrives last (arrival counter, no waiting) sums them in a fixed order, applies the
// RMSNorm factor and runs softmax / top-K / grouping.
// Column chunk of one task: 4 warp-wide 16-byte loads of weights for a single sequence (few,
// long tasks: the phase is one trip to memory either way), 1 for a batch, where the warp also
// has to fetch that chunk of every sequence's hidden state and short chunks keep all of those
// loads in flight at once.
template <int DT> __host__ __device__ constexpr int router_chunk_cols(int batch)
{
    return kWarp * Fmt<DT>::kEpl * (batch == 1 ? 4 : 1);
}
template <int DT> __host__ __device__ constexpr int router_chunks(int hidden, int batch)
{
    return (hidden + router_chunk_cols<DT>(batch) - 1) / router_chunk_cols<DT>(batch);
}

struct RouterArgs {
    const float *h;      // [B][H]
    const uint8_t *W;    // [E][H]
    int H;
    float eps;
    float *part;         // [C][B][E] partial logits, C = router_chunks(H, B) column chunks
    float *ss_part;      // [C][B] partial sums of squares
    unsigned *arrivals;  // [1], zero between launches
    float *inv_rms;      // [B]
    float *logits_out;   // optional [B][E]
    TopkArgs tk;         // tk.logits unused
};

// One split-K task: partial logits of expert row j over column chunk c for every sequence
// (and, for j == 0, the partial sums of squares of that chunk).  U = weight loads per lane
// (4: single sequence, 1: batch).  kPdl: wait for the previous kernel between loading the
// (independent) router weights and reading h.
template <int DT, int U, bool kPdl>
__device__ __forceinline__ void router_task(const RouterArgs &a, int task, int lane)
{
    constexpr int EPL = Fmt<DT>::kEpl, BYTES = Fmt<DT>::kBytes, CH = kWarp * EPL * U;
    constexpr int TB = U == 1 ? 8 : 1;  // sequences whose loads are issued together
    const int B = a.tk.B, E = a.tk.E, H = a.H;
    const int C = (H + CH - 1) / CH;
    const int j = task / C, c = task % C;
    const uint8_t *row = a.W + (size_t)j * H * BYTES;
    float wf[U][EPL];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int k = c * CH + (u * kWarp + lane) * EPL;
        if (k < H) {
            Fmt<DT>::unpack(ld_stream16(row + (size_t)k * BYTES), wf[u]);
        } else {
#pragma unroll
            for (int e = 0; e < EPL; ++e) wf[u][e] = 0.f;
        }
    }
    if (kPdl) pdl_wait();  // the router weights above do not depend on the previous kernel; h does
    for (int b0 = 0; b0 < B; b0 += TB) {
        float4 hv[TB][U][EPL / 4];
#pragma unroll
        for (int t = 0; t < TB; ++t)
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int k = c * CH + (u * kWarp + lane) * EPL;
#pragma unroll
                for (int e = 0; e < EPL / 4; ++e)
                    hv[t][u][e] = (k < H && b0 + t < B) ? ld_f4(a.h + (size_t)(b0 + t) * H + k + 4 * e)
                                                        : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
        for (int t = 0; t < TB; ++t) {
            float acc = 0.f, ss = 0.f;
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int e = 0; e < EPL / 4; ++e) {
                    const float4 v = hv[t][u][e];
                    acc = fmaf(wf[u][4 * e], v.x, acc), acc = fmaf(wf[u][4 * e + 1], v.y, acc);
                    acc = fmaf(wf[u][4 * e + 2], v.z, acc), acc = fmaf(wf[u][4 * e + 3], v.w, acc);
                    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
                }
            acc = warp_sum(acc);
            if (j == 0) ss = warp_sum(ss);
            if (lane == 0 && b0 + t < B) {
                a.part[((size_t)c * B + b0 + t) * E + j] = acc;
                if (j == 0) a.ss_part[c * B + b0 + t] = ss;
            }
        }
    }
}

// All split-K tasks of a layer's gating network, dealt over `n_warps` warps of which this is
// number `w` (tasks w, w + n_warps, ...).
template <int DT, bool kPdl>
__device__ __forceinline__ void router_tasks(const RouterArgs &a, int w, int n_warps, int lane)
{
    const int B = a.tk.B;
    const int n_tasks = a.tk.E * (B == 1 ? router_chunks<DT>(a.H, 1) : router_chunks<DT>(a.H, 2));
    for (int task = w; task < n_tasks; task += n_warps) {
        if (B == 1)
            router_task<DT, 4, kPdl>(a, task, lane);
        else
            router_task<DT, 1, kPdl>(a, task, lane);
    }
}

// Gating of a single sequence by the first 256 threads of the CTA (thread j owns expert j):
// the latency-critical batch-1 case, where one warp would walk K+1 arg-max rounds alone.
// Every thread sums its own logit, the softmax statistics are two block reductions, and the
// top-K is found by rank counting (rank_j = number of experts that beat j; ties: lower id
// wins), which takes E comparisons per thread but no dependent rounds.  scratch: 320 ints.
template <int DT>
__device__ __forceinline__ void route_single_block(const RouterArgs &a, int *s_ids, int *scratch)
{
    const int j = threadIdx.x, lane = j % kWarp, warp = j / kWarp;
    const int E = a.tk.E, K = a.tk.K, H = a.H;
    const int C = router_chunks<DT>(H, 1);
    uint32_t *s_key = reinterpret_cast<uint32_t *>(scratch);      // [256]
    float *s_red = reinterpret_cast<float *>(scratch + 256);      // [8] max, [8] sum, [8] selected sum
    float *s_pick = reinterpret_cast<float *>(scratch + 256 + 24); // [0] K-th logit, [1] (K+1)-th
    int *s_cnt = scratch + 256 + 32;                              // [8] selected per warp
    auto sync256 = []() { asm volatile("bar.sync 2, 256;" ::: "memory"); };

    // Partials in one trip to L2.  The sums of squares are fetched one chunk per lane and summed
    // across the warp: every CTA of a persistent grid reads these same few lines at the same
    // moment, and the L2 slice that holds them serves the requests one by one.
    float ss = 0.f, s = 0.f;
    for (int c = lane; c < C; c += kWarp) ss += __ldcg(a.ss_part + c);
    for (int c0 = 0; c0 < C; c0 += 8) {
        float lp[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) lp[i] = (c0 + i < C && j < E) ? __ldcg(a.part + (size_t)(c0 + i) * E + j) : 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (c0 + i < C) s += lp[i];
    }
    ss = warp_sum(ss);
    const float inv = 1.0f / sqrtf(ss / (float)H + a.eps);
    if (j == 0) a.inv_rms[0] = inv;
    float z = -INFINITY;
    if (j < E) {
        z = s * inv;
        if (a.logits_out) a.logits_out[j] = z;
    }
    const uint32_t key = j < E ? float_key(z) : 0u;
    s_key[j] = key;
    const float wm = warp_max(z);
    if (lane == 0) s_red[warp] = wm;
    sync256();
    float m = s_red[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) m = fmaxf(m, s_red[w]);
    const float ex = j < E ? expf(z - m) : 0.f;
    const float wsum = warp_sum(ex);
    if (lane == 0) s_red[8 + warp] = wsum;

    int rank = 0;
    if (j < E)
        for (int i = 0; i < E; ++i) {
            const uint32_t k = s_key[i];
            rank += (k > key) || (k == key && i < j);
        }
    const bool sel = j < E && rank < K;
    if (j < E && rank == K - 1) s_pick[0] = z;
    if (j < E && rank == K) s_pick[1] = z;
    const unsigned msk = __ballot_sync(kFull, sel);
    const float wsel = warp_sum(sel ? ex : 0.f);
    if (lane == 0) s_cnt[warp] = __popc(msk), s_red[16 + warp] = wsel;
    sync256();
    float sum = 0.f, selsum = 0.f;
    int pos = __popc(msk & ((1u << lane) - 1u));
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        sum += s_red[8 + w], selsum += s_red[16 + w];
        if (w < warp) pos += s_cnt[w];
    }
    if (sel) {
        const float p = ex / (a.tk.renorm ? selsum : sum);
        a.tk.ids[pos] = j, a.tk.w[pos] = p, s_ids[pos] = j;
        if (a.tk.ids_out) a.tk.ids_out[pos] = j;
        if (a.tk.w_out) a.tk.w_out[pos] = p;
    }
    if (j == 0) {
        const float gap = K < E ? s_pick[0] - s_pick[1] : INFINITY;
        const uint32_t f = gap < 1e-4f ? 1u : 0u;
        if (a.tk.flags_out) a.tk.flags_out[0] = f;
        if (f && a.tk.near_tie_counter) atomicAdd(a.tk.near_tie_counter, 1ull);
    }
}

// Sequences b = warp, warp + nw, ...: sum the split-K partials in a fixed order, apply the RMSNorm
// factor, softmax / top-K by one warp each.  VPL = logits per lane (E <= 32*VPL).
template <int VPL>
__device__ __forceinline__ void finalize_tokens(const RouterArgs &a, int *s_ids, int nw, int C)
{
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
    const int B = a.tk.B, E = a.tk.E, H = a.H;
    for (int b = warp; b < B; b += nw) {
        float ss = 0.f;
        for (int c = lane; c < C; c += kWarp) ss += __ldcg(a.ss_part + c * B + b);
        ss = warp_sum(ss);
        const float inv = 1.0f / sqrtf(ss / (float)H + a.eps);
        if (lane == 0) a.inv_rms[b] = inv;
        // partial logits of this lane's experts: eight chunks of every expert per trip to L2,
        // summed in chunk order
        float z[VPL];
#pragma unroll
        for (int v = 0; v < VPL; ++v) z[v] = 0.f;
        for (int c0 = 0; c0 < C; c0 += 8) {
            float t[VPL][8];
#pragma unroll
            for (int v = 0; v < VPL; ++v)
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int j = v * kWarp + lane;
                    t[v][i] = (c0 + i < C && j < E) ? __ldcg(a.part + ((size_t)(c0 + i) * B + b) * E + j) : 0.f;
                }
#pragma unroll
            for (int v = 0; v < VPL; ++v)
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (c0 + i < C) z[v] += t[v][i];
        }
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int j = v * kWarp + lane;
            z[v] = j < E ? z[v] * inv : -INFINITY;
            if (j < E && a.logits_out) a.logits_out[(size_t)b * E + j] = z[v];
        }
        route_token<VPL>(z, nullptr, s_ids + b * a.tk.K, a.tk, b, lane);
    }
}

// Sum the split-K partials, softmax/top-K every sequence and group the batch by expert.  Needs
// all 256+ threads of the CTA for the grouping; s_ids [B*K], s_scan [2*(kMaxExperts+1)].
template <int DT>
__device__ __forceinline__ void router_finalize(const RouterArgs &a, int *s_ids, int *s_scan, int nw)
{
    const int B = a.tk.B, E = a.tk.E, H = a.H;
    const int C = router_chunks<DT>(H, B);
    if (B == 1) {
        if (threadIdx.x < 256) route_single_block<DT>(a, s_ids, s_scan);
    } else if (E <= 32) {
        finalize_tokens<1>(a, s_ids, nw, C);
    } else if (E <= 64) {
        finalize_tokens<2>(a, s_ids, nw, C);
    } else if (E <= 128) {
        finalize_tokens<4>(a, s_ids, nw, C);
    } else {
        finalize_tokens<kVplMax>(a, s_ids, nw, C);
    }
    if (a.tk.wl.n_groups == nullptr) return;
    __syncthreads();
    if (threadIdx.x < 256) group_tokens(s_ids, s_scan, B, E, a.tk.K, a.tk.n_shared, a.tk.mt, a.tk.wl);
}

template <int DT>
__global__ void __launch_bounds__(512) router_fused_kernel(RouterArgs a)
{
    const int NW = blockDim.x / kWarp;  // 8 warps; 16 for larger batches (the last CTA routes one sequence per warp)
    __shared__ int s_ids[kMaxBatch * kMaxTopK];
    __shared__ int s_scan[2 * (kMaxExperts + 1)];
    __shared__ int s_last;
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
    router_tasks<DT, true>(a, blockIdx.x * NW + warp, gridDim.x * NW, lane);
    pdl_wait();  // warps without a task: nothing below may run ahead of the previous kernel either
    // arrival: the CTA barrier orders the warps' partial stores before thread 0's acquire-release
    // atomic, which publishes them and, for the CTA that arrives last, brings in everyone else's
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned prev;
        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(prev) : "l"(a.arrivals) : "memory");
        s_last = prev == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    if (threadIdx.x == 0) *a.arrivals = 0u;
    router_finalize<DT>(a, s_ids, s_scan, NW);
}

}  // namespace stmoe_dev
