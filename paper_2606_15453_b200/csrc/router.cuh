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

// softmax + top-K (K rounds of warp arg-max on (logit, lower id first) keys, one more round
// for the K-th/(K+1)-th gap), then grouping by expert.  One CTA, one warp per sequence.
__global__ void __launch_bounds__(256) topk_group_kernel(TopkArgs a)
{
    constexpr int NW = 8, VPL = kMaxExperts / kWarp;
    __shared__ float s_z[NW][kMaxExperts];
    __shared__ int s_ids[kMaxBatch * kMaxTopK];
    __shared__ int s_scan_g[kMaxExperts + 1], s_scan_p[kMaxExperts + 1];
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
    const int E = a.E, K = a.K;

    for (int b = warp; b < a.B; b += NW) {
        float z[VPL];
        float m = -INFINITY;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int j = v * kWarp + lane;
            z[v] = j < E ? a.logits[(size_t)b * E + j] : -INFINITY;
            if (j < E) s_z[warp][j] = z[v];
            m = fmaxf(m, z[v]);
        }
        m = warp_max(m);
        float sum = 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v)
            if (v * kWarp + lane < E) sum += expf(z[v] - m);
        sum = warp_sum(sum);
        __syncwarp();

        uint32_t taken = 0;  // bit v: my value v is selected
        float kth = 0.f, gap = INFINITY;
        for (int r = 0; r <= K && r < E; ++r) {
            unsigned long long best = 0;
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                const int j = v * kWarp + lane;
                if (j < E && !((taken >> v) & 1u)) {
                    const unsigned long long key =
                        ((unsigned long long)float_key(z[v]) << 32) | (uint32_t)(0xffffffffu - j);
                    best = key > best ? key : best;
                }
            }
            best = warp_max_u64(best);
            const int j = (int)(0xffffffffu - (uint32_t)best);
            if (r < K) {
                if (j % kWarp == lane) taken |= 1u << (j / kWarp);
                kth = s_z[warp][j];
            } else {
                gap = kth - s_z[warp][j];
            }
        }

        float sel = 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v)
            if ((taken >> v) & 1u) sel += expf(z[v] - m);
        sel = warp_sum(sel);
        const float denom = a.renorm ? sel : sum;
        int base = 0;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const unsigned msk = __ballot_sync(kFull, (taken >> v) & 1u);
            if ((taken >> v) & 1u) {
                const int pos = base + __popc(msk & ((1u << lane) - 1u));
                const int j = v * kWarp + lane;
                const float p = expf(z[v] - m) / denom;
                a.ids[(size_t)b * K + pos] = j;
                a.w[(size_t)b * K + pos] = p;
                s_ids[b * K + pos] = j;
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
    }
    if (a.wl.n_groups == nullptr) return;
    __syncthreads();

    // grouping: thread e owns expert e
    const int e = threadIdx.x, KS = K + a.n_shared, mt = a.mt;
    int cnt = 0;
    if (e < E)
        for (int i = 0; i < a.B * K; ++i) cnt += (s_ids[i] == e);
    if (e < kMaxExperts) {
        s_scan_g[e + 1] = (cnt + mt - 1) / mt;
        s_scan_p[e + 1] = cnt;
    }
    if (e == 0) s_scan_g[0] = s_scan_p[0] = 0;
    __syncthreads();
    if (threadIdx.x == 0)
        for (int i = 1; i <= kMaxExperts; ++i) {
            s_scan_g[i] += s_scan_g[i - 1];
            s_scan_p[i] += s_scan_p[i - 1];
        }
    __syncthreads();
    if (e < E && cnt > 0) {
        const int g0 = s_scan_g[e], p0 = s_scan_p[e];
        for (int t = 0, g = g0; t < cnt; t += mt, ++g) {
            a.wl.g_expert[g] = e;
            a.wl.g_start[g] = p0 + t;
            a.wl.g_count[g] = min(mt, cnt - t);
        }
        int n = 0;
        for (int i = 0; i < a.B * K; ++i)
            if (s_ids[i] == e) {
                const int b = i / K, k = i % K;
                a.wl.pair_token[p0 + n] = b;
                a.wl.pair_slot[p0 + n] = b * KS + k;
                ++n;
            }
    }
    const int routed_groups = s_scan_g[kMaxExperts];
    const int tiles = (a.B + mt - 1) / mt;
    if (e < a.n_shared) {
        const int p0 = a.B * K + e * a.B;
        for (int t = 0; t < tiles; ++t) {
            const int g = routed_groups + e * tiles + t;
            a.wl.g_expert[g] = E + e;
            a.wl.g_start[g] = p0 + t * mt;
            a.wl.g_count[g] = min(mt, a.B - t * mt);
        }
        for (int b = 0; b < a.B; ++b) {
            a.wl.pair_token[p0 + b] = b;
            a.wl.pair_slot[p0 + b] = b * KS + K + e;
        }
    }
    if (threadIdx.x == 0) *a.wl.n_groups = routed_groups + a.n_shared * tiles;
}

}  // namespace stmoe_dev
