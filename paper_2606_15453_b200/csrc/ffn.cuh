// Routed SwiGLU expert FFN (Section 2: experts are feed-forward networks whose outputs are
// summed with the gating probabilities as weights), written as weight-streaming GEMVs: the
// step is bound by reading every routed expert's weights once from HBM.
//
// Scheduling.  The rows of all work-list entries form one index space.  Each CTA owns an
// equal contiguous share of it (to within one row), so every SM streams the same number of
// bytes; inside the CTA the warps claim blocks of R rows from a shared-memory ticket, so a
// warp that finishes early takes more.  A warp streams its rows 16 bytes per lane per load
// with R*U loads (per matrix) in flight and reduces the split-K partial sums with shuffles.
// Activations are re-read through L1.  Partial outputs go to fixed places and are summed in
// a fixed order, so results are reproducible run to run (no floating-point atomics).
#pragma once
#include "device_utils.cuh"
#include "router.cuh"

namespace stmoe_dev {

#ifndef STMOE_FFN_THREADS
#define STMOE_FFN_THREADS 512  // one CTA of 16 warps per SM
#endif
constexpr int kFfnThreads = STMOE_FFN_THREADS;

// Tile shapes of the one-token code path (rows per block, loads in flight per row) and the
// longest row segment of the down projection; overridable for tuning builds.
#ifndef STMOE_RG1
#define STMOE_RG1 2
#define STMOE_UG1 4
#define STMOE_RD1 8
#define STMOE_UD1 2
#endif
#ifndef STMOE_SEG_BYTES
#define STMOE_SEG_BYTES 16384
#endif
constexpr int kFfnWarps = kFfnThreads / kWarp;

struct FfnArgs {
    const float *h;          // [B][H] layer input (un-normalised)
    const float *inv_rms;    // [B] or nullptr (x = h)
    WorkList wl;
    const uint8_t *const *blob;  // [E + n_shared] expert image of each expert for this layer
    float *act;              // [B*(K+n_shared)][I]
    float *part;             // [B*(K+n_shared)][S][H]
    int H, I, E;
    int S;                   // column splits of the down projection
    // fused weighted sum + residual (done by whichever warp completes a 32-row tile last)
    const float *w;          // [B][K] gate weights
    float *h_out;            // [B][H]
    unsigned *tile_done;     // [ceil(H/32)] rows finished per tile, zero between launches
    int B, K, n_shared;
    float residual_scale;
};

constexpr int kTileRows = 32;

// Layout of one expert image.
__host__ __device__ inline size_t image_gate(int, int, int) { return 0; }
__host__ __device__ inline size_t image_up(int H, int I, int wb) { return (size_t)H * I * wb; }
__host__ __device__ inline size_t image_down(int H, int I, int wb) { return 2 * (size_t)H * I * wb; }
__host__ __device__ inline size_t image_scales(int H, int I, int wb) { return 3 * (size_t)H * I * wb; }

// acc[m][r][t] += sum over this lane's columns of W_m[row r][col] * x_t[col], rows r < nrows
template <int DT, int NMAT, int R, int MT, int U>
__device__ __forceinline__ void gemv_rows(const uint8_t *(&rowp)[NMAT][R], int nrows, const float *(&xp)[MT],
                                          int cols, int lane, float (&acc)[NMAT][R][MT])
{
    constexpr int EPL = Fmt<DT>::kEpl, BYTES = Fmt<DT>::kBytes, STEP = kWarp * EPL;
    for (int k0 = lane * EPL; k0 < cols; k0 += STEP * U) {
        uint4 wv[U][NMAT][R];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int k = k0 + u * STEP;
#pragma unroll
            for (int m = 0; m < NMAT; ++m)
#pragma unroll
                for (int r = 0; r < R; ++r)
                    if (k < cols && r < nrows)
                        wv[u][m][r] = ld_stream16(rowp[m][r] + (size_t)k * BYTES);
                    else
                        wv[u][m][r] = make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int k = k0 + u * STEP;
            if (k < cols) {
                float xv[MT][EPL];
#pragma unroll
                for (int t = 0; t < MT; ++t)
#pragma unroll
                    for (int e = 0; e < EPL; e += 4) {
                        const float4 v = ld_f4(xp[t] + k + e);
                        xv[t][e] = v.x, xv[t][e + 1] = v.y, xv[t][e + 2] = v.z, xv[t][e + 3] = v.w;
                    }
#pragma unroll
                for (int m = 0; m < NMAT; ++m)
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        float wf[EPL];
                        Fmt<DT>::unpack(wv[u][m][r], wf);
#pragma unroll
                        for (int t = 0; t < MT; ++t)
#pragma unroll
                            for (int e = 0; e < EPL; ++e) acc[m][r][t] = fmaf(wf[e], xv[t][e], acc[m][r][t]);
                    }
            }
        }
    }
}

// Cost of streaming one row for a work-list entry, in units of a one-token row: the
// multi-token code path keeps fewer loads in flight and does more arithmetic per byte, and
// measures about twice as slow per row.
constexpr int kMultiTokenRowCost = 2;

// Hands out the CTA's share [first, last) of the rows (rpe per work-list entry) in blocks of R
// to its warps.  The shares are equal in cost, not in rows: with kWeighted, rows of entries that
// hold more than one token count kMultiTokenRowCost times, so a CTA that gets them gets fewer.
// s_tk: three ints of shared memory (ticket, first, last).
struct BlockTickets {
    int first, last;

    // row index at which the cumulative cost reaches `target` (warp 0, all lanes)
    static __device__ int row_at_cost(const WorkList &wl, int n_groups, int rpe, long long target, int lane)
    {
        long long base = 0;  // cost of the entries before the chunk being scanned
        for (int g0 = 0; g0 < n_groups; g0 += kWarp) {
            const int g = g0 + lane;
            const int w = g < n_groups ? (wl.g_count[g] > 1 ? kMultiTokenRowCost : 1) : 0;
            int incl = w;
#pragma unroll
            for (int o = 1; o < kWarp; o <<= 1) {
                const int t = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += t;
            }
            const long long end = base + (long long)incl * rpe;        // cost up to and including g
            const long long beg = end - (long long)w * rpe;
            const unsigned hit = __ballot_sync(kFull, w > 0 && target >= beg && target < end);
            if (hit) {
                const int src = __ffs(hit) - 1;
                const long long b = __shfl_sync(kFull, beg, src);
                const int ws = __shfl_sync(kFull, w, src);
                return (g0 + src) * rpe + (int)((target - b) / ws);
            }
            base = __shfl_sync(kFull, end, kWarp - 1);
        }
        return n_groups * rpe;
    }

    template <bool kWeighted> __device__ void init(const WorkList &wl, int rpe, int *s_tk)
    {
        const int n_groups = *wl.n_groups;
        if (!kWeighted) {
            const int total = n_groups * rpe;
            first = (int)((long long)total * blockIdx.x / gridDim.x);
            last = (int)((long long)total * (blockIdx.x + 1) / gridDim.x);
            if (threadIdx.x == 0) s_tk[0] = first;
            __syncthreads();
            return;
        }
        if (threadIdx.x < kWarp) {
            const int lane = threadIdx.x;
            long long cost = 0;
            for (int g = lane; g < n_groups; g += kWarp) cost += wl.g_count[g] > 1 ? kMultiTokenRowCost : 1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cost += __shfl_xor_sync(kFull, cost, o);
            cost *= rpe;
            const int f = row_at_cost(wl, n_groups, rpe, cost * blockIdx.x / gridDim.x, lane);
            const int l = blockIdx.x + 1 == gridDim.x ? n_groups * rpe
                                                      : row_at_cost(wl, n_groups, rpe, cost * (blockIdx.x + 1) / gridDim.x, lane);
            if (lane == 0) s_tk[0] = f, s_tk[1] = f, s_tk[2] = l;
        }
        __syncthreads();
        first = s_tk[1], last = s_tk[2];
    }
    __device__ int claim(int *s_tk, int R, int lane) const
    {
        int u = 0;
        if (lane == 0) u = atomicAdd(s_tk, R);
        return __shfl_sync(kFull, u, 0);
    }
};

// Output element (sequence b, column c) of the layer from the down projection's partial sums,
// in a fixed summation order: shared experts, then routed experts, segments innermost:
//   h_out[b][c] = h[b][c] + r * ( sum_shared part + sum_k w[b][k] * part ).
// The loads of eight terms are issued together (each is a trip to L2), the arithmetic keeps the
// fixed order.
__device__ __forceinline__ float finish_value(const FfnArgs &a, int b, int c, int S)
{
    const int H = a.H, KS = a.K + a.n_shared, n_terms = KS * S;
    float y = 0.f, p = 0.f;
    for (int t0 = 0; t0 < n_terms; t0 += 8) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int t = t0 + i, q = t / S, z = t % S;
            const int slot = q < a.n_shared ? a.K + q : q - a.n_shared;
            v[i] = t < n_terms ? __ldcg(a.part + (((size_t)b * KS + slot) * S + z) * H + c) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int t = t0 + i, q = t / S, z = t % S;
            if (t < n_terms) {
                p += v[i];
                if (z == S - 1) {
                    y = q < a.n_shared ? y + p : fmaf(a.w[b * a.K + q - a.n_shared], p, y);
                    p = 0.f;
                }
            }
        }
    }
    return fmaf(a.residual_scale, y, a.h[(size_t)b * H + c]);
}

// Fused weighted sum + residual.  Called by a whole warp after it has stored the partial sums
// of rows [r0, r0+nrows) of one (entry, segment): the rows are counted per 32-row tile, and the
// warp whose count completes a tile (want_per_row contributions for each of its rows) computes
// the tile's outputs.  No waiting is involved; the counter is left at zero for the next launch.
__device__ __forceinline__ void finish_rows(const FfnArgs &a, int r0, int nrows, int want_per_row, int S, int lane)
{
    const int H = a.H;
    // The warp's lanes have stored their partial sums; the warp barrier orders those stores before
    // lane 0's counter update, whose release makes them visible to whoever reads the count, and whose
    // acquire (handed to the other lanes by the shuffle) orders the finisher's loads after every
    // earlier contributor's release: one acquire-release atomic instead of two full fences.
    __syncwarp();
    for (int rr = r0; rr < r0 + nrows;) {
        const int tile = rr / kTileRows;
        const int n = min(r0 + nrows, (tile + 1) * kTileRows) - rr;
        const int tile_rows = min(kTileRows, H - tile * kTileRows);
        unsigned prev = 0;
        if (lane == 0)
            asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], %2;"
                         : "=r"(prev)
                         : "l"(a.tile_done + tile), "r"((unsigned)n)
                         : "memory");
        prev = __shfl_sync(kFull, prev, 0);
        if (prev + n == (unsigned)(want_per_row * tile_rows)) {
            if (lane == 0) a.tile_done[tile] = 0u;
            const int c = tile * kTileRows + lane;
            if (lane < tile_rows)
                for (int b = 0; b < a.B; ++b) a.h_out[(size_t)b * H + c] = finish_value(a, b, c, S);
        }
        rr += n;
    }
}

// What a warp needs to know about a work-list entry, kept in registers across the blocks it
// claims: consecutive blocks nearly always belong to the same entry, and looking the entry up
// costs two dependent trips to L2 before the first weight load can be issued.
template <int MT> struct Entry {
    int g = -1, cnt = 0;
    const uint8_t *img = nullptr;
    int tok[MT], slot[MT];
    float inv[MT];
    __device__ __forceinline__ void load(const FfnArgs &a, int g_new)
    {
        if (g_new == g) return;
        g = g_new;
        img = a.blob[a.wl.g_expert[g]];
        const int start = a.wl.g_start[g];
        cnt = a.wl.g_count[g];
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            const int p = start + min(t, cnt - 1);
            tok[t] = a.wl.pair_token[p], slot[t] = a.wl.pair_slot[p];
            inv[t] = a.inv_rms ? a.inv_rms[tok[t]] : 1.f;
        }
    }
};

// One block of the gate/up projection: rows [r0, r0+nrows) (nrows <= R) of work-list entry g.
// act[slot][i] = silu(g_i) * u_i,  g = W_g x, u = W_u x,  x = h * inv_rms  (folded into g, u)
template <int DT, int R, int MT, int U, int MTE>
__device__ __forceinline__ void gate_up_block(const FfnArgs &a, const Entry<MTE> &en, int r0, int nrows, int lane)
{
    constexpr int BYTES = Fmt<DT>::kBytes;
    const int H = a.H, I = a.I;
    const size_t row_bytes = (size_t)H * BYTES;
    const int cnt = en.cnt;
    const uint8_t *img = en.img;
    const uint8_t *rowp[2][R];
    const float *xp[MT];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        rowp[0][r] = img + image_gate(H, I, BYTES) + (size_t)(r0 + r) * row_bytes;
        rowp[1][r] = img + image_up(H, I, BYTES) + (size_t)(r0 + r) * row_bytes;
    }
#pragma unroll
    for (int t = 0; t < MT; ++t) xp[t] = a.h + (size_t)en.tok[t] * H;
    float acc[2][R][MT];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int t = 0; t < MT; ++t) acc[m][r][t] = 0.f;
    gemv_rows<DT, 2, R, MT, U>(rowp, nrows, xp, H, lane, acc);

    const uint16_t *sc = reinterpret_cast<const uint16_t *>(img + image_scales(H, I, BYTES));
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            float gv = warp_sum(acc[0][r][t]), uv = warp_sum(acc[1][r][t]);
            if (lane == (r * MT + t) % kWarp && r < nrows && t < cnt) {
                gv *= en.inv[t], uv *= en.inv[t];
                if (DT == 2) {
                    gv *= bf16_to_f32(sc[r0 + r]);
                    uv *= bf16_to_f32(sc[I + r0 + r]);
                }
                a.act[(size_t)en.slot[t] * I + r0 + r] = gv / (1.f + expf(-gv)) * uv;
            }
        }
}

// Tile shapes: R rows per block and U loads in flight per row, for entries of one token (the
// batch-1 shape, widest loads) and for entries of up to four tokens.
template <int DT> struct TileShape {
    static constexpr int RG1 = STMOE_RG1, UG1 = STMOE_UG1, RD1 = STMOE_RD1, UD1 = STMOE_UD1;
    static constexpr int RG4 = 2, UG4 = DT == 2 ? 1 : 2, RD4 = DT == 2 ? 2 : 4, UD4 = 2;
};

// Work-list entries are walked in claims of RG1 rows; an entry that holds one token takes the
// one-token code path even in the multi-token kernel (MTMAX = 4), so a batch whose sequences
// mostly route to different experts streams as fast as batch 1.
struct NoSideWork {
    __device__ void operator()() const {}
};

// The rows of the gate/up projection this CTA owns.  side() runs once per warp after the
// ticket counter is set up and before the warp starts claiming blocks (the persistent kernel
// parks the predictor there on one warp).
template <int DT, int MTMAX, typename Side = NoSideWork>
__device__ __forceinline__ void gate_up_phase(const FfnArgs &a, int *s_next, Side side = Side())
{
    using TS = TileShape<DT>;
    constexpr int RC = TS::RG1;
    const int lane = threadIdx.x % kWarp;
    const int I = a.I;
    BlockTickets tk;
    tk.init<(MTMAX > 1)>(a.wl, I, s_next);
    side();
    Entry<MTMAX> en;

    for (int u0 = tk.claim(s_next, RC, lane); u0 < tk.last; u0 = tk.claim(s_next, RC, lane)) {
        const int uend = min(u0 + RC, tk.last);
        for (int u = u0; u < uend;) {
            const int g = u / I, r0 = u % I;
            const int nrows = min(uend - u, I - r0);
            u += nrows;
            en.load(a, g);
            if (MTMAX == 1 || en.cnt == 1) {
                gate_up_block<DT, TS::RG1, 1, TS::UG1>(a, en, r0, nrows, lane);
            } else {
                for (int q = 0; q < nrows; q += TS::RG4)
                    gate_up_block<DT, TS::RG4, MTMAX, TS::UG4>(a, en, r0 + q, min(TS::RG4, nrows - q), lane);
            }
        }
    }
}

// Work-list entries are walked in claims of RG1 rows; an entry that holds one token takes the
// one-token code path even in the multi-token kernel (MTMAX = 4), so a batch whose sequences
// mostly route to different experts streams as fast as batch 1.
template <int DT, int MTMAX>
__global__ void __launch_bounds__(kFfnThreads, 1) gate_up_kernel(FfnArgs a)
{
    __shared__ int s_next[3];
    pdl_launch_dependents();  // the down kernel may move in behind the CTAs of this grid
    gate_up_phase<DT, MTMAX>(a, s_next);
}

// One block of the down projection: rows [r0, r0+nrows) of segment s of entry g.
// part[slot][s][h] = sum over the columns of split s of W_d[h][col] * act[slot][col]
template <int DT, int R, int MT, int U, int MTE>
__device__ __forceinline__ void down_block(const FfnArgs &a, const Entry<MTE> &en, int s, int seg, int r0, int nrows,
                                           int lane)
{
    constexpr int BYTES = Fmt<DT>::kBytes;
    const int H = a.H, I = a.I, S = a.S;
    const size_t row_bytes = (size_t)I * BYTES;
    const int c0 = s * seg, ncols = min(seg, I - c0);
    const int cnt = en.cnt;
    const uint8_t *img = en.img;
    const uint8_t *rowp[1][R];
    const float *xp[MT];
#pragma unroll
    for (int r = 0; r < R; ++r)
        rowp[0][r] = img + image_down(H, I, BYTES) + (size_t)(r0 + r) * row_bytes + (size_t)c0 * BYTES;
#pragma unroll
    for (int t = 0; t < MT; ++t) xp[t] = a.act + (size_t)en.slot[t] * I + c0;
    float acc[1][R][MT];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int t = 0; t < MT; ++t) acc[0][r][t] = 0.f;
    if (ncols > 0) gemv_rows<DT, 1, R, MT, U>(rowp, nrows, xp, ncols, lane, acc);

    const uint16_t *sc = reinterpret_cast<const uint16_t *>(img + image_scales(H, I, BYTES));
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            float v = warp_sum(acc[0][r][t]);
            if (lane == (r * MT + t) % kWarp && r < nrows && t < cnt) {
                if (DT == 2) v *= bf16_to_f32(sc[2 * I + r0 + r]);
                a.part[((size_t)en.slot[t] * S + s) * H + r0 + r] = v;
            }
        }
}

// The rows of the down projection this CTA owns.  kPdl: the stand-alone kernel is launched
// with programmatic serialization behind the gate/up kernel; the work list is older than that
// kernel, so the first claim can be made and the start of its weight rows pulled into L2 while
// gate/up is still finishing; only the activations have to wait.
template <int DT, int MTMAX, bool kPdl>
__device__ __forceinline__ void down_phase(const FfnArgs &a, int *s_next)
{
    using TS = TileShape<DT>;
    constexpr int EPL = Fmt<DT>::kEpl, RC = TS::RD1;
    const int lane = threadIdx.x % kWarp;
    const int H = a.H, I = a.I, S = a.S;
    // columns of one split, a multiple of one warp-wide load
    const int seg = ((I + S - 1) / S + kWarp * EPL - 1) / (kWarp * EPL) * (kWarp * EPL);
    BlockTickets tk;
    tk.init<(MTMAX > 1)>(a.wl, S * H, s_next);
    Entry<MTMAX> en;
    int u0 = tk.claim(s_next, RC, lane);
    if (kPdl) {
        if (u0 < tk.last) {
            const int g = u0 / (S * H), s = (u0 / H) % S, r0 = u0 % H;
            en.load(a, g);
            const int n = min(min(RC, tk.last - u0), H - r0);
            const size_t row_bytes = (size_t)I * Fmt<DT>::kBytes;
            // just what the first load step of each row needs
            const int seg_bytes = min(min(seg, I - s * seg) * Fmt<DT>::kBytes, TS::UD1 * kWarp * 16);
            const uint8_t *base = en.img + image_down(H, I, Fmt<DT>::kBytes) + (size_t)s * seg * Fmt<DT>::kBytes;
            for (int r = 0; r < n; ++r)
                for (int o = lane * 128; o < seg_bytes; o += kWarp * 128)
                    prefetch_l2(base + (size_t)(r0 + r) * row_bytes + o);
        }
        pdl_wait();
    }

    for (; u0 < tk.last; u0 = tk.claim(s_next, RC, lane)) {
        const int uend = min(u0 + RC, tk.last);
        for (int u = u0; u < uend;) {
            const int g = u / (S * H), s = (u / H) % S, r0 = u % H;
            const int nrows = min(uend - u, H - r0);
            u += nrows;
            en.load(a, g);
            if (MTMAX == 1 || en.cnt == 1) {
                down_block<DT, TS::RD1, 1, TS::UD1>(a, en, s, seg, r0, nrows, lane);
            } else {
                for (int q = 0; q < nrows; q += TS::RD4)
                    down_block<DT, TS::RD4, MTMAX, TS::UD4>(a, en, s, seg, r0 + q, min(TS::RD4, nrows - q), lane);
            }
            finish_rows(a, r0, nrows, *a.wl.n_groups * S, S, lane);
        }
    }
}

// ---- single-sequence schedule (persistent decode-step kernel, batch 1) ------------------------
// With one sequence the work of a layer is static once the K routed ids are known: K routed
// entries followed by the shared ones, one token each.  Two things differ from the general
// phases above.
//
// Row-slice partition.  CTA c owns rows [c*RPE/G, (c+1)*RPE/G) of EVERY entry (RPE rows per
// entry, G CTAs) instead of one contiguous range of the concatenated rows, so each CTA streams
// the same share of every expert: when part of the weights already sits in L2 (see below) all
// CTAs gain alike and none runs ahead of the others into the next grid barrier.
//
// On-chip staging.  Weights whose address is known before the phase that reads them are asked
// into L2 (prefetch hints, no data returns to the SM) while HBM would otherwise idle at a phase
// boundary: a warp that runs out of gate/up rows stages this CTA's rows of the down projection
// (known since the top-K) before it waits at the grid barrier; a warp that runs out of
// down-projection rows stages the next layer's shared experts (routing-independent) and a
// bounded prefix of the experts predicted for the next layer (Algorithm 2's prefetch set, one
// memory level below the paper's expert buffer: Section 4.3.4) before the barrier, the router
// GEMV and the top-K of that layer.  Results do not depend on whether a line was staged.
struct SliceTickets {
    int lo, len;     // first row of the slice, rows of the slice (per entry)
    int pitch;       // tickets per entry: len rounded up to whole claims, so no claim spans two entries
    int total;       // entries * pitch
    int base, rot, n;
    __device__ void init(int rpe, int n_entries, int claim_rows)
    {
        n = n_entries;
#ifdef STMOE_SINGLE_CONTIG
        const int all = rpe * n_entries;
        base = (int)((long long)all * blockIdx.x / gridDim.x);
        total = (int)((long long)all * (blockIdx.x + 1) / gridDim.x) - base;
        lo = 0, len = rpe, pitch = rpe, rot = 0;
#else
        base = 0;
        lo = (int)((long long)rpe * blockIdx.x / gridDim.x);
        len = (int)((long long)rpe * (blockIdx.x + 1) / gridDim.x) - lo;
        // whole claims per entry: a claim that spanned two entries would run the row block twice,
        // each time with some rows masked (measured: down phase 36 -> 48 us on the Mixtral shape)
        pitch = (len + claim_rows - 1) / claim_rows * claim_rows;
        rot = 0;
        total = n_entries * pitch;
#endif
    }
    // ticket v -> entry g and row offset o inside the slice (o >= len: padding, no row)
    __device__ __forceinline__ void decode(int v, int &g, int &o) const
    {
        const int q = (base + v) / pitch;
        o = (base + v) - q * pitch;
        g = q + rot;
        if (g >= n) g -= n;
    }
    __device__ int claim(int *s_tk, int R, int lane) const
    {
        int u = 0;
        if (lane == 0) u = atomicAdd(s_tk, R);
        return __shfl_sync(kFull, u, 0);
    }
};

// Where the images of one layer's experts live (resident stacks: one allocation, routed images
// [L][E] followed by the shared ones [L][n_shared]) and who is routed (shared memory).
struct SingleCtx {
    const uint8_t *routed0;  // image of (layer, expert 0)
    const uint8_t *shared0;  // image of (layer, shared 0)
    size_t img_bytes;
    const int *s_ids;        // [K] routed ids, ascending
    const float *s_inv;      // [1]
    int K;
    __device__ __forceinline__ const uint8_t *image(int g) const
    {
        return g < K ? routed0 + (size_t)s_ids[g] * img_bytes : shared0 + (size_t)(g - K) * img_bytes;
    }
    __device__ __forceinline__ void load(Entry<1> &en, int g) const
    {
        if (g == en.g) return;
        en.g = g, en.cnt = 1, en.img = image(g);
        en.tok[0] = 0, en.slot[0] = g, en.inv[0] = s_inv[0];
    }
};

#ifndef STMOE_STAGE_PIECE
#define STMOE_STAGE_PIECE 4096
#endif
// Hint [p, p+bytes) into L2, spread over `nw` warps of which this is number `w`: pieces of 4 KB,
// one 128-byte line per lane.
__device__ __forceinline__ void stage_range(const uint8_t *p, long long bytes, int w, int nw, int lane)
{
    for (long long o = (long long)w * STMOE_STAGE_PIECE; o < bytes; o += (long long)nw * STMOE_STAGE_PIECE) {
        const int n = (int)min((long long)STMOE_STAGE_PIECE, bytes - o);
#pragma unroll
        for (int q = 0; q < STMOE_STAGE_PIECE / (kWarp * 128); ++q)
            if ((q * kWarp + lane) * 128 < n) prefetch_l2(p + o + (q * kWarp + lane) * 128);
    }
}

// This CTA's slice of the down projection of entries [g0, g1), at most cap bytes per entry.
template <int DT>
__device__ __forceinline__ void stage_down_slices(const FfnArgs &a, const SingleCtx &cx, const SliceTickets &td,
                                                  int g0, int g1, long long cap, int w, int nw, int lane)
{
    constexpr int BYTES = Fmt<DT>::kBytes, EPL = Fmt<DT>::kEpl;
    const int H = a.H, I = a.I, S = a.S;
    const size_t row_bytes = (size_t)I * BYTES;
    const int seg = ((I + S - 1) / S + kWarp * EPL - 1) / (kWarp * EPL) * (kWarp * EPL);
    for (int g = g0; g < g1; ++g) {
        const uint8_t *down = cx.image(g) + image_down(H, I, BYTES);
        if (S == 1) {
            stage_range(down + (size_t)td.lo * row_bytes, min(cap, (long long)td.len * (long long)row_bytes), w, nw, lane);
        } else {  // rows cut into segments: one piece per (segment, row) of the slice
            long long done = 0;
            for (int u = td.lo + w; u < td.lo + td.len && done < cap; u += nw) {
                const int sgm = u / H, r = u % H;
                const int nb = min(seg, I - sgm * seg) * BYTES;
                stage_range(down + (size_t)r * row_bytes + (size_t)sgm * seg * BYTES, nb, 0, 1, lane);
                done += (long long)nb * nw;
            }
        }
    }
}

// This CTA's slice of the gate and up matrices of the expert whose image is img: rows
// [tg.lo, tg.lo + rows) of each.
template <int DT>
__device__ __forceinline__ void stage_gate_up_slice(const FfnArgs &a, const uint8_t *img, const SliceTickets &tg,
                                                    int rows, int w, int nw, int lane)
{
    constexpr int BYTES = Fmt<DT>::kBytes;
    const size_t row_bytes = (size_t)a.H * BYTES;
    const long long n = (long long)min(rows, tg.len) * (long long)row_bytes;
    stage_range(img + image_gate(a.H, a.I, BYTES) + (size_t)tg.lo * row_bytes, n, w, nw, lane);
    stage_range(img + image_up(a.H, a.I, BYTES) + (size_t)tg.lo * row_bytes, n, w, nw, lane);
}

// Gate/up rows of this CTA's slices.  side(): once per warp before it starts claiming.
// done(): once per warp when no rows are left (staging of what comes next).
template <int DT, typename Side, typename Done>
__device__ __forceinline__ void gate_up_single(const FfnArgs &a, const SingleCtx &cx, const SliceTickets &tk, int *s_tk,
                                               Side side, Done done)
{
    using TS = TileShape<DT>;
    constexpr int RC = TS::RG1;
    const int lane = threadIdx.x % kWarp;
    side();
    Entry<1> en;
    for (int v0 = tk.claim(s_tk, RC, lane); v0 < tk.total; v0 = tk.claim(s_tk, RC, lane)) {
        const int vend = min(v0 + RC, tk.total);
        for (int v = v0; v < vend;) {
            int g, o;
            tk.decode(v, g, o);
            if (o >= tk.len) break;  // padding at the end of an entry's tickets
            const int nrows = min(vend - v, tk.len - o);
            v += nrows;
            cx.load(en, g);
            gate_up_block<DT, TS::RG1, 1, TS::UG1>(a, en, tk.lo + o, nrows, lane);
        }
    }
    done();
}

// Down-projection rows of this CTA's slices with the fused weighted sum (n_entries entries
// contribute to every output row).
template <int DT, typename Done>
__device__ __forceinline__ void down_single(const FfnArgs &a, const SingleCtx &cx, const SliceTickets &tk, int *s_tk,
                                            int n_entries, Done done)
{
    using TS = TileShape<DT>;
    constexpr int EPL = Fmt<DT>::kEpl, RC = TS::RD1;
    const int lane = threadIdx.x % kWarp;
    const int H = a.H, I = a.I, S = a.S;
    const int seg = ((I + S - 1) / S + kWarp * EPL - 1) / (kWarp * EPL) * (kWarp * EPL);
    Entry<1> en;
    for (int v0 = tk.claim(s_tk, RC, lane); v0 < tk.total; v0 = tk.claim(s_tk, RC, lane)) {
        const int vend = min(v0 + RC, tk.total);
        for (int v = v0; v < vend;) {
            int g, o;
            tk.decode(v, g, o);
            if (o >= tk.len) break;  // padding at the end of an entry's tickets
            const int u = tk.lo + o, sgm = u / H, r0 = u % H;
            const int nrows = min(min(vend - v, tk.len - o), H - r0);
            v += nrows;
            cx.load(en, g);
            down_block<DT, TS::RD1, 1, TS::UD1>(a, en, sgm, seg, r0, nrows, lane);
            finish_rows(a, r0, nrows, n_entries * S, S, lane);
        }
    }
    done();
}

template <int DT, int MTMAX>
__global__ void __launch_bounds__(kFfnThreads, 1) down_kernel(FfnArgs a)
{
    __shared__ int s_next[3];
    pdl_launch_dependents();  // the next layer's router may move in behind this grid
    down_phase<DT, MTMAX, true>(a, s_next);
}

}  // namespace stmoe_dev
