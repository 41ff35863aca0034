// One decode step of a resident stack for a single sequence with ONE weight-streaming phase per
// layer (Section 2: y = sum_k s_k FFN_k(x); Algorithms 1-3 beside it).
//
// The three-phase kernel (token_kernel.cuh) pays, per layer, for a gate/up phase, a grid barrier,
// a down phase with its own ramp-up and tail, and a third barrier; on small experts those
// boundaries cost as much as the streaming itself.  Here the down projection is consumed row by
// row together with the gate and up rows, from a transposed copy of the matrix:
//
//   for every row i of an expert:   a_i = silu(w_g[i].x) * (w_u[i].x)
//                                   y  += s_k * a_i * w_dT[i]          (w_dT[i] = column i of W_d)
//
// so a row triple (gate row, up row, transposed-down row: three contiguous rows of H elements) is
// a self-contained unit of work and a layer needs no barrier between its two projections.
//
// Column ownership.  A unit of TPR = H / EPL threads (EPL = elements per 16-byte load) owns a row
// at a time: thread t holds columns [t*EPL, (t+1)*EPL) of the hidden state, of x and of the
// output accumulator in registers for the whole launch, so no activation is ever re-read from
// memory.  A 512-thread CTA holds 512 / TPR independent units; all units of the grid but those
// of the last CTA stream an equal slice of the rows of every expert.  The two dot products of a
// row are reduced over the unit (a transposed warp butterfly, then one shared-memory exchange and
// a named barrier per block of two rows).  The rows reach the SM by bulk asynchronous copies
// (cp.async.bulk, completion counted on an mbarrier; no multicast) into a shared-memory ring of
// four blocks per unit, issued by the unit's first thread three blocks ahead of the arithmetic:
// 192 KB in flight per SM without holding a register, which the column-owner layout needs for its
// state.  A stage is free again once the unit has passed the barrier of the block that read it.
//
// Reductions across units are exact: every unit adds its part of the layer's MoE term to a
// per-layer accumulator in 64-bit fixed point (2^-40 units, integer atomics), which makes the
// result independent of the order of arrival; after the closing grid barrier every unit reads
// the sums for its own columns and forms h' = h + r*y.  The gating network needs one more
// barrier (router rows are dealt over the units, logits go through global memory, every unit
// runs softmax/top-K itself); the shared experts, which do not depend on the routing, are
// streamed between the arrival at that barrier and the wait for it.
// The last CTA streams nothing: its first warp runs the predictor and it writes the step's
// outputs.  Every wait is bounded as in token_kernel.cuh.
#pragma once
#include "dense_group.cuh"
#include "device_utils.cuh"
#include "ffn.cuh"
#include "predictor.cuh"
#include "router.cuh"
#include "token_kernel.cuh"

namespace stmoe_dev {

struct FusedArgs {
    TokenArgs t;                // shapes, router, images (store, img_bytes), outputs, predictor, barrier, err
    const uint8_t *down_t;      // transposed down projections [I][H], one per image, in image order
    size_t down_t_bytes;        // bytes of one of them
    float *zpart;               // [L][E] router dot products before the RMSNorm factor
    unsigned long long *acc;    // [L][H] fixed-point sums of the layers' MoE terms, zero at launch
    int poll_limit;             // polls before a grid-barrier wait gives up
};

constexpr int kFusedRows = 2;          // rows per block
constexpr int kFusedStages = 4;        // ring stages per unit (blocks in flight)
// ring bytes: units * stages * 3 matrices * rows * (H * element bytes) = 512 threads * 16 B * 24
constexpr int kFusedRingBytes = kFfnThreads * 16 * 3 * kFusedRows * kFusedStages;
constexpr int kFusedMaxUnits = 8;      // units per CTA (TPR >= 64)
constexpr float kFixScale = 1099511627776.0f;            // 2^40
constexpr double kFixInv = 9.094947017729282379150390625e-13;  // 2^-40

// Which shapes the kernel covers: a unit must be 2..16 whole warps.
__host__ __device__ inline bool fused_shape_ok(int H, int epl)
{
    const int tpr = H / epl;
    return H % epl == 0 && (tpr == 64 || tpr == 128 || tpr == 256 || tpr == 512);
}

struct UnitCtx {
    int tpr, grp, t, wig, nwg, lane, bar_id;
    float *red;      // [2][16][4] this unit's exchange buffers
    int par;         // which of the two is written next
};

__device__ __forceinline__ void unit_sync(const UnitCtx &u)
{
    asm volatile("bar.sync %0, %1;" ::"r"(u.bar_id), "r"(u.tpr) : "memory");
}

// Sum of one value over the unit, the same bits in every thread: warp butterfly, one slot per
// warp, barrier, slots added in warp order.
__device__ __forceinline__ float unit_sum(UnitCtx &u, float v)
{
    v = warp_sum(v);
    float *buf = u.red + u.par * 64;
    u.par ^= 1;
    if (u.lane == 0) buf[u.wig * 4] = v;
    unit_sync(u);
    float s = 0.f;
    for (int w = 0; w < u.nwg; ++w) s += buf[w * 4];
    return s;
}

__device__ __forceinline__ float unit_max(UnitCtx &u, float v)
{
    v = warp_max(v);
    float *buf = u.red + u.par * 64;
    u.par ^= 1;
    if (u.lane == 0) buf[u.wig * 4] = v;
    unit_sync(u);
    float s = -INFINITY;
    for (int w = 0; w < u.nwg; ++w) s = fmaxf(s, buf[w * 4]);
    return s;
}

// Sums of four values over the unit.  Inside a warp the four butterflies are folded into one:
// the first exchange leaves each half of the warp with two of the values, the second each
// quarter with one, three more finish it (6 shuffles instead of 20); lanes 0, 8, 16, 24 then
// hold the warp's sums of values 0..3.
__device__ __forceinline__ void unit_sum4(UnitCtx &u, float (&v)[4])
{
    const bool hi = u.lane & 16, q8 = u.lane & 8;
    float k0 = hi ? v[2] : v[0], k1 = hi ? v[3] : v[1];
    const float s0 = hi ? v[0] : v[2], s1 = hi ? v[1] : v[3];
    k0 += __shfl_xor_sync(kFull, s0, 16);
    k1 += __shfl_xor_sync(kFull, s1, 16);
    float k = q8 ? k1 : k0;
    const float s = q8 ? k0 : k1;
    k += __shfl_xor_sync(kFull, s, 8);
    k += __shfl_xor_sync(kFull, k, 4);
    k += __shfl_xor_sync(kFull, k, 2);
    k += __shfl_xor_sync(kFull, k, 1);
    float *buf = u.red + u.par * 64;
    u.par ^= 1;
    if ((u.lane & 7) == 0) buf[u.wig * 4 + (u.lane >> 3)] = k;
    unit_sync(u);
    // every warp adds the warps' sums up again for itself, spread over its lanes: lane i takes
    // slots i and i + 32 (slot = warp * 4 + value), lanes of equal i % 4 are folded together
    const int n = u.nwg * 4;
    float t = (u.lane < n ? buf[u.lane] : 0.f) + (u.lane + 32 < n ? buf[u.lane + 32] : 0.f);
    t += __shfl_xor_sync(kFull, t, 4);
    t += __shfl_xor_sync(kFull, t, 8);
    t += __shfl_xor_sync(kFull, t, 16);
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = __shfl_sync(kFull, t, i);
}

// Grid barrier whose participants are the units (one arrival each).
__device__ __forceinline__ void units_arrive(const UnitCtx &u, unsigned *counter)
{
    unit_sync(u);  // orders every thread's writes before the leader's release
    if (u.t == 0) asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(counter), "r"(1u) : "memory");
}

__device__ __forceinline__ void units_wait(const UnitCtx &u, unsigned *counter, unsigned *err, unsigned target,
                                           volatile int *s_dead, int poll_limit)
{
    if (u.t == 0 && !*s_dead) {
        int spins = 0;
        for (;;) {
            unsigned seen;
            asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if (seen >= target) break;
            if (++spins > poll_limit || ((spins & 255) == 0 && *((volatile unsigned *)err))) {
                *err = 1u;
                *s_dead = 1;
                break;
            }
        }
        asm volatile("{.reg .u32 t;\n\tld.acquire.gpu.global.u32 t, [%0];}" ::"l"(counter) : "memory");
    }
    unit_sync(u);
}

// Registers of one block in flight: kFusedRows rows of the three matrices (16 bytes each).
struct FusedBlock {
    uint4 g[kFusedRows], u[kFusedRows], d[kFusedRows];
};

// The row blocks a unit streams for a list of entries.  The blocks of all entries form one index
// space (bpe = ceil(I / R) blocks per entry); a unit owns a contiguous range of it, equal to
// within one block for all units.  Block q of the unit is global block first + q: rows
// [bi*R, bi*R + nrows) of entry (first + q) / bpe, bi = (first + q) % bpe.
template <int DT> struct FusedStream {
    static constexpr int EPL = Fmt<DT>::kEpl, BYTES = Fmt<DT>::kBytes, R = kFusedRows;
    const FusedArgs &fa;
    int layer, rows, bpe, first;   // rows per entry (I), blocks per entry, this unit's first global block
    bool shared;            // entries are the shared experts (weight 1), else the routed ones
    const int *s_ids;
    const float *s_w;
    size_t col_off;         // byte offset of this thread's columns in a row

    __device__ __forceinline__ size_t image_index(int entry) const
    {
        const TokenArgs &a = fa.t;
        return shared ? (size_t)a.L * a.E + (size_t)layer * a.n_shared + entry : (size_t)layer * a.E + s_ids[entry];
    }
    // the unit's first thread: bulk copies of block q into ring stage `stage`
    __device__ __forceinline__ void issue(int q, uint8_t *stage, uint64_t *full) const
    {
        const TokenArgs &a = fa.t;
        const int entry = (first + q) / bpe, bi = (first + q) % bpe;
        const int i0 = bi * R, nrows = min(R, rows - i0);
        const size_t idx = image_index(entry), row_bytes = (size_t)a.H * BYTES;
        const uint8_t *img = a.store + idx * a.img_bytes;
        const uint8_t *src[3] = {img + image_gate(a.H, a.I, BYTES) + (size_t)i0 * row_bytes,
                                 img + image_up(a.H, a.I, BYTES) + (size_t)i0 * row_bytes,
                                 fa.down_t + idx * fa.down_t_bytes + (size_t)i0 * row_bytes};
        const uint32_t bytes = (uint32_t)(nrows * row_bytes);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the stage was last read through the generic proxy
        dmbar_expect_tx(full, 3 * bytes);
#pragma unroll
        for (int m = 0; m < 3; ++m)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         :
                         : "r"(dsmem_u32(stage + (size_t)m * R * row_bytes)), "l"(src[m]), "r"(bytes), "r"(dsmem_u32(full))
                         : "memory");
    }
    // every thread: its 16 bytes of each row of block q from the stage
    __device__ __forceinline__ void fetch(int q, const uint8_t *stage, FusedBlock &b) const
    {
        const TokenArgs &a = fa.t;
        const int nrows = min(R, rows - ((first + q) % bpe) * R);
        const size_t row_bytes = (size_t)a.H * BYTES;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (r < nrows) {
                b.g[r] = *reinterpret_cast<const uint4 *>(stage + (size_t)r * row_bytes + col_off);
                b.u[r] = *reinterpret_cast<const uint4 *>(stage + (size_t)(R + r) * row_bytes + col_off);
                b.d[r] = *reinterpret_cast<const uint4 *>(stage + (size_t)(2 * R + r) * row_bytes + col_off);
            } else {
                b.g[r] = b.u[r] = b.d[r] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }
};

template <int DT, int RDT>
__global__ void __launch_bounds__(kFfnThreads, 1) decode_token_fused_kernel(FusedArgs fa)
{
    constexpr int EPL = Fmt<DT>::kEpl, BYTES = Fmt<DT>::kBytes, R = kFusedRows;
    constexpr int EPLR = Fmt<RDT>::kEpl, NRL = EPL / EPLR;  // router loads per thread and row
    static_assert(R == 2, "unit_sum4 reduces the two dot products of two rows");
    const TokenArgs &a = fa.t;
    const int L = a.L, E = a.E, K = a.K, H = a.H, I = a.I;
    __shared__ __align__(16) float s_red[kFusedMaxUnits][2 * 64];
    __shared__ uint32_t s_key[kFusedMaxUnits][kMaxExperts];
    __shared__ uint8_t s_sel[kFusedMaxUnits][kMaxExperts];
    __shared__ int s_ids[kFusedMaxUnits][kMaxTopK];
    __shared__ float s_w[kFusedMaxUnits][kMaxTopK];
    __shared__ float s_pick[kFusedMaxUnits][2];
    __shared__ int s_prev[kMaxTopK];
    __shared__ int s_dead;
    __shared__ __align__(8) uint64_t s_full[kFusedMaxUnits][kFusedStages];
    extern __shared__ __align__(128) uint8_t ring[];  // [unit][stage][gate rows | up rows | down^T rows]

    UnitCtx u;
    u.tpr = H / EPL;
    u.grp = threadIdx.x / u.tpr, u.t = threadIdx.x % u.tpr;
    u.wig = u.t / kWarp, u.nwg = u.tpr / kWarp, u.lane = threadIdx.x % kWarp;
    u.bar_id = 1 + u.grp;
    u.red = s_red[u.grp], u.par = 0;
    const int ng = kFfnThreads / u.tpr;
    const int unit = blockIdx.x * ng + u.grp, n_units = gridDim.x * ng;
    const bool service = blockIdx.x == gridDim.x - 1;
    const int n_stream = (gridDim.x - 1) * ng;
    if (threadIdx.x == 0) {
        s_dead = 0;
        for (int i = 0; i < kFusedMaxUnits * kFusedStages; ++i) dmbar_init(&s_full[0][0] + i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    unsigned target = 0;
    const size_t stage_bytes = (size_t)3 * R * H * BYTES;
    uint8_t *my_ring = ring + (size_t)u.grp * kFusedStages * stage_bytes;
    uint64_t *my_full = s_full[u.grp];
    unsigned blocks_done = 0;  // blocks this unit has consumed so far: ring position and phase

    // this thread's columns of the hidden state, carried in registers through all layers
    const int c0 = u.t * EPL;
    float h[EPL], y[EPL];
#pragma unroll
    for (int e = 0; e < EPL; e += 4) {
        const float4 v = ld_f4(a.h_in + c0 + e);
        h[e] = v.x, h[e + 1] = v.y, h[e + 2] = v.z, h[e + 3] = v.w;
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) y[e] = 0.f;

    FusedStream<DT> fs{fa};
    fs.rows = I, fs.bpe = (I + R - 1) / R;
    fs.col_off = (size_t)c0 * BYTES;
    fs.s_ids = s_ids[u.grp], fs.s_w = s_w[u.grp];

    for (int l = 0; l < L; ++l) {
        fs.layer = l;
        // ---- RMSNorm factor (every unit, same bits) -------------------------------------------
        float ss = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) ss = fmaf(h[e], h[e], ss);
        ss = unit_sum(u, ss);
        const float inv = 1.0f / sqrtf(ss / (float)H + a.eps);

        // ---- router rows dealt over the units ------------------------------------------------
        DBG_STAMP(l * 8 + 0);
        for (int j = unit; j < E; j += n_units) {
            const uint8_t *row = a.router + ((size_t)l * E + j) * H * Fmt<RDT>::kBytes + (size_t)c0 * Fmt<RDT>::kBytes;
            float p = 0.f;
#pragma unroll
            for (int q = 0; q < NRL; ++q) {
                float wf[EPLR];
                Fmt<RDT>::unpack(ld_stream16(row + q * 16), wf);
#pragma unroll
                for (int e = 0; e < EPLR; ++e) p = fmaf(wf[e], h[q * EPLR + e], p);
            }
            p = unit_sum(u, p);
            if (u.t == 0) fa.zpart[(size_t)l * E + j] = p;
        }
        target += n_units;
        units_arrive(u, a.barrier);
        DBG_STAMP(l * 8 + 1);

        // One pass over a list of entries: loads run one block ahead of the arithmetic.
        auto stream = [&](bool shared_entries, int n_entries) {
            fs.shared = shared_entries;
            const long long all = (long long)n_entries * fs.bpe;
            fs.first = (int)(all * unit / n_stream);
            const int nq = (int)(all * (unit + 1) / n_stream) - fs.first;
            if (nq == 0) return;
            float ye[DT == 2 ? EPL : 1];  // fp8: per-expert sums before the output-channel scales
            if (DT == 2) {
#pragma unroll
                for (int e = 0; e < EPL; ++e) ye[e] = 0.f;
            }
            auto compute = [&](int q, const FusedBlock &b) {
                const int entry = (fs.first + q) / fs.bpe, bi = (fs.first + q) % fs.bpe;
                const int i0 = bi * R;
                float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float wg[EPL], wu[EPL];
                    Fmt<DT>::unpack(b.g[r], wg);
                    Fmt<DT>::unpack(b.u[r], wu);
#pragma unroll
                    for (int e = 0; e < EPL; ++e) {
                        v[2 * r] = fmaf(wg[e], h[e], v[2 * r]);
                        v[2 * r + 1] = fmaf(wu[e], h[e], v[2 * r + 1]);
                    }
                }
                unit_sum4(u, v);
                const float wgt = shared_entries ? 1.f : fs.s_w[entry];
                const uint16_t *sc = nullptr;
                if (DT == 2)
                    sc = reinterpret_cast<const uint16_t *>(a.store + fs.image_index(entry) * a.img_bytes +
                                                            image_scales(H, I, BYTES));
                // odd lanes evaluate row 1, even lanes row 0; one exchange gives every lane both
                const int r_mine = u.lane & 1;
                float gv = (r_mine ? v[2] : v[0]) * inv, uv = (r_mine ? v[3] : v[1]) * inv;
                if (DT == 2 && i0 + r_mine < I) {
                    gv *= bf16_to_f32(sc[i0 + r_mine]);
                    uv *= bf16_to_f32(sc[I + i0 + r_mine]);
                }
                const float act_mine = gv / (1.f + expf(-gv)) * uv;  // rows past the end: zero weights, act = 0
                const float act_other = __shfl_xor_sync(kFull, act_mine, 1);
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float act = (r == r_mine) ? act_mine : act_other;
                    float wd[EPL];
                    Fmt<DT>::unpack(b.d[r], wd);
                    if (DT == 2) {
#pragma unroll
                        for (int e = 0; e < EPL; ++e) ye[e] = fmaf(act, wd[e], ye[e]);
                    } else {
                        const float aw = act * wgt;
#pragma unroll
                        for (int e = 0; e < EPL; ++e) y[e] = fmaf(aw, wd[e], y[e]);
                    }
                }
                if (DT == 2 && (bi == fs.bpe - 1 || q == nq - 1)) {  // done with this expert: output-channel scales, gate weight
#pragma unroll
                    for (int e = 0; e < EPL; ++e) {
                        y[e] = fmaf(wgt * bf16_to_f32(sc[2 * I + c0 + e]), ye[e], y[e]);
                        ye[e] = 0.f;
                    }
                }
            };
            constexpr int D = kFusedStages - 1;  // blocks the copies run ahead
            if (u.t == 0)
                for (int d = 0; d < D && d < nq; ++d) {
                    const unsigned pos = blocks_done + d;
                    fs.issue(d, my_ring + (pos % kFusedStages) * stage_bytes, my_full + pos % kFusedStages);
                }
            for (int q = 0; q < nq; ++q) {
                const unsigned pos = blocks_done + q;
                if (u.t == 0 && q + D < nq) {  // into the stage of block q-1, which the unit has left behind
                    const unsigned pn = pos + D;
                    fs.issue(q + D, my_ring + (pn % kFusedStages) * stage_bytes, my_full + pn % kFusedStages);
                }
                dmbar_wait(my_full + pos % kFusedStages, (pos / kFusedStages) & 1u, &s_dead);
                FusedBlock b;
                fs.fetch(q, my_ring + (pos % kFusedStages) * stage_bytes, b);
                compute(q, b);
            }
            blocks_done += nq;
        };

        // ---- shared experts: independent of the routing, streamed while the logits travel -----
        if (!service) stream(true, a.n_shared);
        units_wait(u, a.barrier, a.err, target, &s_dead, fa.poll_limit);
        DBG_STAMP(l * 8 + 2);

        // ---- softmax / top-K, by every unit for itself ----------------------------------------
        {
            constexpr int VPT = kMaxExperts / 64;  // experts a thread owns at the smallest unit
            float z[VPT], ex[VPT];
            uint32_t key[VPT];
            float zmax = -INFINITY;
#pragma unroll
            for (int q = 0; q < VPT; ++q) {
                const int j = u.t + q * u.tpr;
                z[q] = j < E ? __ldcg(fa.zpart + (size_t)l * E + j) * inv : -INFINITY;
                key[q] = j < E ? float_key(z[q]) : 0u;
                if (j < kMaxExperts) s_key[u.grp][j] = key[q];
                zmax = fmaxf(zmax, z[q]);
            }
            zmax = unit_max(u, zmax);
            float sum = 0.f;
#pragma unroll
            for (int q = 0; q < VPT; ++q) {
                ex[q] = (u.t + q * u.tpr) < E ? expf(z[q] - zmax) : 0.f;
                sum += ex[q];
            }
            sum = unit_sum(u, sum);
            bool sel[VPT];
            float selsum = 0.f;
#pragma unroll
            for (int q = 0; q < VPT; ++q) {
                const int j = u.t + q * u.tpr;
                sel[q] = false;
                if (j < E) {
                    int rank = 0;
                    for (int i = 0; i < E; ++i) {
                        const uint32_t k = s_key[u.grp][i];
                        rank += (k > key[q]) || (k == key[q] && i < j);
                    }
                    sel[q] = rank < K;
                    if (rank == K - 1) s_pick[u.grp][0] = z[q];
                    if (rank == K) s_pick[u.grp][1] = z[q];
                    s_sel[u.grp][j] = sel[q];
                    if (sel[q]) selsum += ex[q];
                }
            }
            selsum = unit_sum(u, selsum);  // its barrier also publishes s_sel and s_pick
#pragma unroll
            for (int q = 0; q < VPT; ++q) {
                const int j = u.t + q * u.tpr;
                if (j < E && sel[q]) {
                    int pos = 0;
                    for (int i = 0; i < j; ++i) pos += s_sel[u.grp][i];
                    s_ids[u.grp][pos] = j;
                    s_w[u.grp][pos] = ex[q] / (a.renorm ? selsum : sum);
                }
            }
            unit_sync(u);
            if (service && u.grp == 0) {  // the step's outputs
                if (u.t < K) {
                    const int id = s_ids[0][u.t];
                    a.ids_all[(size_t)l * a.Bmax * K + u.t] = id;
                    if (a.ids_out) a.ids_out[(size_t)l * K + u.t] = id;
                    if (a.w_out) a.w_out[(size_t)l * K + u.t] = s_w[0][u.t];
                }
                if (u.t == 0) {
                    const float gap = K < E ? s_pick[0][0] - s_pick[0][1] : INFINITY;
                    const uint32_t f = gap < 1e-4f ? 1u : 0u;
                    if (a.flags_out) a.flags_out[l] = f;
                    if (f) atomicAdd(a.pst.stats + 4, 1ull);
                }
            }
        }
        DBG_STAMP(l * 8 + 3);

        // ---- routed experts (streaming units); predictor (first warp of the service CTA) ------
        if (!service) {
            stream(false, K);
            DBG_STAMP(l * 8 + 4);
            // the CTA's units add up in shared memory (unit order), then one exact atomic per column
            float *ysum = reinterpret_cast<float *>(ring);  // every copy into the ring has been consumed
            __syncthreads();
#pragma unroll
            for (int e = 0; e < EPL; e += 4)
                *reinterpret_cast<float4 *>(ysum + (size_t)u.grp * H + c0 + e) = make_float4(y[e], y[e + 1], y[e + 2], y[e + 3]);
#pragma unroll
            for (int e = 0; e < EPL; ++e) y[e] = 0.f;
            __syncthreads();
            for (int c = threadIdx.x; c < H; c += kFfnThreads) {
                float v = 0.f;
                for (int g = 0; g < ng; ++g) v += ysum[(size_t)g * H + c];
                const long long fx = __float2ll_rn(v * kFixScale);
                asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(fa.acc + (size_t)l * H + c), "l"(fx) : "memory");
            }
            __syncthreads();  // the ring is written again only after everyone has read the sums
        } else if (threadIdx.x < kWarp) {
            predictor_step_group(a, l, s_ids[0], s_prev, 0, 1, u.lane);
            if (u.lane < K) s_prev[u.lane] = s_ids[0][u.lane];
            __syncwarp();
        }
        DBG_STAMP(l * 8 + 5);

        // ---- h' = h + r * y, from the exact sums ----------------------------------------------
        target += n_units;
        units_arrive(u, a.barrier);
        DBG_STAMP(l * 8 + 6);
        units_wait(u, a.barrier, a.err, target, &s_dead, fa.poll_limit);
        {
            const unsigned long long *acc = fa.acc + (size_t)l * H + c0;
#pragma unroll
            for (int e = 0; e < EPL; e += 2) {
                const ulonglong2 v = __ldcg(reinterpret_cast<const ulonglong2 *>(acc + e));
                h[e] = fmaf(a.residual_scale, (float)((double)(long long)v.x * kFixInv), h[e]);
                h[e + 1] = fmaf(a.residual_scale, (float)((double)(long long)v.y * kFixInv), h[e + 1]);
            }
        }
        DBG_STAMP(l * 8 + 7);
    }
    if (s_dead) {  // a bounded wait ran out: report it, and do not leave while a copy may still land
        if (threadIdx.x == 0) *a.err = 1u;
        if (u.t == 0)
            for (unsigned k = 0; k < (unsigned)kFusedStages && k < blocks_done; ++k) {
                const unsigned pos = blocks_done - 1 - k;
                for (int spins = 0; spins < (1 << 20); ++spins) {
                    uint32_t done;
                    asm volatile(
                        "{.reg .pred p;\n\t"
                        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                        "selp.u32 %0, 1, 0, p;}"
                        : "=r"(done)
                        : "r"(dsmem_u32(my_full + pos % kFusedStages)), "r"((pos / kFusedStages) & 1u)
                        : "memory");
                    if (done) break;
                }
            }
        __syncthreads();
    }
    if (unit == 0) {
#pragma unroll
        for (int e = 0; e < EPL; e += 4)
            *reinterpret_cast<float4 *>(a.h_out + c0 + e) = make_float4(h[e], h[e + 1], h[e + 2], h[e + 3]);
    }
}

// Transposed copy of a matrix of `rows` x `cols` elements of `bytes` bytes each (1, 2 or 4).
template <typename T> __global__ void transpose_kernel(const T *__restrict__ in, T *__restrict__ out, int rows, int cols)
{
    __shared__ T tile[32][33];
    const int bx = blockIdx.x * 32, by = blockIdx.y * 32;
    for (int r = threadIdx.y; r < 32; r += blockDim.y)
        if (by + r < rows && bx + threadIdx.x < cols) tile[r][threadIdx.x] = in[(size_t)(by + r) * cols + bx + threadIdx.x];
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y)
        if (bx + r < cols && by + threadIdx.x < rows) out[(size_t)(bx + r) * rows + by + threadIdx.x] = tile[threadIdx.x][r];
}

}  // namespace stmoe_dev
