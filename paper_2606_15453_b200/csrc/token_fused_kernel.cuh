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
// (cp.async.bulk, one destination CTA, completion counted on an mbarrier) into a shared-memory ring of
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

constexpr int kFusedRows = 2;          // rows per block (four for some fp8 shapes, see fused_rows)
constexpr int kFusedStages = 4;        // ring stages per unit (blocks in flight) with one chunk per thread
// ring bytes: units * stages * 3 matrices * rows * (H * element bytes) = 512 threads * 16 B * 24
constexpr int kFusedRingBytes = kFfnThreads * 16 * 3 * kFusedRows * kFusedStages;
// dynamic shared memory: the ring, then H floats in which the CTA's units add up their outputs
__host__ __device__ inline int fused_smem_bytes(int H) { return kFusedRingBytes + H * 4; }
constexpr int kFusedMaxUnits = 8;      // units per CTA (TPR >= 64)
constexpr float kFixScale = 1099511627776.0f;            // 2^40
constexpr float kFixInv = 9.094947017729282379150390625e-13f;  // 2^-40 (exact in fp32)

// Which shapes the kernel covers: a unit must be 2..16 whole warps (with one chunk per thread).
__host__ __device__ inline bool fused_shape_ok(int H, int epl)
{
    const int tpr = H / epl;
    return H % epl == 0 && H <= 4096 && (tpr == 64 || tpr == 128 || tpr == 256 || tpr == 512);
}
// Chunks per thread: two where the unit then still has two whole warps, the registers allow it
// (not the 16-column fp8 layout) and every unit still gets at least six row blocks of the routed
// experts per layer: two chunks halve the per-block bookkeeping per byte but double the number
// of units, and with few blocks per unit the one-block difference between units shows at the
// layer's closing barrier (measured: Qwen3-30B shape, 5.2 blocks per unit, 25.8 us per layer with
// two chunks against 24.0 with one; DeepSeek-V2-Lite shape, 7.2 blocks, 30.7 against 32.2).
#ifndef STMOE_FUSED_MAX_CHUNKS
#define STMOE_FUSED_MAX_CHUNKS 2
#endif
__host__ __device__ inline int fused_chunks(int H, int epl, int I, int K, int n_ctas)
{
    if (STMOE_FUSED_MAX_CHUNKS < 2 || epl >= 16 || H / epl < 128) return 1;
    const long long units = (long long)(n_ctas - 1) * (kFfnThreads / (H / (epl * 2)));
    const long long blocks = (long long)K * ((I + kFusedRows - 1) / kFusedRows);
    return blocks >= 6 * units ? 2 : 1;
}

// Rows per block: four for fp8 stacks with enough row blocks per unit (the same test as for a second
// chunk, which their 16-column layout has no registers for).  A block's cost beside its bytes is a
// serial chain (shared-memory reads, the unit's reduction with its barrier, the exponential, the
// exchange of the activations); with four rows the chain is paid once per 48 KB instead of 24 KB.
__host__ __device__ inline int fused_rows(int H, int epl, int I, int K, int n_ctas, int chunks)
{
    if (epl < 16 || chunks != 1) return kFusedRows;
    const long long units = (long long)(n_ctas - 1) * (kFfnThreads / (H / epl));
    const long long blocks = (long long)K * ((I + 3) / 4);
    return blocks >= 6 * units ? 4 : kFusedRows;
}

constexpr int kRedStride = 128;  // floats of one exchange buffer of a unit: up to 16 warps x 8 values
struct UnitCtx {
    int tpr, grp, t, wig, nwg, lane, bar_id;
    float *red;      // [2][kRedStride] this unit's exchange buffers
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
    float *buf = u.red + u.par * kRedStride;
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
    float *buf = u.red + u.par * kRedStride;
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
    float *buf = u.red + u.par * kRedStride;
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

// Sums of eight values over the unit, the same way: three folding exchanges leave every lane with
// one value's sum over eight lanes, two more finish the warp (9 shuffles); lane 4 i holds value i.
__device__ __forceinline__ void unit_sum8(UnitCtx &u, float (&v)[8])
{
    const bool b16 = u.lane & 16, b8 = u.lane & 8, b4 = u.lane & 4;
    float k[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        k[i] = b16 ? v[4 + i] : v[i];
        const float s = b16 ? v[i] : v[4 + i];
        k[i] += __shfl_xor_sync(kFull, s, 16);
    }
    float k2[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        k2[i] = b8 ? k[2 + i] : k[i];
        const float s = b8 ? k[i] : k[2 + i];
        k2[i] += __shfl_xor_sync(kFull, s, 8);
    }
    float kk = b4 ? k2[1] : k2[0];
    kk += __shfl_xor_sync(kFull, b4 ? k2[0] : k2[1], 4);
    kk += __shfl_xor_sync(kFull, kk, 2);
    kk += __shfl_xor_sync(kFull, kk, 1);
    float *buf = u.red + u.par * kRedStride;
    u.par ^= 1;
    if ((u.lane & 3) == 0) buf[u.wig * 8 + (u.lane >> 2)] = kk;
    unit_sync(u);
    // slot = warp * 8 + value: lane i adds the slots i, i + 32, ..., lanes of equal i % 8 are folded
    const int n = u.nwg * 8;
    float t = 0.f;
    for (int i = u.lane; i < n; i += kWarp) t += buf[i];
    t += __shfl_xor_sync(kFull, t, 8);
    t += __shfl_xor_sync(kFull, t, 16);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __shfl_sync(kFull, t, i);
}

// Grid barrier with one arrival and one poller per CTA (the units of a CTA meet at a CTA barrier
// first: with several hundred units on the GPU, per-unit arrivals and pollers on one counter cost
// several microseconds per barrier).
// The CTA barrier of the threads that take part in the layer loop: all 512 of a streaming CTA, the
// first 256 of the service CTA (its last warp runs the predictor on its own, the rest idle).
struct CtaBar {
    int id, width;
    __device__ __forceinline__ void sync() const { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(width) : "memory"); }
};
__device__ __forceinline__ void cta_arrive(const CtaBar &cb, unsigned *counter)
{
    cb.sync();  // orders every thread's writes before the release below
    if (threadIdx.x == 0) asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(counter), "r"(1u) : "memory");
}
__device__ __forceinline__ void cta_wait(const CtaBar &cb, unsigned *counter, unsigned *err, unsigned target,
                                         volatile int *s_dead, int poll_limit)
{
    if (threadIdx.x == 0 && !*s_dead) {
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
    cb.sync();
}

// The row blocks a unit streams in one layer.  The blocks of a list of entries form one index
// space (bpe = ceil(I / R) blocks per entry); a unit owns a contiguous range of the shared
// experts' space and one of the routed experts' space, each equal to within one block for all
// units.  Block q of the unit's layer sequence: q < nq_s is global block first_s + q of the shared
// experts, the others are global block first_r + q - nq_s of the routed ones; global block g is
// rows [bi*R, bi*R + nrows) of entry g / bpe, bi = g % bpe.
struct FusedPlan {
    int rows, R, bpe, first_s, nq_s, first_r, nq_r;  // R: rows per block
    __device__ __forceinline__ int nq() const { return nq_s + nq_r; }
    __device__ __forceinline__ int nrows(int bi) const { return min(R, rows - bi * R); }
};

// Walks the blocks of a unit's layer sequence without a division: next rows of the entry, next
// entry, next segment (shared -> routed).
struct FusedCursor {
    bool sh;
    int entry, bi;
    __device__ __forceinline__ void start(const FusedPlan &pl, bool shared_seg)
    {
        sh = shared_seg;
        const int g = shared_seg ? pl.first_s : pl.first_r;
        entry = g / pl.bpe, bi = g - entry * pl.bpe;
    }
    __device__ __forceinline__ void next(const FusedPlan &pl)
    {
        if (++bi == pl.bpe) bi = 0, ++entry;
    }
};

__device__ __forceinline__ size_t fused_image_index(const TokenArgs &a, int layer, bool shared, int entry, const int *s_ids)
{
    return shared ? (size_t)a.L * a.E + (size_t)layer * a.n_shared + entry : (size_t)layer * a.E + s_ids[entry];
}

// The unit's first thread: bulk copies of one block (rows [i0, i0+nrows) of the three matrices of
// image idx) into a ring stage.
template <int DT, int R>
__device__ __forceinline__ void fused_issue(const FusedArgs &fa, size_t idx, int i0, int nrows, uint8_t *stage, uint64_t *full)
{
    constexpr int BYTES = Fmt<DT>::kBytes;
    const TokenArgs &a = fa.t;
    const size_t row_bytes = (size_t)a.H * BYTES;
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

// Bounded wait for a stage's copies: the hardware suspends the thread inside try_wait (up to the
// hint, in nanoseconds), so a waiting unit issues few instructions beside a working one.
__device__ __forceinline__ bool fused_wait(uint64_t *bar, uint32_t parity, volatile int *dead, int spin_limit = 1 << 22)
{
    for (int spins = 0; spins < spin_limit; ++spins) {
        uint32_t ok;
        asm volatile(
            "{.reg .pred p;\n\t"
#ifdef STMOE_FUSED_WAIT_HINT
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
#else
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
#endif
            "selp.u32 %0, 1, 0, p;}"
            : "=r"(ok)
            : "r"(dsmem_u32(bar)), "r"(parity), "r"(2000u)
            : "memory");
        if (ok) return true;
        if ((spins & 15) == 15 && *dead) return false;
    }
    *dead = 1;
    return false;
}

// Sixteen e4m3 weights (one 16-byte chunk) times sixteen f16 activations held as eight pairs:
// exact e4m3 -> f16 conversions two at a time, f16 pair FMAs on two independent accumulators, the
// four partial sums added in fp32.
__device__ __forceinline__ float dot_e4m3_f16(const uint4 &w4, const uint32_t (&hx)[8])
{
    const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
    __half2 acc0 = __float2half2_rn(0.f), acc1 = acc0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t lo, hi;  // weights 4i, 4i+1 and 4i+2, 4i+3 as f16 pairs
        asm("{.reg .b16 a, b;\n\t"
            "mov.b32 {a, b}, %2;\n\t"
            "cvt.rn.f16x2.e4m3x2 %0, a;\n\t"
            "cvt.rn.f16x2.e4m3x2 %1, b;}"
            : "=r"(lo), "=r"(hi)
            : "r"(w[i]));
        acc0 = __hfma2(*reinterpret_cast<const __half2 *>(&lo), *reinterpret_cast<const __half2 *>(&hx[2 * i]), acc0);
        acc1 = __hfma2(*reinterpret_cast<const __half2 *>(&hi), *reinterpret_cast<const __half2 *>(&hx[2 * i + 1]), acc1);
    }
    const float2 a = __half22float2(acc0), b = __half22float2(acc1);
    return (a.x + a.y) + (b.x + b.y);
}

// CH: 16-byte chunks of a row a thread owns (chunk j = columns [(t + j*TPR)*EPL, +EPL)).  Two
// chunks halve the per-block bookkeeping (waits, reductions, barriers) per byte, which is what
// bounds the kernel once the copies keep HBM busy; they need twice the registers for the
// thread's columns of h and of the output, which the 16-column fp8 layout does not have.
template <int DT, int RDT, int CH, int R = kFusedRows>
__global__ void __launch_bounds__(kFfnThreads, 1) decode_token_fused_kernel(FusedArgs fa)
{
    constexpr int EPL = Fmt<DT>::kEpl, BYTES = Fmt<DT>::kBytes;
    // The ring is 192 KB per CTA whatever the unit size: a CTA of two-chunk threads has twice the
    // units, each with half the stages (the bytes in flight per SM are the same).
    constexpr int NS = kFusedStages * kFusedRows / (CH * R);
    constexpr int EPLR = Fmt<RDT>::kEpl, NRL = EPL / EPLR;  // router loads per chunk and row
    static_assert((R == 2 || R == 4) && CH * R <= 4, "the ring holds at least two stages per unit");
    const TokenArgs &a = fa.t;
    const int L = a.L, E = a.E, K = a.K, H = a.H, I = a.I;
    __shared__ __align__(16) float s_red[kFusedMaxUnits][2 * kRedStride];
    __shared__ uint32_t s_key[kMaxExperts];
    __shared__ float s_tk[3][8];   // top-K: per-warp maxima, sums, selected sums
    __shared__ int s_cnt[8];       // top-K: selected experts per warp
    __shared__ int s_ids[kMaxTopK];
    __shared__ float s_w[kMaxTopK];
    __shared__ float s_pick[2];
    __shared__ int s_prev[kMaxTopK];
    __shared__ int s_dead, s_ready;  // s_ready: layers whose routing the service CTA has recorded
    __shared__ __align__(8) uint64_t s_full[kFusedMaxUnits][kFusedStages];
    extern __shared__ __align__(128) uint8_t ring[];  // [unit][stage][gate rows | up rows | down^T rows], then H floats

    UnitCtx u;
    u.tpr = H / (EPL * CH);
    u.grp = threadIdx.x / u.tpr, u.t = threadIdx.x % u.tpr;
    u.wig = u.t / kWarp, u.nwg = u.tpr / kWarp, u.lane = threadIdx.x % kWarp;
    u.bar_id = 1 + u.grp;
    u.red = s_red[u.grp], u.par = 0;
    const int ng = kFfnThreads / u.tpr;
    const bool service = blockIdx.x == gridDim.x - 1;
    const int n_stream = (gridDim.x - 1) * ng;
    // The service CTA's last warp runs the predictor on its own, layer after layer, from the
    // routing its first 256 threads record (whole units when a unit has at most 256 threads); the
    // threads between idle.  The predictor then never holds up a grid barrier.
    const bool async_pred = service && u.tpr <= 256;
    const CtaBar cb{async_pred ? 13 : 0, async_pred ? 256 : kFfnThreads};
    const int unit = blockIdx.x * ng + u.grp;
    const int n_units = async_pred ? n_stream + 256 / u.tpr : gridDim.x * ng;  // who router rows are dealt to
    if (threadIdx.x == 0) {
        s_dead = 0, s_ready = 0;
        for (int i = 0; i < kFusedMaxUnits * kFusedStages; ++i) dmbar_init(&s_full[0][0] + i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    unsigned target = 0;
    const size_t row_bytes = (size_t)H * BYTES, stage_bytes = 3 * R * row_bytes;
    uint8_t *my_ring = ring + (size_t)u.grp * NS * stage_bytes;
    float *ysum = reinterpret_cast<float *>(ring + kFusedRingBytes);
    uint64_t *my_full = s_full[u.grp];

    // this thread's columns of the hidden state, carried in registers through all layers
    int c0[CH];
    float h[CH][EPL], y[CH][EPL];
#pragma unroll
    for (int j = 0; j < CH; ++j) {
        c0[j] = (u.t + j * u.tpr) * EPL;
#pragma unroll
        for (int e = 0; e < EPL; e += 4) {
            const float4 v = ld_f4(a.h_in + c0[j] + e);
            h[j][e] = v.x, h[j][e + 1] = v.y, h[j][e + 2] = v.z, h[j][e + 3] = v.w;
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) y[j][e] = 0.f;
    }

    // The service CTA keeps the predictor's tables (CCT of every layer pair, history table, the
    // predicted set, the step counter) in its unused ring for the whole launch and writes them back
    // at the end: with the other SMs streaming at full rate a dependent access to global memory
    // costs two to three microseconds, and Algorithms 2 and 3 are chains of such accesses (measured:
    // 17-38 us per layer from global memory, which made this CTA the last to arrive at every barrier).
    TokenArgs ap = a;
    const size_t cct_bytes = (size_t)(L > 1 ? L - 1 : 0) * E * K, ht_bytes = (size_t)L * K * 2;
    const size_t cct_pad = (cct_bytes + 15) / 16 * 16, ht_pad = (ht_bytes + 15) / 16 * 16;
    const bool tables_staged = service && 2 * cct_pad + ht_pad + 64 <= (size_t)kFusedRingBytes;
    auto copy_bytes = [&](uint8_t *dst, const uint8_t *src, size_t n) {
        for (size_t i = threadIdx.x; i < n; i += kFfnThreads) dst[i] = src[i];
    };
    if (tables_staged) {
        uint8_t *sm = ring;
        copy_bytes(sm, a.pst.cct_id, cct_bytes);
        copy_bytes(sm + cct_pad, a.pst.cct_conf, cct_bytes);
        copy_bytes(sm + 2 * cct_pad, reinterpret_cast<const uint8_t *>(a.pst.HT), ht_bytes);
        copy_bytes(sm + 2 * cct_pad + ht_pad, reinterpret_cast<const uint8_t *>(a.pst.pred_mask), 32);
        copy_bytes(sm + 2 * cct_pad + ht_pad + 32, reinterpret_cast<const uint8_t *>(a.pst.pred_valid), 4);
        copy_bytes(sm + 2 * cct_pad + ht_pad + 48, reinterpret_cast<const uint8_t *>(a.pst.t), 8);
        ap.pst.cct_id = sm, ap.pst.cct_conf = sm + cct_pad;
        ap.pst.HT = reinterpret_cast<int16_t *>(sm + 2 * cct_pad);
        ap.pst.pred_mask = reinterpret_cast<uint32_t *>(sm + 2 * cct_pad + ht_pad);
        ap.pst.pred_valid = reinterpret_cast<uint32_t *>(sm + 2 * cct_pad + ht_pad + 32);
        ap.pst.t = reinterpret_cast<long long *>(sm + 2 * cct_pad + ht_pad + 48);
    }
    int *s_hist = reinterpret_cast<int *>(ring + (tables_staged ? 2 * cct_pad + ht_pad + 64 : 0));  // [L][K], service CTA
    __syncthreads();
    if (async_pred && threadIdx.x >= kFfnThreads - kWarp) {
        for (int l = 0; l < L; ++l) {
            int spins = 0;
            while (*(volatile int *)&s_ready <= l && !*(volatile int *)&s_dead) {
                if (++spins > (1 << 24)) {
                    s_dead = 1;
                    break;
                }
                __nanosleep(64);
            }
            if (*(volatile int *)&s_ready <= l) break;  // gave up: the error word is set at the end
            __syncwarp();
            predictor_step_group(ap, l, s_hist + (size_t)l * K, s_hist + (size_t)(l > 0 ? l - 1 : 0) * K, 0, 1, u.lane);
        }
    }
    const bool in_loop = !(async_pred && threadIdx.x >= 256);

    FusedPlan pl;
    pl.rows = I, pl.R = R, pl.bpe = (I + R - 1) / R;
    {
        const long long all_s = (long long)a.n_shared * pl.bpe, all_r = (long long)K * pl.bpe;
        pl.first_s = service ? 0 : (int)(all_s * unit / n_stream);
        pl.nq_s = service ? 0 : (int)(all_s * (unit + 1) / n_stream) - pl.first_s;
        if (all_s > 0 && all_r >= n_stream) {
            // both kinds together are dealt evenly (to within one block per unit, not one of each
            // kind): a unit with one shared block more takes one routed block less.  The routed
            // ranges stay contiguous: unit u starts where the units before it end.
            const long long all = all_s + all_r;
            const long long t0 = all * unit / n_stream, t1 = all * (unit + 1) / n_stream;
            pl.first_r = service ? 0 : (int)(t0 - pl.first_s);
            pl.nq_r = service ? 0 : (int)(t1 - t0) - pl.nq_s;
        } else {
            pl.first_r = service ? 0 : (int)(all_r * unit / n_stream);
            pl.nq_r = service ? 0 : (int)(all_r * (unit + 1) / n_stream) - pl.first_r;
        }
    }
    const int nq = pl.nq();
    // Ring position: `done` = blocks the unit has consumed since the start of the launch (stage =
    // count % NS, phase = count / NS).  The copies run up to NS blocks ahead and do not stop at a
    // layer's end: the next layer's shared experts are known, its routed experts only after its
    // top-K.  What is issued next is the first thread's business alone.
    unsigned done = 0, issued = 0;
    int iss_layer = 0, iss_seq = 0;
    FusedCursor iss;
    iss.start(pl, pl.nq_s > 0);

    for (int l = 0; in_loop && l < L; ++l) {
        // ---- RMSNorm factor (every unit, same bits) -------------------------------------------
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < CH; ++j)
#pragma unroll
            for (int e = 0; e < EPL; ++e) ss = fmaf(h[j][e], h[j][e], ss);
        ss = unit_sum(u, ss);
        const float inv = 1.0f / sqrtf(ss / (float)H + a.eps);
        // fp8 stacks: the gate/up dot products run on f16 pairs (an e4m3 weight is exact in f16, and
        // converting it on to fp32 costs more issue slots than the FMA it feeds).  The normalised
        // hidden state is at most sqrt(H) <= 64 in magnitude, so x / 8 times a weight (<= 448), summed
        // over the eight products a lane adds up in f16, stays below 28672: no overflow; the partial
        // sums go to fp32 before they are added across lanes.
        uint32_t hx[DT == 2 ? EPL / 2 : 1];
        if (DT == 2) {
#pragma unroll
            for (int e2 = 0; e2 < EPL / 2; ++e2) {
                const __half2 p = __floats2half2_rn(h[0][2 * e2] * inv * 0.125f, h[0][2 * e2 + 1] * inv * 0.125f);
                hx[e2] = *reinterpret_cast<const uint32_t *>(&p);
            }
        }

        // ---- router rows dealt over the units ------------------------------------------------
        for (int jr = unit; jr < E; jr += n_units) {
            const uint8_t *row = a.router + ((size_t)l * E + jr) * H * Fmt<RDT>::kBytes;
            float p = 0.f;
#pragma unroll
            for (int j = 0; j < CH; ++j)
#pragma unroll
                for (int q = 0; q < NRL; ++q) {
                    float wf[EPLR];
                    Fmt<RDT>::unpack(ld_stream16(row + (size_t)c0[j] * Fmt<RDT>::kBytes + q * 16), wf);
#pragma unroll
                    for (int e = 0; e < EPLR; ++e) p = fmaf(wf[e], h[j][q * EPLR + e], p);
                }
            p = unit_sum(u, p);
            if (u.t == 0) fa.zpart[(size_t)l * E + jr] = p;
        }
        target += gridDim.x;
        cta_arrive(cb, a.barrier);

        // ---- softmax / top-K once the logits have arrived: the CTA's first 256 threads, thread j
        // owns expert j (rank counting: no dependent rounds); the other threads wait at the CTA
        // barrier.  Every unit calls this once per layer, at the block where it first needs routing.
        bool routed_known = false;
        auto route = [&]() {
            cta_wait(cb, a.barrier, a.err, target, &s_dead, fa.poll_limit);
            if (threadIdx.x < 256) {
                auto sync256 = []() { asm volatile("bar.sync 14, 256;" ::: "memory"); };
                const int j = threadIdx.x, wj = j / kWarp;
                const float z = j < E ? __ldcg(fa.zpart + (size_t)l * E + j) * inv : -INFINITY;
                const uint32_t key = j < E ? float_key(z) : 0u;
                s_key[j] = key;
                const float wm = warp_max(z);
                if (u.lane == 0) s_tk[0][wj] = wm;
                sync256();
                float zmax = s_tk[0][0];
#pragma unroll
                for (int w = 1; w < 8; ++w) zmax = fmaxf(zmax, s_tk[0][w]);
                const float ex = j < E ? expf(z - zmax) : 0.f;
                const float ws = warp_sum(ex);
                if (u.lane == 0) s_tk[1][wj] = ws;
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
                if (u.lane == 0) s_cnt[wj] = __popc(msk), s_tk[2][wj] = wsel;
                sync256();
                float sum = 0.f, selsum = 0.f;
                int pos = __popc(msk & ((1u << u.lane) - 1u));
#pragma unroll
                for (int w = 0; w < 8; ++w) {
                    sum += s_tk[1][w], selsum += s_tk[2][w];
                    if (w < wj) pos += s_cnt[w];
                }
                if (sel) s_ids[pos] = j, s_w[pos] = ex / (a.renorm ? selsum : sum);
            }
            cb.sync();
            if (service) {  // the step's outputs
                if (threadIdx.x < K) {
                    const int id = s_ids[threadIdx.x];
                    if (async_pred) s_hist[(size_t)l * K + threadIdx.x] = id;
                    a.ids_all[(size_t)l * a.Bmax * K + threadIdx.x] = id;
                    if (a.ids_out) a.ids_out[(size_t)l * K + threadIdx.x] = id;
                    if (a.w_out) a.w_out[(size_t)l * K + threadIdx.x] = s_w[threadIdx.x];
                }
                if (threadIdx.x == 0) {
                    const float gap = K < E ? s_pick[0] - s_pick[1] : INFINITY;
                    const uint32_t f = gap < 1e-4f ? 1u : 0u;
                    if (a.flags_out) a.flags_out[l] = f;
                    if (f) atomicAdd(a.pst.stats + 4, 1ull);
                }
                if (async_pred && threadIdx.x < kWarp) {  // K <= 32: the ids were written by this warp
                    __syncwarp();
                    if (threadIdx.x == 0) {
                        __threadfence_block();
                        *(volatile int *)&s_ready = l + 1;
                    }
                }
            }
            routed_known = true;
        };

        // Keep the ring full (the unit's first thread only).
        auto top_up = [&]() {
            while (nq > 0 && issued - done < (unsigned)NS && iss_layer < L) {
                // a routed block of a later layer, or of this one before its top-K: not known yet
                if (!iss.sh && (iss_layer != l || !routed_known)) break;
                const unsigned st = issued % NS;
                fused_issue<DT, R>(fa, fused_image_index(a, iss_layer, iss.sh, iss.entry, s_ids), iss.bi * R,
                                pl.nrows(iss.bi), my_ring + st * stage_bytes, my_full + st);
                ++issued, ++iss_seq;
                iss.next(pl);
                if (iss_seq == pl.nq_s && pl.nq_r > 0) iss.start(pl, false);
                if (iss_seq == nq) iss_seq = 0, ++iss_layer, iss.start(pl, pl.nq_s > 0);
            }
        };

        // ---- the layer's row blocks: shared experts first (they need no routing) ---------------
        float ye[DT == 2 ? EPL : 1];  // fp8 (CH = 1): per-expert sums before the output-channel scales
        if (DT == 2) {
#pragma unroll
            for (int e = 0; e < EPL; ++e) ye[e] = 0.f;
        }
        FusedCursor cu;
        cu.start(pl, pl.nq_s > 0);
        for (int q = 0; q < nq; ++q) {
            // the block the first thread would issue now is a routed one: time for the top-K
            if (!routed_known && q + NS - 1 >= pl.nq_s) route();
            if (u.t == 0) top_up();
            const unsigned st = done % NS;
            fused_wait(my_full + st, (done / NS) & 1u, &s_dead);
            if (q == pl.nq_s && q > 0) cu.start(pl, false);
            const int i0 = cu.bi * R, nrows = pl.nrows(cu.bi);
            const uint8_t *stage = my_ring + st * stage_bytes;
            float v[2 * R];
#pragma unroll
            for (int i = 0; i < 2 * R; ++i) v[i] = 0.f;
            uint4 wd[R][CH];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    const size_t off = (size_t)r * row_bytes + (size_t)c0[j] * BYTES;
                    uint4 wg4 = make_uint4(0u, 0u, 0u, 0u), wu4 = wg4;
                    wd[r][j] = wg4;
                    if (r < nrows) {
                        wg4 = *reinterpret_cast<const uint4 *>(stage + off);
                        wu4 = *reinterpret_cast<const uint4 *>(stage + R * row_bytes + off);
                        wd[r][j] = *reinterpret_cast<const uint4 *>(stage + 2 * R * row_bytes + off);
                    }
                    if constexpr (DT == 2) {
                        v[2 * r] += dot_e4m3_f16(wg4, hx);
                        v[2 * r + 1] += dot_e4m3_f16(wu4, hx);
                    } else {
                        float wg[EPL], wu[EPL];
                        Fmt<DT>::unpack(wg4, wg);
                        Fmt<DT>::unpack(wu4, wu);
#pragma unroll
                        for (int e = 0; e < EPL; ++e) {
                            v[2 * r] = fmaf(wg[e], h[j][e], v[2 * r]);
                            v[2 * r + 1] = fmaf(wu[e], h[j][e], v[2 * r + 1]);
                        }
                    }
                }
            // past the reduction's barrier every thread has read the stage: it may be refilled
            if constexpr (R == 2)
                unit_sum4(u, v);
            else
                unit_sum8(u, v);
            ++done;
            const float wgt = cu.sh ? 1.f : s_w[cu.entry];
            const uint16_t *sc = nullptr;
            if (DT == 2)
                sc = reinterpret_cast<const uint16_t *>(a.store + fused_image_index(a, l, cu.sh, cu.entry, s_ids) * a.img_bytes +
                                                        image_scales(H, I, BYTES));
            // lane i evaluates row i % R; an exchange inside each group of R lanes gives every lane all
            const int r_mine = u.lane & (R - 1);
            const float vs = DT == 2 ? 8.f : inv;  // fp8: the f16 pairs carry inv / 8 already
            float gsel = v[0], usel = v[1];
#pragma unroll
            for (int r = 1; r < R; ++r)
                if (r_mine == r) gsel = v[2 * r], usel = v[2 * r + 1];
            float gv = gsel * vs, uv = usel * vs;
            if (DT == 2 && i0 + r_mine < I) {
                gv *= bf16_to_f32(sc[i0 + r_mine]);
                uv *= bf16_to_f32(sc[I + i0 + r_mine]);
            }
            const float act_mine = gv / (1.f + expf(-gv)) * uv;  // rows past the end: zero weights, act = 0
            float acts[R];
            if constexpr (R == 2) {
                const float act_other = __shfl_xor_sync(kFull, act_mine, 1);
                acts[0] = r_mine ? act_other : act_mine, acts[1] = r_mine ? act_mine : act_other;
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r) acts[r] = __shfl_sync(kFull, act_mine, (u.lane & ~(R - 1)) | r);
            }
            if constexpr (DT == 2) {
                // fp8: the block's rows are combined in f16 pairs before they meet the fp32 sums.  The
                // activations are scaled by the block's largest magnitude, so a product is at most 448
                // and a column's sum over the block's rows at most 448 R: no overflow whatever the
                // activations are; the scale goes back in with the one fp32 FMA per column.
                float amax = fabsf(acts[0]);
#pragma unroll
                for (int r = 1; r < R; ++r) amax = fmaxf(amax, fabsf(acts[r]));
                const float rs = amax > 0.f ? 1.f / amax : 0.f;
                __half2 a2[R];
#pragma unroll
                for (int r = 0; r < R; ++r) a2[r] = __float2half2_rn(acts[r] * rs);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    __half2 plo = __float2half2_rn(0.f), phi = plo;
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const uint32_t w = i == 0 ? wd[r][0].x : i == 1 ? wd[r][0].y : i == 2 ? wd[r][0].z : wd[r][0].w;
                        uint32_t lo, hi;  // weights 4i, 4i+1 and 4i+2, 4i+3 of the row as f16 pairs
                        asm("{.reg .b16 a, b;\n\t"
                            "mov.b32 {a, b}, %2;\n\t"
                            "cvt.rn.f16x2.e4m3x2 %0, a;\n\t"
                            "cvt.rn.f16x2.e4m3x2 %1, b;}"
                            : "=r"(lo), "=r"(hi)
                            : "r"(w));
                        plo = __hfma2(*reinterpret_cast<const __half2 *>(&lo), a2[r], plo);
                        phi = __hfma2(*reinterpret_cast<const __half2 *>(&hi), a2[r], phi);
                    }
                    const float2 fl = __half22float2(plo), fh = __half22float2(phi);
                    ye[4 * i] = fmaf(amax, fl.x, ye[4 * i]);
                    ye[4 * i + 1] = fmaf(amax, fl.y, ye[4 * i + 1]);
                    ye[4 * i + 2] = fmaf(amax, fh.x, ye[4 * i + 2]);
                    ye[4 * i + 3] = fmaf(amax, fh.y, ye[4 * i + 3]);
                }
            } else {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float act = acts[r] * wgt;
#pragma unroll
                    for (int j = 0; j < CH; ++j) {
                        float wf[EPL];
                        Fmt<DT>::unpack(wd[r][j], wf);
#pragma unroll
                        for (int e = 0; e < EPL; ++e) y[j][e] = fmaf(act, wf[e], y[j][e]);
                    }
                }
            }
            if (DT == 2 && (cu.bi == pl.bpe - 1 || q == pl.nq_s - 1 || q == nq - 1)) {  // done with this expert
#pragma unroll
                for (int e = 0; e < EPL; ++e) {
                    y[0][e] = fmaf(wgt * bf16_to_f32(sc[2 * I + c0[0] + e]), ye[e], y[0][e]);
                    ye[e] = 0.f;
                }
            }
            cu.next(pl);
        }
        if (!routed_known) route();  // units without a routed block (the service CTA among them)

        if (!service) {
            // the CTA's units add up in shared memory, unit by unit, then one exact atomic per column
            for (int g = 0; g < ng; ++g) {
                if (u.grp == g) {
#pragma unroll
                    for (int j = 0; j < CH; ++j)
#pragma unroll
                        for (int e = 0; e < EPL; e += 4) {
                            float4 *p = reinterpret_cast<float4 *>(ysum + c0[j] + e);
                            float4 sv = make_float4(y[j][e], y[j][e + 1], y[j][e + 2], y[j][e + 3]);
                            if (g > 0) {
                                const float4 o = *p;
                                sv.x += o.x, sv.y += o.y, sv.z += o.z, sv.w += o.w;
                            }
                            *p = sv;
                        }
                }
                cb.sync();
            }
#pragma unroll
            for (int j = 0; j < CH; ++j)
#pragma unroll
                for (int e = 0; e < EPL; ++e) y[j][e] = 0.f;
            for (int c = threadIdx.x; c < H; c += kFfnThreads) {
                const long long fx = __float2ll_rn(ysum[c] * kFixScale);
                asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(fa.acc + (size_t)l * H + c), "l"(fx) : "memory");
            }
        } else if (!async_pred && threadIdx.x < kWarp) {
            // (units of 512 threads: no warp to spare, the predictor runs here, between the barriers)
            // one warp: spreading Algorithms 2 and 3 of a single sequence over eight warps measured
            // two to three times slower (the rows of one sequence are too few to split)
            predictor_step_group(ap, l, s_ids, s_prev, 0, 1, u.lane);
            if (u.lane < K) s_prev[u.lane] = s_ids[u.lane];
            __syncwarp();
        }

        // ---- h' = h + r * y, from the exact sums ----------------------------------------------
        target += gridDim.x;
        cta_arrive(cb, a.barrier);  // (its CTA barrier also orders the reads of ysum before the next layer's writes)
        // the next layer's shared experts start to arrive while the barrier completes (top_up stops at
        // that layer's routed blocks: iss_layer is past l by now)
        if (u.t == 0) top_up();
        cta_wait(cb, a.barrier, a.err, target, &s_dead, fa.poll_limit);
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            const unsigned long long *acc = fa.acc + (size_t)l * H + c0[j];
#pragma unroll
            for (int e = 0; e < EPL; e += 2) {
                const ulonglong2 v = __ldcg(reinterpret_cast<const ulonglong2 *>(acc + e));
                // one rounding (64-bit integer -> fp32), then an exact power of two: no fp64 arithmetic,
                // which this GPU executes at a small fraction of the fp32 rate
                h[j][e] = fmaf(a.residual_scale, __ll2float_rn((long long)v.x) * kFixInv, h[j][e]);
                h[j][e + 1] = fmaf(a.residual_scale, __ll2float_rn((long long)v.y) * kFixInv, h[j][e + 1]);
            }
        }
    }
    __syncthreads();  // the service CTA's predictor warp and its other threads meet again here
    if (tables_staged) {
        const uint8_t *sm = ring;
        copy_bytes(a.pst.cct_id, sm, cct_bytes);
        copy_bytes(a.pst.cct_conf, sm + cct_pad, cct_bytes);
        copy_bytes(reinterpret_cast<uint8_t *>(a.pst.HT), sm + 2 * cct_pad, ht_bytes);
        copy_bytes(reinterpret_cast<uint8_t *>(a.pst.pred_mask), sm + 2 * cct_pad + ht_pad, 32);
        copy_bytes(reinterpret_cast<uint8_t *>(a.pst.pred_valid), sm + 2 * cct_pad + ht_pad + 32, 4);
        copy_bytes(reinterpret_cast<uint8_t *>(a.pst.t), sm + 2 * cct_pad + ht_pad + 48, 8);
    }
    if (s_dead) {  // a bounded wait ran out: report it, and do not leave while a copy may still land
        if (threadIdx.x == 0) *a.err = 1u;
        if (u.t == 0)
            for (unsigned k = 0; k < (unsigned)NS && k < issued; ++k) {
                const unsigned pos = issued - 1 - k;
                for (int spins = 0; spins < (1 << 20); ++spins) {
                    uint32_t ok;
                    asm volatile(
                        "{.reg .pred p;\n\t"
                        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                        "selp.u32 %0, 1, 0, p;}"
                        : "=r"(ok)
                        : "r"(dsmem_u32(my_full + pos % NS)), "r"((pos / NS) & 1u)
                        : "memory");
                    if (ok) break;
                }
            }
        __syncthreads();
    }
    if (unit == 0) {
#pragma unroll
        for (int j = 0; j < CH; ++j)
#pragma unroll
            for (int e = 0; e < EPL; e += 4)
                *reinterpret_cast<float4 *>(a.h_out + c0[j] + e) = make_float4(h[j][e], h[j][e + 1], h[j][e + 2], h[j][e + 3]);
    }
}

// The bounded waits of the persistent kernels, run on barriers that nobody completes: two CTAs of
// 64 threads call the same helpers the kernels use, with a small poll limit; every wait gives up,
// raises the error word and returns.  which: 0 grid_barrier (token_kernel.cuh), 1 cta_wait
// (this file), 2 dmbar_wait (tensor-core kernels), 3 fused_wait (this file's copy ring), 4
// group_wait_counter (the tensor-core kernel's hand-over between its projections).
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(unsigned *counter, unsigned *err, int which, int limit)
{
    __shared__ int s_dead;
    __shared__ __align__(8) uint64_t s_bar;
    if (threadIdx.x == 0) {
        s_dead = 0;
        dmbar_init(&s_bar, 1);  // one arrival expected, none comes
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (which == 0) {
        unsigned target = 1;  // one more arrival than there are CTAs
        grid_barrier(counter, err, target, &s_dead, limit);
    } else if (which == 1) {
        const CtaBar cb{0, 64};
        cta_arrive(cb, counter);
        cta_wait(cb, counter, err, gridDim.x + 1, &s_dead, limit);
    } else if (which == 2) {
        if (!dmbar_wait(&s_bar, 0u, &s_dead, limit) && threadIdx.x == 0) *err = 1u;
    } else if (which == 3) {
        if (!fused_wait(&s_bar, 0u, &s_dead, limit) && threadIdx.x == 0) *err = 1u;
    } else {
        // a completion counter that stays one short (the grid barrier's counter: zero, nobody adds)
        if (threadIdx.x == 0 && !group_wait_counter(counter, 1u, &s_dead, limit)) *err = 1u;
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
