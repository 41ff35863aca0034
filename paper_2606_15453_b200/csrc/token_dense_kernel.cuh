// One decode step of a resident bf16 or fp8 stack with several sequences as a single persistent
// kernel whose expert FFN runs on the tensor cores (the batched counterpart of token_kernel.cuh).
//
// One 512-thread CTA per SM, launched cooperatively, walks the layers:
//   F   weighted sum + residual of the previous layer from its down-projection partial sums
//       (layer 0: the input), written as fp32 (router, residual) and as the gate/up operand (bf16,
//       or three e5m2 planes for fp8 stacks)
//                                                                          -> grid barrier
//   R   split-K router GEMV tasks over all warps of the grid               -> grid barrier
//   T   every CTA runs softmax / top-K / grouping (one work-list entry per expert) itself
//   GU  gate/up tiles on tcgen05: warp 0 feeds TMA, warp 1 issues MMAs, warps 2-5 read the
//       accumulators; the predictor (Algorithms 1-3) runs on the remaining warps of the last CTA
//   D   down-projection tiles the same way, with no grid barrier before them: a CTA that has
//       finished its gate/up tiles goes on, and the loads of an entry's down tiles wait for that
//       entry's gate/up tiles only (a counter per entry; gate/up tiles wait for nothing, so
//       every counter fills)                                                -> grid barrier
// The tensor-memory columns and the accumulator hand-off barriers are set up once and carried
// through all phases and layers; the stage ring is laid out anew for every GU and D phase (its
// stage size differs between the two, and every stage is empty at a phase boundary).  Data
// written with ordinary stores and then fetched by TMA from another SM (the gate/up operand of
// the hidden state, the gated activations) is fenced for the async proxy on both sides of the
// grid barrier in between.
#pragma once
#include "dense8_group.cuh"
#include "dense_group.cuh"
#include "token_kernel.cuh"

namespace stmoe_dev {

struct TokenDenseArgs {
    TokenArgs t;            // mt = 64; act/part/tile_done/blob unused
    int splits, seg;        // down projection: splits of the reduction dimension, columns per split
    int img_shared_base;    // image index of layer 0's first shared expert (= L * E)
    int dyn_bytes;          // dynamic shared memory of the launch
    void *xb;               // [64][H] bf16 (bf16 weights) or [3][64][H] e5m2 planes (fp8 weights)
    void *actb;             // [pairs + 64][I] bf16 or [3][pairs + 64][I] e5m2 planes
    float *part;            // [pairs][splits][H]
    const uint8_t *store;   // fp8: first expert image (for the row scales) and the image pitch
    unsigned long long img_bytes;
    unsigned *gu_done;      // [L][E + n_shared]: finished gate/up tiles x epilogue warps per work-list entry
};

// RDT: router weight type; WDT: expert weight type, 1 = bf16, 2 = fp8 e4m3 (operand formats of
// dense_group.cuh).
template <int RDT, int WDT>
__global__ void __launch_bounds__(kFfnThreads, 1)
decode_token_dense_kernel(const __grid_constant__ CUtensorMap map_gate, const __grid_constant__ CUtensorMap map_up,
                          const __grid_constant__ CUtensorMap map_down, const __grid_constant__ CUtensorMap map_x,
                          const __grid_constant__ CUtensorMap map_act, TokenDenseArgs d)
{
    constexpr int NW = kFfnThreads / kWarp;
    const TokenArgs &a = d.t;
    extern __shared__ __align__(16) int dyn[];  // work list | ids | prev ids | gate weights | stage ring
    __shared__ int s_scan[2 * (kMaxExperts + 1)];
    __shared__ float s_inv[kMaxBatch];
    constexpr int kTmemCols = WDT == 1 ? kGroupTmemCols : kGroup8TmemCols;
    __shared__ uint64_t full[kGroupMaxStages], empty[kGroupMaxStages], tfull[2], tempty[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_dead;
    const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
    const int L = a.L, B = a.B, E = a.E, K = a.K, H = a.H, I = a.I;
    const int KS = K + a.n_shared, pairs = B * KS, np = (B + 15) / 16 * 16;
    const int C = router_chunks<RDT>(H, B);

    WorkList wl;
    wl.n_groups = dyn, wl.g_expert = dyn + 4, wl.g_start = dyn + 4 + pairs, wl.g_count = dyn + 4 + 2 * pairs;
    wl.pair_token = dyn + 4 + 3 * pairs, wl.pair_slot = dyn + 4 + 4 * pairs;
    int *s_ids = dyn + 4 + 5 * pairs;
    int *s_prev = s_ids + B * K;
    float *s_w = reinterpret_cast<float *>(s_prev + B * K);
    const int list_bytes = (int)sizeof(int) * (4 + 5 * pairs + 3 * B * K);

    GroupRing r;
    r.dsm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dyn) + list_bytes + 1023) & ~(uintptr_t)1023);
    r.full = full, r.empty = empty, r.tfull = tfull, r.tempty = tempty, r.dead = &s_dead;
    const int ring_bytes = (int)(reinterpret_cast<uint8_t *>(dyn) + d.dyn_bytes - r.dsm);
    // the ring of one phase: as many stages of that projection's size as fit (the host checked that
    // one of the larger kind fits)
    auto ring_for = [&](int stage_bytes) {
        r.slot = stage_bytes;
        r.NS = min(kGroupMaxStages, ring_bytes / stage_bytes);
    };
    ring_for(max(group_stage_bytes<1, WDT>(np), group_stage_bytes<2, WDT>(np)));
    if (threadIdx.x == 0) {
        s_dead = r.NS < 1;  // cannot happen with the host's sizing; never run a ring without stages
        GroupRing all = r;
        all.NS = kGroupMaxStages;  // the barriers of every stage any phase's layout can have
        group_ring_init(all);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dsmem_u32(&s_tmem)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    r.tmem = s_tmem;

    unsigned target = 0;
    const bool lead = blockIdx.x == 0;
    const bool pred_cta = blockIdx.x == gridDim.x - 1;
    RingPos ppos, mpos;              // producer / MMA thread
    AccPos macc, eacc;               // accumulator hand-off state of the MMA thread / the epilogue threads
    int issued = 0;                  // loads issued in the current phase (producer)
    // Start of a GU or D phase: every stage of the ring is empty (the MMA thread consumed every
    // load), so the ring is laid out for this phase's stage size and both roles restart at stage 0;
    // the barriers keep their state, the roles their per-stage parities.
    auto ring_restart = [&](int stage_bytes) {
        ring_for(stage_bytes);
        ppos.s = 0, mpos.s = 0, issued = 0;
    };
    const size_t x_plane = (size_t)kDenseMaxTokens * H;
    auto store_x = [&](int i, float v) {  // the gate/up operand of element i of the hidden state
        if constexpr (WDT == 1)
            static_cast<__nv_bfloat16 *>(d.xb)[i] = __float2bfloat16_rn(v);
        else
            store_e5m2_planes(static_cast<uint8_t *>(d.xb), x_plane, (size_t)i, v);
    };
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gthreads = gridDim.x * blockDim.x;

    // arguments of the weighted sum that finishes layer lp
    auto finish_args = [&](int lp) {
        FfnArgs f{};
        f.part = d.part, f.w = s_w;
        f.h = lp == 0 ? a.h_in : a.hbuf + (size_t)lp * B * H;
        f.H = H, f.B = B, f.K = K, f.n_shared = a.n_shared, f.residual_scale = a.residual_scale;
        return f;
    };

    for (int l = 0; l < L && !s_dead; ++l) {
        const float *h = l == 0 ? a.h_in : a.hbuf + (size_t)l * B * H;

        // ---- F ---------------------------------------------------------------------------------
        if (l == 0) {
            for (int i = gtid; i < B * H; i += gthreads) store_x(i, h[i]);
            for (int i = gtid; i < L * (E + a.n_shared); i += gthreads) d.gu_done[i] = 0u;  // read after later barriers
        } else {
            const FfnArgs fp = finish_args(l - 1);
            float *hl = a.hbuf + (size_t)l * B * H;
            for (int i = gtid; i < B * H; i += gthreads) {
                const float v = finish_value(fp, i / H, i % H, d.splits);
                hl[i] = v;
                store_x(i, v);
            }
        }
        fence_async_proxy();
        grid_barrier(a.barrier, a.err, target, &s_dead);

        // ---- R ---------------------------------------------------------------------------------
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
        router_tasks<RDT, false>(ra, warp * gridDim.x + blockIdx.x, NW * gridDim.x, lane);
        grid_barrier(a.barrier, a.err, target, &s_dead);

        // ---- T ---------------------------------------------------------------------------------
        router_finalize<RDT>(ra, s_ids, s_scan, NW);
        __syncthreads();
        if (lead)
            for (int i = threadIdx.x; i < B * K; i += blockDim.x) a.ids_all[(size_t)l * a.Bmax * K + i] = s_ids[i];

        // ---- GU (+ the predictor on one warp of the last CTA) -----------------------------------
        GroupArgs g{};
        g.wl = wl, g.E = E, g.img_routed0 = l * E, g.img_shared0 = d.img_shared_base + l * a.n_shared;
        g.np = np, g.KS = KS, g.inv_rms = s_inv, g.part = d.part, g.err = a.err;
        g.store = d.store, g.img_bytes = d.img_bytes;
        if constexpr (WDT == 1)
            g.act = static_cast<__nv_bfloat16 *>(d.actb);
        else
            g.act8 = static_cast<uint8_t *>(d.actb), g.act_rows = pairs + kDenseMaxTokens;
        constexpr int kGuStage = group_kstage<2, WDT>();
        g.rows = I, g.kd = H, g.splits = 1, g.seg = (H + kGuStage - 1) / kGuStage * kGuStage;
        g.scale_off = 0, g.x_rows = kDenseMaxTokens;
        g.signal = d.gu_done + (size_t)l * (E + a.n_shared), g.ready = nullptr;
        ring_restart(group_stage_bytes<2, WDT>(np));
        if (warp == 0) {
            if (lane == 0) {
                fence_async_proxy();
                group_produce<2, WDT>(&map_gate, &map_up, &map_x, g, r, ppos, issued);
            }
        } else if (warp == 1) {
            if (lane == 0) group_mma<2, WDT>(g, r, mpos, macc);
        } else if (warp < 6) {
            group_epilogue<2, WDT>(g, r, eacc, warp % 4, lane);
        } else if (pred_cta) {  // the ten warps without a role in this phase
            predictor_step_group(a, l, s_ids, s_prev, warp - 6, NW - 6, lane);
        }

        // ---- D (every role moves on by itself) ----------------------------------------------------
        g.rows = H, g.kd = I, g.splits = d.splits, g.seg = d.seg;
        g.scale_off = 2 * I, g.x_rows = pairs + kDenseMaxTokens;
        g.ready = g.signal, g.signal = nullptr, g.ready_target = 4u * (unsigned)((I + kDenseRows - 1) / kDenseRows);
        // the MMAs have read every gate/up stage before the producer lays the ring out for this phase
        if (warp == 0 && lane == 0) group_wait_stages_free(r, ppos);
        ring_restart(group_stage_bytes<1, WDT>(np));
        if (warp == 0) {
            if (lane == 0) {
                fence_async_proxy();
                group_produce<1, WDT>(&map_down, &map_down, &map_act, g, r, ppos, issued);
            }
        } else if (warp == 1) {
            if (lane == 0) group_mma<1, WDT>(g, r, mpos, macc);
        } else if (warp < 6) {
            group_epilogue<1, WDT>(g, r, eacc, warp % 4, lane);
        }
        grid_barrier(a.barrier, a.err, target, &s_dead);
        // (after the barrier: the predictor warps of the last CTA read s_prev until they reach it)
        for (int i = threadIdx.x; i < B * K; i += blockDim.x) s_prev[i] = s_ids[i];
    }
    // the last layer's output
    if (!s_dead) {
        const FfnArgs fl = finish_args(L - 1);
        for (int i = gtid; i < B * H; i += gthreads) a.h_out[i] = finish_value(fl, i / H, i % H, d.splits);
    }
    if (warp == 0 && lane == 0) group_drain(r, ppos, issued);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && s_dead) *a.err = 1u;
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(r.tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace stmoe_dev
