// Grouped expert FFN on the tensor cores for fp8 (e4m3) expert weights.
//
// Same task structure as dense_group.cuh (one work-list entry per expert, a task = entry x 128
// weight rows x one split, persistent CTA per SM, weights as the MMA's M operand).  tcgen05 has no
// fp8 x 16-bit mode, and rounding the activations to fp8 would not fit the error bound, so the
// weights are widened on the way: TMA lands e4m3 boxes (128 rows x 128 columns, 16 KB) in a
// staging ring, eight converter warps turn each row into f16 pairs (e4m3 -> f16 is exact) and write
// them straight into tensor memory (tcgen05.st; a thread owns the row = TMEM lane of its warp's
// lane quarter), and the MMA runs f16 x f16 -> fp32 with its A operand from tensor memory and the
// f16 activations from shared memory.  A weight byte thus crosses shared memory twice (TMA write,
// converter read).  The per-output-channel scales belong to the weight rows = accumulator lanes and
// are applied in the epilogue.
//   warp 0       TMA producer: two weight boxes (gate and up of the same columns, or two
//                consecutive column boxes of the down matrix) + the activation boxes of a stage
//   warp 1       MMA issue (8 K=16 steps per box), tensor-memory owner
//   warps 2-5    epilogue (two accumulator buffers)
//   warps 6-13   converters, two per lane quarter: one weight box each
// Tensor memory: columns [0,256) two accumulator buffers, [256,512) two A buffers of 2 x 64 columns
// (a box = 128 reduction columns, two f16 per 32-bit column).  Every wait is bounded.
#pragma once
#include <cuda_fp16.h>

#include "dense_group.cuh"

namespace stmoe_dev {

constexpr int kGroup8Threads = 448;
constexpr int kGroup8BoxCols = 128;                                 // fp8 columns of a weight box
constexpr int kGroup8BoxBytes = kDenseRows * kGroup8BoxCols;        // 16 KB of e4m3
// reduction columns per stage: gate/up share one box position, the down projection takes two
template <int NMAT> __host__ __device__ constexpr int group8_kstage() { return NMAT == 2 ? kGroup8BoxCols : 2 * kGroup8BoxCols; }

struct Group8Args {
    GroupArgs g;                 // act/part as in GroupArgs (act unused), inv_rms, work list, sizes
    const uint8_t *store;        // first expert image of the stack
    unsigned long long img_bytes;
    __half *act16;               // gate/up out, down in: [pairs + 64][I]
    int scale_off;               // element offset of this projection's scales in the image's scale vector
};

// two weight boxes + one 64-column f16 activation box per 64 reduction columns
template <int NMAT> __host__ __device__ constexpr int group8_stage_bytes(int np)
{
    return 2 * kGroup8BoxBytes + (group8_kstage<NMAT>() / kDenseKStep) * group_act_bytes(np);
}
template <int NMAT> __host__ __device__ constexpr int group8_stages(int np)
{
    const int n = (kGroupSmemBytes - 1024) / group8_stage_bytes<NMAT>(np);
    return n < kGroupMaxStages ? n : kGroupMaxStages;
}
__host__ __device__ constexpr uint32_t umma_idesc_f16(int n)
{
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kDenseRows >> 4) << 24);  // f16 x f16 -> f32
}
// 16 e4m3 values -> 16 f16 values (two 16-byte chunks)
__device__ __forceinline__ void e4m3x16_to_f16(const uint4 &v, uint4 &lo, uint4 &hi)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        asm("{.reg .b16 a, b;\n\t"
            "mov.b32 {a, b}, %2;\n\t"
            "cvt.rn.f16x2.e4m3x2 %0, a;\n\t"
            "cvt.rn.f16x2.e4m3x2 %1, b;}"
            : "=r"(o[2 * i]), "=r"(o[2 * i + 1])
            : "r"(w[i]));
    lo = make_uint4(o[0], o[1], o[2], o[3]);
    hi = make_uint4(o[4], o[5], o[6], o[7]);
}

__device__ __forceinline__ void umma_f16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t b, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;}"
        :
        : "r"(tmem_d), "r"(tmem_a), "l"(b), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t (&v)[16])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                 :
                 : "r"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                   "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
                 : "memory");
}

// The stage ring of dense_group.cuh plus the hand-off barriers of the two A buffers in tensor memory.
struct Group8Ring {
    GroupRing r;  // r.tmem: base of 512 columns
    uint64_t *afull, *aempty;
};
struct Group8Pos {  // per role: ring position and the number of stages handled so far
    int s = 0;
    uint32_t ph = 0;
    int stage_no = 0;
};
constexpr int kGroup8ACols = 128;  // tensor-memory columns of one A buffer (two boxes)

__device__ __forceinline__ void group8_ring_init(const Group8Ring &q)
{
    for (int b = 0; b < 2; ++b) dmbar_init(&q.afull[b], 8), dmbar_init(&q.aempty[b], 1);
    group_ring_init(q.r);
}

// One thread: the TMA loads of this CTA's tasks.  NMAT = 2: gate and up; NMAT = 1: down.
template <int NMAT>
__device__ __forceinline__ void group8_produce(const CUtensorMap *map_w0, const CUtensorMap *map_w1,
                                               const CUtensorMap *map_x, const GroupArgs &a, const Group8Ring &q,
                                               Group8Pos &pos, int &issued)
{
    constexpr int KSTAGE = group8_kstage<NMAT>(), XBOXES = KSTAGE / kDenseKStep;
    const GroupRing &r = q.r;
    const int np = a.np, act_bytes = group_act_bytes(np);
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    const int n_tasks = *a.wl.n_groups * tiles * a.splits;
    for (int task = blockIdx.x; task < n_tasks && !*r.dead; task += gridDim.x) {
        const GroupTask t = group_task(a, task);
        const int ge = a.wl.g_expert[t.g];
        const int img = ge < a.E ? a.img_routed0 + ge : a.img_shared0 + (ge - a.E);
        const int xrow = NMAT == 2 ? 0 : a.wl.g_start[t.g];
        for (int k = t.k0; k < t.k1; k += KSTAGE) {
            if (!dmbar_wait(&r.empty[pos.s], pos.ph ^ 1u, r.dead)) return;
            uint8_t *st = r.dsm + (size_t)pos.s * r.slot;
            // boxes past the end of the reduction dimension are zero-filled and still count
            dmbar_expect_tx(&r.full[pos.s], (uint32_t)(2 * kGroup8BoxBytes + XBOXES * np * kDenseKStep * 2));
            tma_load_3d(st, map_w0, k, t.row0, img, &r.full[pos.s]);
            if (NMAT == 2)
                tma_load_3d(st + kGroup8BoxBytes, map_w1, k, t.row0, img, &r.full[pos.s]);
            else
                tma_load_3d(st + kGroup8BoxBytes, map_w0, k + kGroup8BoxCols, t.row0, img, &r.full[pos.s]);
#pragma unroll
            for (int x = 0; x < XBOXES; ++x)
                tma_load_2d(st + 2 * kGroup8BoxBytes + x * act_bytes, map_x, k + x * kDenseKStep, xrow, &r.full[pos.s]);
            ++issued;
            if (++pos.s == r.NS) pos.s = 0, pos.ph ^= 1u;
        }
    }
}

// One thread: MMAs with A from tensor memory, B (activations) from shared memory.  `it` counts
// the CTA's tasks across calls (accumulator buffer = it & 1).
template <int NMAT>
__device__ __forceinline__ void group8_mma(const GroupArgs &a, const Group8Ring &q, Group8Pos &pos, int &it)
{
    constexpr int KSTAGE = group8_kstage<NMAT>();
    const GroupRing &r = q.r;
    const int np = a.np, act_bytes = group_act_bytes(np);
    const uint32_t idesc = umma_idesc_f16(np);
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    const int n_tasks = *a.wl.n_groups * tiles * a.splits;
    for (int task = blockIdx.x; task < n_tasks && !*r.dead; task += gridDim.x, ++it) {
        const GroupTask t = group_task(a, task);
        const int ab = it & 1;
        if (!dmbar_wait(&r.tempty[ab], (((uint32_t)it >> 1) & 1u) ^ 1u, r.dead)) return;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = r.tmem + ab * 128;
        bool first = true;
        for (int k = t.k0; k < t.k1; k += KSTAGE, ++pos.stage_no) {
            const int buf = pos.stage_no & 1;
            if (!dmbar_wait(&q.afull[buf], ((uint32_t)pos.stage_no >> 1) & 1u, r.dead)) return;  // converted (implies landed)
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t xs = dsmem_u32(r.dsm + (size_t)pos.s * r.slot + 2 * kGroup8BoxBytes);
            const uint32_t abuf = r.tmem + 256 + buf * kGroup8ACols;
#pragma unroll
            for (int bx = 0; bx < 2; ++bx)
#pragma unroll
                for (int j = 0; j < kGroup8BoxCols / 16; ++j) {
                    // gate/up: both boxes multiply the same activation columns into their own
                    // accumulators; down: the second box continues the reduction
                    const int xb = (NMAT == 2 ? 0 : bx * 2) + (j >> 2);
                    const uint64_t bd = umma_desc_sw128(xs + xb * act_bytes, j & 3);
                    umma_f16_ts(acc + (NMAT == 2 ? bx * 64 : 0), abuf + bx * 64 + j * 8, bd, idesc,
                                !first || j > 0 || (NMAT == 1 && bx > 0));
                }
            first = false;
            umma_commit(&q.aempty[buf]);      // this A buffer may be rewritten
            umma_commit(&r.empty[pos.s]);     // and the stage reloaded
            if (++pos.s == r.NS) pos.s = 0;
        }
        umma_commit(&r.tfull[ab]);
    }
}

// Four warps (lg = warp index % 4): thread = one weight row (TMEM lane); applies the row scales.
template <int NMAT>
__device__ __forceinline__ void group8_epilogue(const Group8Args &a8, const Group8Ring &q, int &it, int lg, int lane)
{
    const GroupArgs &a = a8.g;
    const GroupRing &r = q.r;
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    const int n_tasks = *a.wl.n_groups * tiles * a.splits;
    for (int task = blockIdx.x; task < n_tasks; task += gridDim.x, ++it) {
        const GroupTask t = group_task(a, task);
        const int ab = it & 1;
        const int start = a.wl.g_start[t.g], count = a.wl.g_count[t.g];
        const int ge = a.wl.g_expert[t.g];
        const int img = ge < a.E ? a.img_routed0 + ge : a.img_shared0 + (ge - a.E);
        const int row = t.row0 + lg * kWarp + lane;
        // bf16 scales behind the three matrices: [gate I | up I | down H]
        const uint16_t *sc = reinterpret_cast<const uint16_t *>(a8.store + (size_t)img * a8.img_bytes +
                                                                3 * (size_t)a.rows * a.kd) + a8.scale_off;
        const int srow = min(row, a.rows - 1);
        const float s0 = bf16_to_f32(sc[srow]), s1 = NMAT == 2 ? bf16_to_f32(sc[a.rows + srow]) : 0.f;
        const bool ok = dmbar_wait(&r.tfull[ab], ((uint32_t)it >> 1) & 1u, r.dead);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = r.tmem + ab * 128 + ((uint32_t)(lg * kWarp) << 16);
        if (NMAT == 2) {
            for (int i = 0; i < count; ++i) {
                const int tok = a.wl.pair_token[start + i];
                const float inv = a.inv_rms[tok];  // W (inv * h) = inv * (W h)
                const float g = inv * s0 * tmem_ld1(acc + tok), u = inv * s1 * tmem_ld1(acc + 64 + tok);
                if (ok && row < a.rows) a8.act16[(size_t)(start + i) * a.rows + row] = __float2half_rn(g / (1.f + expf(-g)) * u);
            }
        } else {
            for (int i0 = 0; i0 < count; i0 += 8) {
                float y[8];
                tmem_ld8(acc + i0, y);
                if (ok && row < a.rows) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (i0 + i < count) {
                            const int slot = a.wl.pair_slot[start + i0 + i];
                            a.part[((size_t)slot * a.splits + t.z) * a.rows + row] = s0 * y[i];
                        }
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) dmbar_arrive(&r.tempty[ab]);
        if (!ok) return;
    }
}

// Eight warps, two per lane quarter lq (cw = 0..7: the warp's number among the converters; the
// warp must sit in lane quarter lq = its warp index % 4): thread = one weight row; the e4m3
// columns of its box become f16 pairs in tensor memory.
template <int NMAT>
__device__ __forceinline__ void group8_convert(const GroupArgs &a, const Group8Ring &q, Group8Pos &pos, int cw, int lq,
                                               int lane)
{
    constexpr int KSTAGE = group8_kstage<NMAT>();
    const GroupRing &r = q.r;
    const int bx = cw >> 2;
    const int row = lq * kWarp + lane, r7 = row & 7;
    const uint32_t lane_base = r.tmem + 256 + ((uint32_t)(lq * kWarp) << 16) + bx * 64;
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    const int n_tasks = *a.wl.n_groups * tiles * a.splits;
    for (int task = blockIdx.x; task < n_tasks; task += gridDim.x) {
        const GroupTask t = group_task(a, task);
        for (int k = t.k0; k < t.k1; k += KSTAGE, ++pos.stage_no) {
            const int buf = pos.stage_no & 1, use = pos.stage_no >> 1;
            if (!dmbar_wait(&r.full[pos.s], pos.ph, r.dead)) return;                                         // the boxes have landed
            if (use > 0 && !dmbar_wait(&q.aempty[buf], (uint32_t)(use - 1) & 1u, r.dead)) return;  // its previous MMAs are done
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint8_t *row_ptr = r.dsm + (size_t)pos.s * r.slot + bx * kGroup8BoxBytes + row * 128;
#pragma unroll
            for (int c0 = 0; c0 < 8; c0 += 2) {
                uint32_t v[16];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint4 raw = *reinterpret_cast<const uint4 *>(row_ptr + (((c0 + h) ^ r7) << 4));
                    uint4 lo, hi;
                    e4m3x16_to_f16(raw, lo, hi);
                    v[8 * h] = lo.x, v[8 * h + 1] = lo.y, v[8 * h + 2] = lo.z, v[8 * h + 3] = lo.w;
                    v[8 * h + 4] = hi.x, v[8 * h + 5] = hi.y, v[8 * h + 6] = hi.z, v[8 * h + 7] = hi.w;
                }
                tmem_st16(lane_base + buf * kGroup8ACols + c0 * 8, v);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) dmbar_arrive(&q.afull[buf]);
            if (++pos.s == r.NS) pos.s = 0, pos.ph ^= 1u;
        }
    }
}

// One projection as a kernel of its own (per-layer launches).
// NMAT = 2: gate and up projections with the SiLU epilogue; NMAT = 1: down projection.
template <int NMAT>
__global__ void __launch_bounds__(kGroup8Threads, 1)
dense8_group_kernel(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
                    const __grid_constant__ CUtensorMap map_x, Group8Args a8)
{
    const GroupArgs &a = a8.g;
    extern __shared__ uint8_t dsm_raw[];
    __shared__ uint64_t full[kGroupMaxStages], empty[kGroupMaxStages], tfull[2], tempty[2], afull[2], aempty[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_dead;
    const int tid = threadIdx.x, warp = tid / kWarp, lane = tid % kWarp;
    Group8Ring q;
    GroupRing &r = q.r;
    r.dsm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dsm_raw) + 1023) & ~(uintptr_t)1023);
    r.full = full, r.empty = empty, r.tfull = tfull, r.tempty = tempty, r.dead = &s_dead;
    q.afull = afull, q.aempty = aempty;
    r.NS = group8_stages<NMAT>(a.np), r.slot = group8_stage_bytes<NMAT>(a.np);
    if (tid == 0) {
        s_dead = r.NS < 1;
        group8_ring_init(q);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dsmem_u32(&s_tmem)), "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    r.tmem = s_tmem;

    if (warp == 0) {
        if (lane == 0) {
            Group8Pos pos;
            int issued = 0;
            group8_produce<NMAT>(&map_w0, &map_w1, &map_x, a, q, pos, issued);
            RingPos rp;
            rp.s = pos.s, rp.ph = pos.ph;
            group_drain(r, rp, issued);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            Group8Pos pos;
            int it = 0;
            group8_mma<NMAT>(a, q, pos, it);
        }
    } else if (warp < 6) {
        int it = 0;
        group8_epilogue<NMAT>(a8, q, it, warp % 4, lane);
    } else {
        Group8Pos pos;
        group8_convert<NMAT>(a, q, pos, warp - 6, warp % 4, lane);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(r.tmem), "r"(512) : "memory");
    }
    if (tid == 0 && s_dead) *a.err = 1u;
}

// h_out[b][c] = h[b][c] + r * (weighted sum of the partial sums); the f16 copy is the next
// layer's gate/up operand
__global__ void __launch_bounds__(256) dense8_combine_kernel(FfnArgs a, int S, __half *xb)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < a.B * a.H; i += gridDim.x * blockDim.x) {
        const float v = finish_value(a, i / a.H, i % a.H, S);
        a.h_out[i] = v;
        xb[i] = __float2half_rn(v);
    }
}

__global__ void __launch_bounds__(256) dense8_cast_kernel(const float *__restrict__ h, int n, __half *__restrict__ xb)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) xb[i] = __float2half_rn(h[i]);
}

}  // namespace stmoe_dev
