// Grouped expert FFN on the tensor cores for fp8 (e4m3) expert weights.
//
// Same task structure as dense_group.cuh (one work-list entry per expert, a task = entry x 128
// weight rows x one split, persistent CTA per SM, weights as the MMA's M operand).  tcgen05 has no
// fp8 x 16-bit mode, and rounding the activations to fp8 would not fit the error bound, so the
// weights are widened on the way: TMA lands the e4m3 tile (128 rows x 128 columns, 16 KB) in a
// staging ring, eight converter warps rewrite it as two f16 operand tiles (e4m3 -> f16 is exact) in
// the 128-byte swizzled layout, and the MMA runs in f16 x f16 -> fp32 against f16 activations.
// The per-output-channel scales belong to the weight rows = accumulator lanes and are applied in
// the epilogue.
//   warp 0       TMA producer: weight tile(s) + two activation boxes per stage
//   warp 1       MMA issue (4 K=16 steps per 64-column half of a stage and matrix), tensor-memory owner
//   warps 2-5    epilogue (two accumulator buffers)
//   warps 6-13   converters
// Rings: `NS` staging stages (fp8 weights + activation boxes) and two operand buffers, so the
// conversion of one unit overlaps the MMAs of the other; a stage is released when its MMAs have
// completed.  Every wait is bounded.
#pragma once
#include <cuda_fp16.h>

#include "dense_group.cuh"

namespace stmoe_dev {

constexpr int kGroup8Threads = 448;
constexpr int kGroup8ConvWarps = 8;
constexpr int kGroup8KStage = 128;                                  // fp8 columns per stage
constexpr int kGroup8StageW = kDenseRows * kGroup8KStage;           // 16 KB of e4m3 per matrix and stage
// Two operand buffers, so that the conversion of one unit overlaps the MMAs of the other.  A unit
// is one 64-column half of a stage for gate/up (two matrices) and the whole stage for the down
// projection (one matrix: fewer, longer hand-offs), 32 KB of f16 either way.
template <int NMAT> __host__ __device__ constexpr int group8_unit_halves() { return NMAT == 2 ? 1 : 2; }
template <int NMAT> __host__ __device__ constexpr int group8_operand_buffers() { return 2; }

struct Group8Args {
    GroupArgs g;                 // act/part as in GroupArgs (act unused), inv_rms, work list, sizes
    const uint8_t *store;        // first expert image of the stack
    unsigned long long img_bytes;
    __half *act16;               // gate/up out, down in: [pairs + 64][I]
    int scale_off;               // element offset of this projection's scales in the image's scale vector
};

template <int NMAT> __host__ __device__ constexpr int group8_stage_bytes(int np)
{
    return NMAT * kGroup8StageW + 2 * group_act_bytes(np);
}
template <int NMAT> __host__ __device__ constexpr int group8_stages(int np)
{
    const int n = (kGroupSmemBytes - 1024 - group8_operand_buffers<NMAT>() * group8_unit_halves<NMAT>() * NMAT * kGroupTileBytes) /
                  group8_stage_bytes<NMAT>(np);
    return n < kGroupMaxStages ? n : kGroupMaxStages;
}
__host__ __device__ constexpr uint32_t umma_idesc_f16(int n)
{
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kDenseRows >> 4) << 24);  // f16 x f16 -> f32
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t idesc, bool accumulate)
{
    umma_bf16(tmem_d, a, b, idesc, accumulate);  // same instruction; the operand types are in idesc
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

template <int NMAT>
__global__ void __launch_bounds__(kGroup8Threads, 1)
dense8_group_kernel(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
                    const __grid_constant__ CUtensorMap map_x, Group8Args a8)
{
    const GroupArgs &a = a8.g;
    extern __shared__ uint8_t dsm_raw[];
    constexpr int NOB = group8_operand_buffers<NMAT>(), UH = group8_unit_halves<NMAT>(), UNIT = UH * NMAT * kGroupTileBytes;
    __shared__ uint64_t full[kGroupMaxStages], empty[kGroupMaxStages], tfull[2], tempty[2], ofull[NOB], oempty[NOB];
    __shared__ uint32_t s_tmem;
    __shared__ int s_dead;
    const int tid = threadIdx.x, warp = tid / kWarp, lane = tid % kWarp;
    const int np = a.np, act_bytes = group_act_bytes(np);
    const int NS = group8_stages<NMAT>(np), STAGE = group8_stage_bytes<NMAT>(np);
    uint8_t *dsm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dsm_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *opnd = dsm + (size_t)NS * STAGE;  // NOB buffers x (NMAT x UH) f16 half-tiles
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    const int n_tasks = *a.wl.n_groups * tiles * a.splits;
    volatile int *dead = &s_dead;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) dmbar_init(&full[s], 1), dmbar_init(&empty[s], 1);
        for (int b = 0; b < 2; ++b) dmbar_init(&tfull[b], 1), dmbar_init(&tempty[b], 4);
        for (int b = 0; b < NOB; ++b) dmbar_init(&ofull[b], kGroup8ConvWarps), dmbar_init(&oempty[b], 1);
        s_dead = NS < 1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dsmem_u32(&s_tmem)),
                     "r"(kGroupTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    if (warp == 0) {
        // ---- TMA producer -----------------------------------------------------------------------
        if (lane == 0) {
            int s = 0, issued = 0;
            uint32_t ph = 0;
            for (int task = blockIdx.x; task < n_tasks && !*dead; task += gridDim.x) {
                const GroupTask t = group_task(a, task);
                const int ge = a.wl.g_expert[t.g];
                const int img = ge < a.E ? a.img_routed0 + ge : a.img_shared0 + (ge - a.E);
                const int xrow = NMAT == 2 ? 0 : a.wl.g_start[t.g];
                bool ok = true;
                for (int k = t.k0; k < t.k1 && ok; k += kGroup8KStage) {
                    ok = dmbar_wait(&empty[s], ph ^ 1u, dead);
                    if (!ok) break;
                    uint8_t *st = dsm + (size_t)s * STAGE;
                    dmbar_expect_tx(&full[s], (uint32_t)(NMAT * kGroup8StageW + 2 * np * kDenseKStep * 2));
                    tma_load_3d(st, &map_w0, k, t.row0, img, &full[s]);
                    if (NMAT == 2) tma_load_3d(st + kGroup8StageW, &map_w1, k, t.row0, img, &full[s]);
                    tma_load_2d(st + NMAT * kGroup8StageW, &map_x, k, xrow, &full[s]);
                    tma_load_2d(st + NMAT * kGroup8StageW + act_bytes, &map_x, k + kDenseKStep, xrow, &full[s]);
                    ++issued;
                    if (++s == NS) s = 0, ph ^= 1u;
                }
                if (!ok) break;
            }
            for (int i = 0; i < min(issued, NS); ++i) {  // every load that was issued has to land
                if (s == 0) s = NS, ph ^= 1u;
                --s;
                dmbar_wait(&full[s], ph, dead);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issue ----------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(np);
            int s = 0, it = 0, half_no = 0;  // half_no counts units; operand buffer = half_no % NOB
            for (int task = blockIdx.x; task < n_tasks && !*dead; task += gridDim.x, ++it) {
                const GroupTask t = group_task(a, task);
                const int ab = it & 1;
                if (!dmbar_wait(&tempty[ab], (((uint32_t)it >> 1) & 1u) ^ 1u, dead)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem + ab * 128;
                bool first = true, ok = true;
                for (int k = t.k0; k < t.k1 && ok; k += kGroup8KStage) {
                    const uint32_t xs = dsmem_u32(dsm + (size_t)s * STAGE + NMAT * kGroup8StageW);
#pragma unroll
                    for (int unit = 0; unit < 2 / UH; ++unit, ++half_no) {
                        const int ob = half_no % NOB;
                        ok = ok && dmbar_wait(&ofull[ob], (uint32_t)(half_no / NOB) & 1u, dead);  // converted (implies landed)
                        if (!ok) break;
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t ws = dsmem_u32(opnd) + ob * UNIT;
#pragma unroll
                        for (int h = 0; h < UH; ++h) {
                            const int sub = unit * UH + h;
#pragma unroll
                            for (int j = 0; j < kDenseKStep / 16; ++j) {
                                const uint64_t bd = umma_desc_sw128(xs + sub * act_bytes, j);
#pragma unroll
                                for (int mat = 0; mat < NMAT; ++mat)
                                    umma_f16(acc + mat * 64, umma_desc_sw128(ws + (mat * UH + h) * kGroupTileBytes, j), bd,
                                             idesc, !first || sub > 0 || j > 0);
                            }
                        }
                        umma_commit(&oempty[ob]);  // this operand buffer may be rewritten
                    }
                    if (!ok) break;
                    first = false;
                    umma_commit(&empty[s]);  // the stage: fp8 tile consumed by the converters, activation boxes by these MMAs
                    if (++s == NS) s = 0;
                }
                if (!ok) break;
                umma_commit(&tfull[ab]);
            }
        }
    } else if (warp < 6) {
        // ---- epilogue: thread = one weight row (TMEM lane) -------------------------------------
        const int lg = warp % 4;
        int it = 0;
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
            const bool ok = dmbar_wait(&tfull[ab], ((uint32_t)it >> 1) & 1u, dead);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t acc = tmem + ab * 128 + ((uint32_t)(lg * kWarp) << 16);
            if (NMAT == 2) {
                for (int i = 0; i < count; ++i) {
                    const int tok = a.wl.pair_token[start + i];
                    const float inv = a.inv_rms[tok];
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
            if (lane == 0) dmbar_arrive(&tempty[ab]);
            if (!ok) break;
        }
    } else {
        // ---- converters: e4m3 staging tile -> two f16 operand tiles per matrix -------------------
        // Thread = (row rb of 64, one of a half's four 16-byte fp8 chunks); it handles rows rb and
        // rb + 64 of every matrix, so all of its shared-memory offsets are fixed up front.
        const int ct = (warp - 6) * kWarp + lane;  // 0 .. 255
        const int cl = ct & 3, rb = ct >> 2, r7 = rb & 7;
        const int src_off[2] = {rb * 128 + ((cl ^ r7) << 4), rb * 128 + (((4 + cl) ^ r7) << 4)};
        const int dst_lo = rb * 128 + (((cl * 2) ^ r7) << 4), dst_hi = rb * 128 + (((cl * 2 + 1) ^ r7) << 4);
        int s = 0, half_no = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int task = blockIdx.x; task < n_tasks && ok; task += gridDim.x) {
            const GroupTask t = group_task(a, task);
            for (int k = t.k0; k < t.k1 && ok; k += kGroup8KStage) {
                ok = dmbar_wait(&full[s], ph, dead);  // the fp8 tile has landed
                const uint8_t *st = dsm + (size_t)s * STAGE;
#pragma unroll
                for (int unit = 0; unit < 2 / UH; ++unit, ++half_no) {
                    if (!ok) break;
                    const int ob = half_no % NOB, use = half_no / NOB;
                    if (use > 0) ok = dmbar_wait(&oempty[ob], (uint32_t)(use - 1) & 1u, dead);  // its previous MMAs are done
                    if (!ok) break;
                    uint8_t *ow = opnd + ob * UNIT;
#pragma unroll
                    for (int h = 0; h < UH; ++h)
#pragma unroll
                        for (int mat = 0; mat < NMAT; ++mat)
#pragma unroll
                            for (int pass = 0; pass < 2; ++pass) {
                                const uint4 v = *reinterpret_cast<const uint4 *>(st + mat * kGroup8StageW + pass * 64 * 128 +
                                                                                 src_off[unit * UH + h]);
                                uint4 lo, hi;
                                e4m3x16_to_f16(v, lo, hi);
                                uint8_t *dst = ow + (mat * UH + h) * kGroupTileBytes + pass * 64 * 128;
                                *reinterpret_cast<uint4 *>(dst + dst_lo) = lo;
                                *reinterpret_cast<uint4 *>(dst + dst_hi) = hi;
                            }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) dmbar_arrive(&ofull[ob]);
                }
                if (++s == NS) s = 0, ph ^= 1u;
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kGroupTmemCols) : "memory");
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
