// Expert FFN for many tokens per expert as a tensor-core GEMM (tcgen05 + TMEM, sm_100a).
//
// With m tokens sharing one expert the FFN does m flop per weight byte; from about 8 tokens on
// the CUDA-core GEMV kernels are bound by their own arithmetic and activation loads instead of
// HBM.  Here the weights stay the streamed operand ("swap-AB"): one CTA owns 128 weight rows
// (the MMA's M), the tokens are the MMA's N (padded to a multiple of 16, <= 64), and the CTA
// walks the reduction dimension in 64-column steps:
//   warps 0-3  copy the 128x64 bf16 weight tile(s) and the Nx64 activation tile of each step
//              into a ring of shared-memory stages with 16-byte cp.async, laid out as the
//              K-major "interleaved" (no swizzle) canonical UMMA layout: 8 rows x 16 bytes per
//              core matrix; then read the accumulators back from TMEM for the epilogue;
//   warp 4     (one elected lane) issues tcgen05.mma.kind::f16 (bf16 x bf16 -> fp32 in TMEM),
//              four K=16 instructions per step and matrix, and releases each stage with
//              tcgen05.commit on the stage's "empty" mbarrier.
// Every wait is bounded; a wait that runs out raises the error word, the kernel drains and
// frees its TMEM columns.
#pragma once
#include <cuda_bf16.h>

#include "device_utils.cuh"
#include "ffn.cuh"

namespace stmoe_dev {

constexpr int kDenseStages = 4;
constexpr int kDenseThreads = 160;       // 4 load/epilogue warps + 1 MMA warp
constexpr int kDenseRows = 128;          // weight rows per CTA = MMA M
constexpr int kDenseKStep = 64;          // reduction columns per stage
constexpr int kDenseMaxTokens = 64;
constexpr int kDenseSpinLimit = 1 << 22;
constexpr int kDenseTmemCols = 128;      // gate accumulators in columns [0,64), up in [64,128)

__device__ __forceinline__ uint32_t dsmem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void dmbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(dsmem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void dmbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(dsmem_u32(bar)) : "memory");
}
// bounded wait on a phase parity; false when the limit ran out or another thread gave up
__device__ __forceinline__ bool dmbar_wait(uint64_t *bar, uint32_t parity, volatile int *dead,
                                           int spin_limit = kDenseSpinLimit)
{
    for (int spins = 0; spins < spin_limit; ++spins) {
        uint32_t done;
        asm volatile(
            "{.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;}"
            : "=r"(done)
            : "r"(dsmem_u32(bar)), "r"(parity)
            : "memory");
        if (done) return true;
        if (*dead) return false;
    }
    *dead = 1;
    return false;
}

// K-major, no-swizzle shared-memory matrix descriptor: 8-row groups `sbo` bytes apart, the two
// 16-byte K chunks of one MMA `lbo` bytes apart (descriptor version 1 = sm_100).
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kDenseRows >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;}"
        :
        : "r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(dsmem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t addr, float (&v)[8])
{
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(addr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

struct DenseArgs {
    const __nv_bfloat16 *W0;   // [rows][kd] gate (or down) weights, row-major
    const __nv_bfloat16 *W1;   // [rows][kd] up weights (NMAT = 2), else unused
    const __nv_bfloat16 *X;    // [np][kd] activations, token-major
    int rows, kd, m, np;       // np = tokens padded to a multiple of 16
    __nv_bfloat16 *act_out;    // NMAT = 2: [np][rows] silu(gate) * up
    float *y_out;              // NMAT = 1: [m][rows]
    unsigned *err;
};

// x_b[t][i] = bf16(h[t][i] * inv_rms[t]) for t < m, zeros for the padding tokens
__global__ void __launch_bounds__(256)
dense_cast_kernel(const float *__restrict__ h, const float *__restrict__ inv_rms, int m, int np, int H,
                  __nv_bfloat16 *__restrict__ xb)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)np * H; i += (size_t)gridDim.x * blockDim.x) {
        const int t = (int)(i / H);
        const float v = t < m ? h[i] * (inv_rms ? inv_rms[t] : 1.f) : 0.f;
        xb[i] = __float2bfloat16_rn(v);
    }
}

// out^T tile = W[row0 .. row0+127][:] * X^T  (NMAT = 2: gate and up with the SiLU epilogue).
template <int NMAT>
__global__ void __launch_bounds__(kDenseThreads, 1) dense_ffn_kernel(DenseArgs a)
{
    constexpr int NS = kDenseStages, KS = kDenseKStep, CH = KS / 8;  // CH 16-byte chunks per row and step
    constexpr int A_BYTES = kDenseRows * KS * 2;                     // one weight tile of a stage
    extern __shared__ __align__(128) uint8_t dsm[];
    __shared__ uint64_t full[NS], empty[NS], done;
    __shared__ uint32_t s_tmem;
    __shared__ int s_dead;
    const int tid = threadIdx.x, warp = tid / kWarp, lane = tid % kWarp;
    const int np = a.np, kd = a.kd;
    const int b_bytes = np * KS * 2;
    const int stage_bytes = NMAT * A_BYTES + b_bytes;
    const int row0 = blockIdx.x * kDenseRows;
    const int nk = kd / KS;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) dmbar_init(&full[s], 128), dmbar_init(&empty[s], 1);
        dmbar_init(&done, 1);
        s_dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 4) {  // one warp allocates (and later frees) the accumulator columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dsmem_u32(&s_tmem)),
                     "r"(kDenseTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    if (warp < 4) {
        // ---- producers: stage it holds reduction columns [it*64, it*64+64) -------------------
        constexpr int LA = NS - 1;
        for (int it = 0; it < nk + LA; ++it) {
            if (it < nk) {
                const int s = it % NS;
                if (it >= NS) dmbar_wait(&empty[s], (uint32_t)((it / NS) - 1) & 1u, &s_dead);
                uint8_t *st = dsm + (size_t)s * stage_bytes;
                // weight tiles: piece p = (row r, chunk kc); chunk-major core-matrix layout
                for (int p = tid; p < NMAT * kDenseRows * CH; p += 128) {
                    const int mat = p / (kDenseRows * CH), q = p % (kDenseRows * CH);
                    const int r = q / CH, kc = q % CH;
                    const int row = min(row0 + r, a.rows - 1);
                    const __nv_bfloat16 *src = (mat == 0 ? a.W0 : a.W1) + (size_t)row * kd + it * KS + kc * 8;
                    uint8_t *dst = st + mat * A_BYTES + kc * (kDenseRows * 16) + (r / 8) * 128 + (r % 8) * 16;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dsmem_u32(dst)), "l"(src) : "memory");
                }
                for (int p = tid; p < np * CH; p += 128) {
                    const int t = p / CH, kc = p % CH;
                    const __nv_bfloat16 *src = a.X + (size_t)t * kd + it * KS + kc * 8;
                    uint8_t *dst = st + NMAT * A_BYTES + kc * (np * 16) + (t / 8) * 128 + (t % 8) * 16;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dsmem_u32(dst)), "l"(src) : "memory");
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            if (it >= LA) {  // the stage issued LA iterations ago has landed: publish it
                asm volatile("cp.async.wait_group %0;" ::"n"(LA) : "memory");
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                dmbar_arrive(&full[(it - LA) % NS]);
            }
        }
        // ---- epilogue: thread = one weight row (TMEM lane), columns = tokens -------------------
        const bool ok = dmbar_wait(&done, 0u, &s_dead);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int row = row0 + warp * kWarp + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(warp * kWarp) << 16);
        for (int c0 = 0; c0 < np; c0 += 8) {
            float g[8], u[8];
            tmem_ld8(lane_base + c0, g);
            if (NMAT == 2) tmem_ld8(lane_base + 64 + c0, u);
            if (ok && row < a.rows) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int t = c0 + i;
                    if (NMAT == 2) {
                        const float v = t < a.m ? g[i] / (1.f + expf(-g[i])) * u[i] : 0.f;
                        a.act_out[(size_t)t * a.rows + row] = __float2bfloat16_rn(v);
                    } else if (t < a.m) {
                        a.y_out[(size_t)t * a.rows + row] = g[i];
                    }
                }
            }
        }
    } else if (lane == 0) {
        // ---- MMA issue: one thread ---------------------------------------------------------------
        const uint32_t idesc = umma_idesc_bf16(np);
        for (int it = 0; it < nk; ++it) {
            const int s = it % NS;
            if (!dmbar_wait(&full[s], (uint32_t)(it / NS) & 1u, &s_dead)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t st = dsmem_u32(dsm + (size_t)s * stage_bytes);
#pragma unroll
            for (int j = 0; j < KS / 16; ++j) {
                const uint64_t bd = umma_desc(st + NMAT * A_BYTES + 2 * j * (np * 16), np * 16, 128);
#pragma unroll
                for (int mat = 0; mat < NMAT; ++mat) {
                    const uint64_t ad = umma_desc(st + mat * A_BYTES + 2 * j * (kDenseRows * 16), kDenseRows * 16, 128);
                    umma_bf16(tmem + mat * 64, ad, bd, idesc, it > 0 || j > 0);
                }
            }
            umma_commit(&empty[s]);  // arrives when the MMAs above have finished reading the stage
        }
        umma_commit(&done);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 4) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kDenseTmemCols) : "memory");
    }
    if (tid == 0 && s_dead) *a.err = 1u;
}

}  // namespace stmoe_dev
