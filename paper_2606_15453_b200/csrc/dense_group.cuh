// Grouped expert FFN on the tensor cores for decode steps with several tokens per expert
// (tcgen05.mma, accumulators in tensor memory, operands staged by TMA; sm_100a).
//
// The work list holds one entry per active expert (all of its tokens).  A task is one entry x
// one tile of 128 weight rows (x one split of the reduction dimension for the down
// projection); tasks are dealt round-robin over a persistent grid of one CTA per SM.  Weights
// stay the streamed operand: the 128 weight rows are the MMA's M, the tokens its N (the batch
// padded to a multiple of 16), and the CTA walks the reduction dimension in boxes of 128 bytes
// per row (64 bf16 or 128 fp8 columns), one or more boxes per stage.
//   warp 0      one thread issues the TMA loads of a stage: the 128-row weight tile(s) through a
//               3-D tensor map over the expert store (column, row, image; for offloaded stacks
//               the slot store, the image index taken from the step's pointer table) and the
//               activation tile(s), all in the 128-byte swizzled layout the MMA reads
//   warp 1      one thread issues four tcgen05.mma per box and matrix (one per 32-byte slice),
//               frees the stage with tcgen05.commit and hands a finished accumulator to the
//               epilogue; the warp also owns the tensor-memory allocation
//   warps 2-5   epilogue: read the accumulator (two buffers, so the next task's MMAs overlap),
//               apply SiLU(gate)*up or nothing, store the rows of the entry's tokens
// Gate/up multiplies against the whole batch's hidden state (tensor work is free next to the
// weight stream); the epilogue keeps the entry's tokens and applies their RMSNorm factors.  The
// down projection multiplies against the entry's own rows of the activation buffer, which are
// consecutive.
// Every wait is bounded; a wait that runs out raises the error word and the kernel drains.
//
// Two operand formats (template parameter WDT):
//   1  bf16 weights x bf16 activations (kind::f16), 64 reduction columns per 128-byte box row;
//   2  fp8 stacks: e4m3 weights straight from the expert images x activations held as three
//      e5m2 planes whose sum is the activation (kind::f8f6f4, 128 reduction columns per box row).
//      e5m2 has the exponent range of f16, so no scaling pass is needed; each plane takes the
//      rounding residue of the one before (2 mantissa bits each: relative error 2^-9 after three,
//      the precision of a bf16 operand).  The planes' tiles lie one after the other in shared
//      memory and form ONE B operand of 3 x np rows: one MMA per weight tile and reduction slice
//      (an MMA's cost here is reading its 128 x 32-byte A tile from shared memory: one MMA per
//      plane into shared columns measured slower than widening the weights), three accumulator
//      columns per token that the epilogue adds.  Gate and up accumulators of more than 32 tokens
//      fit tensor memory only once, so those tasks run with a single accumulator buffer.  The
//      per-output-channel weight scales belong to the accumulator lanes and are applied in the
//      epilogue.
#pragma once
#include <cuda.h>
#include <cuda_fp8.h>

#include "dense_ffn.cuh"

namespace stmoe_dev {

constexpr int kGroupThreads = 192;
constexpr int kGroupTileBytes = kDenseRows * kDenseKStep * 2;     // 16 KB weight tile of a stage
constexpr int kGroupActBytes = kDenseMaxTokens * kDenseKStep * 2; // 8 KB activation tile (64 tokens)
constexpr int kGroupTmemCols = 256;                               // two accumulator buffers of 128 columns
constexpr int kGroup8TmemCols = 512;                              // fp8 format: two buffers of 192 columns (power of two)
// Accumulator layout in tensor memory.  bf16: two buffers of 128 columns, gate at +0 and up at +64.
// fp8 (three columns per token, np apart): buffers 192 columns apart; gate/up of up to 32 tokens at
// +0 / +96 in each of two buffers, of more tokens at +0 / +192 in a single buffer.
__host__ __device__ constexpr int group_acc_bufs(int nmat, int wdt, int np) { return wdt == 2 && nmat == 2 && np > 32 ? 1 : 2; }
__host__ __device__ constexpr int group_acc_stride(int wdt) { return wdt == 2 ? 192 : 128; }
__host__ __device__ constexpr int group_mat_stride(int wdt, int np) { return wdt == 1 ? 64 : (np > 32 ? 192 : 96); }
// which accumulator buffer the next task takes and how often each was used (its barriers' phase);
// the MMA thread and the epilogue threads each keep one and walk the same task sequence
struct AccPos {
    int use0 = 0, use1 = 0;  // scalars (an indexed array would live in local memory)
    int next = 0;
    __device__ __forceinline__ int take(int bufs)
    {
        const int ab = bufs == 1 ? 0 : next;
        if (bufs == 2) next ^= 1;
        return ab;
    }
    __device__ __forceinline__ uint32_t parity(int ab) const { return (uint32_t)(ab ? use1 : use0) & 1u; }
    __device__ __forceinline__ void used(int ab)
    {
        if (ab)
            ++use1;
        else
            ++use0;
    }
};

#ifndef STMOE_GROUP_KBOXES_GU
#define STMOE_GROUP_KBOXES_GU 2
#endif
#ifndef STMOE_GROUP_KBOXES_D
#define STMOE_GROUP_KBOXES_D 4
#endif
#ifndef STMOE_GROUP8_KBOXES_GU
#define STMOE_GROUP8_KBOXES_GU 1
#endif
#ifndef STMOE_GROUP8_KBOXES_D
#define STMOE_GROUP8_KBOXES_D 2
#endif
// reduction columns of a box row (128 bytes) and activation planes per operand format
template <int WDT> __host__ __device__ constexpr int group_box_cols() { return WDT == 1 ? kDenseKStep : 2 * kDenseKStep; }
template <int WDT> __host__ __device__ constexpr int group_planes() { return WDT == 1 ? 1 : 3; }
// Boxes per matrix and stage: consecutive boxes continue the same rows, so a stage asks for
// boxes * 128 contiguous bytes of every row at once.  bf16, measured on C1 batch 4 / C2 batch 8:
// (gate/up, down) = (1,1) 0.893 / 0.728 of the HBM roofline, (2,2) 0.919 / 0.754, (2,4) 0.927 /
// 0.762; 4 for gate/up leaves a single stage.
template <int NMAT, int WDT> __host__ __device__ constexpr int group_kboxes()
{
    return WDT == 1 ? (NMAT == 2 ? STMOE_GROUP_KBOXES_GU : STMOE_GROUP_KBOXES_D)
                    : (NMAT == 2 ? STMOE_GROUP8_KBOXES_GU : STMOE_GROUP8_KBOXES_D);
}
template <int NMAT, int WDT> __host__ __device__ constexpr int group_kstage() { return group_kboxes<NMAT, WDT>() * group_box_cols<WDT>(); }  // columns per stage
constexpr int kGroupMaxStages = 12;
constexpr int kGroupSmemBytes = 226 * 1024;                       // dynamic shared memory of a CTA (one per SM)
// A box holds NMAT weight tiles and, per activation plane, np rows of 128 bytes (np a multiple
// of 16, so every tile base stays 1024-byte aligned once rounded up); as many stages as fit.
__host__ __device__ constexpr int group_act_bytes(int np) { return (np * 128 + 1023) / 1024 * 1024; }
template <int NMAT, int WDT> __host__ __device__ constexpr int group_box_bytes(int np)
{
    return NMAT * kGroupTileBytes + group_planes<WDT>() * group_act_bytes(np);
}
template <int NMAT, int WDT> __host__ __device__ constexpr int group_stage_bytes(int np)
{
    return group_kboxes<NMAT, WDT>() * group_box_bytes<NMAT, WDT>(np);
}
template <int NMAT, int WDT> __host__ __device__ constexpr int group_stages(int np)
{
    const int n = (kGroupSmemBytes - 1024) / group_stage_bytes<NMAT, WDT>(np);
    return n < kGroupMaxStages ? n : kGroupMaxStages;
}

struct GroupArgs {
    WorkList wl;
    int E;                 // routed experts (entries with g_expert >= E are shared experts)
    int img_routed0;       // image index of this layer's expert 0 in the store
    int img_shared0;       // image index of this layer's shared expert 0
    const uint8_t *const *blob;  // offloaded stacks: this step's image pointer of every expert (into the slot
                                 // store the tensor maps cover); nullptr: images in layer order
    // Hand-over of the gated activations between the two projections of a layer inside one kernel,
    // entry by entry instead of by a grid barrier (nullptr: the caller separates the projections):
    unsigned *signal;            // gate/up: every epilogue warp adds 1 to signal[entry] per finished tile
    const unsigned *ready;       // down: an entry's tasks are loaded once ready[entry] >= ready_target
    unsigned ready_target;       // = epilogue warps x gate/up row tiles
    int rows;              // weight rows: I (gate/up) or H (down)
    int kd;                // reduction length: H (gate/up) or I (down)
    int np;                // batch padded to a multiple of 16 (MMA N and activation box rows)
    int splits, seg;       // down: splits of the reduction dimension, columns per split (multiple of 64)
    int KS;                // K + n_shared
    const float *inv_rms;  // gate/up: RMSNorm factor per sequence, applied to the accumulators
    __nv_bfloat16 *act;    // bf16 weights: gate/up out, down in: [pairs][I]
    float *part;           // down out: [B*KS][splits][H]
    unsigned *err;
    // fp8 stacks
    uint8_t *act8;         // gate/up out, down in: three e5m2 planes [3][act_rows][I]
    int act_rows;          // rows of one plane of act8
    int x_rows;            // rows of one plane of this projection's activation operand (hidden state: 64)
    const uint8_t *store;  // first expert image the tensor maps cover (stack or slot store); fp8: the row scales
                           // sit behind the matrices of an image
    unsigned long long img_bytes;
    int scale_off;         // element offset of this projection's scales in the image's scale vector
};

__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Bounded wait (one thread) until a counter that other CTAs raise with release semantics reaches
// `target`; false when the limit ran out or another thread of the CTA gave up.
__device__ __forceinline__ bool group_wait_counter(const unsigned *counter, unsigned target, volatile int *dead,
                                                   int spin_limit = kDenseSpinLimit)
{
    for (int spins = 0; spins < spin_limit; ++spins) {
        unsigned seen;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
        if (seen >= target) return true;
        if (*dead) return false;
        __nanosleep(64);
    }
    *dead = 1;
    return false;
}

// image index (third tensor-map coordinate) of work-list expert ge
__device__ __forceinline__ int group_image(const GroupArgs &a, int ge)
{
    if (a.blob) return (int)((size_t)(a.blob[ge] - a.store) / a.img_bytes);
    return ge < a.E ? a.img_routed0 + ge : a.img_shared0 + (ge - a.E);
}

// e4m3 weights x e5m2 activations -> fp32, both operands K-major, M = 128, N = n
__host__ __device__ constexpr uint32_t umma_idesc_e4m3_e5m2(int n)
{
    return (1u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kDenseRows >> 4) << 24);
}
__device__ __forceinline__ void umma_f8(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;}"
        :
        : "r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// v = t[0] + t[1] + t[2] up to 2^-9 |v|: each e5m2 term rounds what the terms before it left
// (an e5m2 value is the upper byte of the f16 with the same value)
__device__ __forceinline__ float e5m2_to_f32(uint8_t b)
{
    return __half2float(__ushort_as_half((unsigned short)((unsigned short)b << 8)));
}
__device__ __forceinline__ void split_e5m2x3(float v, uint8_t (&t)[3])
{
#pragma unroll
    for (int p = 0; p < 3; ++p) {
        t[p] = (uint8_t)__nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E5M2);
        v -= e5m2_to_f32(t[p]);
    }
}

__device__ __forceinline__ void dmbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(dsmem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dsmem_u32(dst)), "l"(map), "r"(dsmem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dsmem_u32(dst)), "l"(map), "r"(dsmem_u32(bar)), "r"(c0), "r"(c1)
        : "memory");
}
// K-major operand tile in the 128-byte swizzled layout (rows of 128 bytes, 8-row groups 1024
// bytes apart, tile base 1024-byte aligned); kstep = which 32-byte slice of the row (one MMA's
// reduction depth: 16 two-byte or 32 one-byte elements).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr, int kstep)
{
    return (uint64_t)(((smem_addr + kstep * 32) >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ float tmem_ld1(uint32_t addr)
{
    uint32_t r;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(addr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    return __uint_as_float(r);
}

struct GroupTask {
    int g, row0, k0, k1, z;
};
// task -> (entry, row tile, split); gate/up has one split
__device__ __forceinline__ GroupTask group_task(const GroupArgs &a, int task)
{
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    GroupTask t;
    t.g = task / (tiles * a.splits);
    const int r = task - t.g * tiles * a.splits;
    t.row0 = (r / a.splits) * kDenseRows;
    t.z = r % a.splits;
    t.k0 = t.z * a.seg;
    t.k1 = min(a.kd, t.k0 + a.seg);
    return t;
}

// Shared-memory ring of stages with its barriers, and the accumulator hand-off barriers.
struct GroupRing {
    uint8_t *dsm;                           // 1024-byte aligned
    uint64_t *full, *empty, *tfull, *tempty;
    int NS, slot;                           // stages, bytes per stage slot
    uint32_t tmem;                          // base of the 256 accumulator columns
    volatile int *dead;
};
// A role's place in the ring: the stage it handles next and, per stage, the parity of the barrier
// phase it waits for next (bit s toggles each time the role has used stage s).  Per-stage bits,
// not one wrap-around bit, so that a caller may restart at stage 0 with another stage count at a
// moment when every stage is empty (the persistent kernel does between its phases) without
// touching the barriers.
struct RingPos {
    int s = 0;
    uint32_t par = 0;
    __device__ __forceinline__ uint32_t parity() const { return (par >> s) & 1u; }
    __device__ __forceinline__ void advance(int NS)
    {
        par ^= 1u << s;
        if (++s == NS) s = 0;
    }
};

__device__ __forceinline__ void group_ring_init(const GroupRing &r)
{
    for (int s = 0; s < r.NS; ++s) dmbar_init(&r.full[s], 1), dmbar_init(&r.empty[s], 1);
    for (int b = 0; b < 2; ++b) dmbar_init(&r.tfull[b], 1), dmbar_init(&r.tempty[b], 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// One thread: issue the TMA loads of this CTA's tasks.  pos/issued carry on from earlier calls.
// NMAT = 2: gate and up projections; NMAT = 1: down projection.
template <int NMAT, int WDT>
__device__ __forceinline__ void group_produce(const CUtensorMap *map_w0, const CUtensorMap *map_w1,
                                              const CUtensorMap *map_x, const GroupArgs &a, const GroupRing &r,
                                              RingPos &pos, int &issued)
{
    constexpr int KB = group_kboxes<NMAT, WDT>(), KSTAGE = group_kstage<NMAT, WDT>(), COLS = group_box_cols<WDT>();
    constexpr int PLANES = group_planes<WDT>();
    const int np = a.np, act_bytes = group_act_bytes(np), box = group_box_bytes<NMAT, WDT>(np);
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    const int n_tasks = *a.wl.n_groups * tiles * a.splits;
    for (int task = blockIdx.x; task < n_tasks && !*r.dead; task += gridDim.x) {
        const GroupTask t = group_task(a, task);
        const int ge = a.wl.g_expert[t.g];
        const int img = group_image(a, ge);
        const int xrow = NMAT == 2 ? 0 : a.wl.g_start[t.g];
        if (NMAT == 1 && a.ready) {
            // the entry's gated activations: every gate/up tile of it has been stored and fenced
            if (!group_wait_counter(a.ready + t.g, a.ready_target, r.dead)) return;
            fence_async_proxy();  // they were written through the generic proxy, TMA reads them
        }
        for (int k = t.k0; k < t.k1; k += KSTAGE) {
            if (!dmbar_wait(&r.empty[pos.s], pos.parity() ^ 1u, r.dead)) return;
            uint8_t *st = r.dsm + (size_t)pos.s * r.slot;
            // boxes past the end of the reduction dimension are zero-filled and still count
            dmbar_expect_tx(&r.full[pos.s], (uint32_t)(KB * (NMAT * kGroupTileBytes + PLANES * np * 128)));
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                uint8_t *sb = st + kb * box;
                tma_load_3d(sb, map_w0, k + kb * COLS, t.row0, img, &r.full[pos.s]);
                if (NMAT == 2) tma_load_3d(sb + kGroupTileBytes, map_w1, k + kb * COLS, t.row0, img, &r.full[pos.s]);
#pragma unroll
                for (int p = 0; p < PLANES; ++p)
                    tma_load_2d(sb + NMAT * kGroupTileBytes + p * act_bytes, map_x, k + kb * COLS, p * a.x_rows + xrow,
                                &r.full[pos.s]);
            }
            ++issued;
            pos.advance(r.NS);
        }
    }
}

// Every load that was issued has to land before the CTA may exit.
__device__ __forceinline__ void group_drain(const GroupRing &r, RingPos pos, int issued)
{
    for (int i = 0; i < min(issued, r.NS); ++i) {  // the last loads, newest first: one per stage at most
        if (pos.s == 0) pos.s = r.NS;
        --pos.s;
        dmbar_wait(&r.full[pos.s], pos.parity() ^ 1u, r.dead);  // the phase before the producer's last toggle
    }
}

// The producer thread, before the ring is laid out anew: every stage it filled has been read by
// the MMAs (the waits it would do before refilling each stage; they change no state).
__device__ __forceinline__ bool group_wait_stages_free(const GroupRing &r, const RingPos &pos)
{
    for (int s = 0; s < r.NS; ++s)
        if (!dmbar_wait(&r.empty[s], ((pos.par >> s) & 1u) ^ 1u, r.dead)) return false;
    return true;
}

// One thread: issue the MMAs of this CTA's tasks.  `ap` carries the accumulator hand-off state
// across calls.
template <int NMAT, int WDT>
__device__ __forceinline__ void group_mma(const GroupArgs &a, const GroupRing &r, RingPos &pos, AccPos &ap)
{
    constexpr int KB = group_kboxes<NMAT, WDT>(), KSTAGE = group_kstage<NMAT, WDT>();
    const int np = a.np, box = group_box_bytes<NMAT, WDT>(np);
    const uint32_t idesc = WDT == 1 ? umma_idesc_bf16(np) : umma_idesc_e4m3_e5m2(3 * np);
    const int mat_stride = group_mat_stride(WDT, np), bufs = group_acc_bufs(NMAT, WDT, np);
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    const int n_tasks = *a.wl.n_groups * tiles * a.splits;
    for (int task = blockIdx.x; task < n_tasks && !*r.dead; task += gridDim.x) {
        const GroupTask t = group_task(a, task);
        const int ab = ap.take(bufs);
        if (!dmbar_wait(&r.tempty[ab], ap.parity(ab) ^ 1u, r.dead)) return;
        ap.used(ab);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = r.tmem + ab * group_acc_stride(WDT);
        bool first = true;
        for (int k = t.k0; k < t.k1; k += KSTAGE) {
            if (!dmbar_wait(&r.full[pos.s], pos.parity(), r.dead)) return;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                const uint32_t st = dsmem_u32(r.dsm + (size_t)pos.s * r.slot) + kb * box;
#pragma unroll
                for (int j = 0; j < 4; ++j) {  // four 32-byte slices of the 128-byte box row
                    // fp8: the planes' tiles follow one another and are the rows np.. of one operand
                    const uint64_t bd = umma_desc_sw128(st + NMAT * kGroupTileBytes, j);
#pragma unroll
                    for (int mat = 0; mat < NMAT; ++mat) {
                        const uint64_t ad = umma_desc_sw128(st + mat * kGroupTileBytes, j);
                        const bool accumulate = !first || kb > 0 || j > 0;
                        if constexpr (WDT == 1)
                            umma_bf16(acc + mat * mat_stride, ad, bd, idesc, accumulate);
                        else
                            umma_f8(acc + mat * mat_stride, ad, bd, idesc, accumulate);
                    }
                }
            }
            first = false;
            umma_commit(&r.empty[pos.s]);
            pos.advance(r.NS);
        }
        umma_commit(&r.tfull[ab]);
    }
}

// Four warps (lg = the TMEM lane quarter the warp may read = warp index % 4): thread = one
// weight row.  `ap` as in group_mma.
template <int NMAT, int WDT>
__device__ __forceinline__ void group_epilogue(const GroupArgs &a, const GroupRing &r, AccPos &ap, int lg, int lane)
{
    const int tiles = (a.rows + kDenseRows - 1) / kDenseRows;
    const int n_tasks = *a.wl.n_groups * tiles * a.splits;
    const int bufs = group_acc_bufs(NMAT, WDT, a.np);
    for (int task = blockIdx.x; task < n_tasks; task += gridDim.x) {
        const GroupTask t = group_task(a, task);
        const int ab = ap.take(bufs);
        const int start = a.wl.g_start[t.g], count = a.wl.g_count[t.g];
        const int row = t.row0 + lg * kWarp + lane;
        float s0 = 1.f, s1 = 1.f;
        if constexpr (WDT == 2) {
            // bf16 scales per output channel behind the three matrices: [gate I | up I | down H]
            const int ge = a.wl.g_expert[t.g];
            const int img = group_image(a, ge);
            const uint16_t *sc = reinterpret_cast<const uint16_t *>(a.store + (size_t)img * a.img_bytes +
                                                                    3 * (size_t)a.rows * a.kd) + a.scale_off;
            const int srow = min(row, a.rows - 1);
            s0 = bf16_to_f32(sc[srow]);
            if (NMAT == 2) s1 = bf16_to_f32(sc[a.rows + srow]);
        }
        const bool ok = dmbar_wait(&r.tfull[ab], ap.parity(ab), r.dead);
        ap.used(ab);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = r.tmem + ab * group_acc_stride(WDT) + ((uint32_t)(lg * kWarp) << 16);
        constexpr bool stacked = WDT == 2;  // three columns per token, np apart: add them
        const int mat_stride = group_mat_stride(WDT, a.np);
        if (NMAT == 2) {
            for (int i = 0; i < count; ++i) {
                const int tok = a.wl.pair_token[start + i];
                const float inv = a.inv_rms[tok];  // W (inv * h) = inv * (W h)
                float ga = tmem_ld1(acc + tok), ua = tmem_ld1(acc + mat_stride + tok);
                if (stacked) {
                    ga = (ga + tmem_ld1(acc + a.np + tok)) + tmem_ld1(acc + 2 * a.np + tok);
                    ua = (ua + tmem_ld1(acc + mat_stride + a.np + tok)) + tmem_ld1(acc + mat_stride + 2 * a.np + tok);
                }
                const float g = inv * s0 * ga, u = inv * s1 * ua;
                const float v = g / (1.f + expf(-g)) * u;
                if (ok && row < a.rows) {
                    if constexpr (WDT == 1) {
                        a.act[(size_t)(start + i) * a.rows + row] = __float2bfloat16_rn(v);
                    } else {
                        uint8_t tp[3];
                        split_e5m2x3(v, tp);
#pragma unroll
                        for (int p = 0; p < 3; ++p) a.act8[((size_t)p * a.act_rows + start + i) * a.rows + row] = tp[p];
                    }
                }
            }
        } else {
            for (int i0 = 0; i0 < count; i0 += 8) {
                float y[8];
                tmem_ld8(acc + i0, y);
                if (stacked) {
                    float y1[8], y2[8];
                    tmem_ld8(acc + a.np + i0, y1);
                    tmem_ld8(acc + 2 * a.np + i0, y2);
#pragma unroll
                    for (int i = 0; i < 8; ++i) y[i] = (y[i] + y1[i]) + y2[i];
                }
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
        if (NMAT == 2 && a.signal) fence_async_proxy();  // this thread's activation stores, for the TMA of another SM
        __syncwarp();
        if (lane == 0) {
            dmbar_arrive(&r.tempty[ab]);
            if (NMAT == 2 && a.signal && ok)
                asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(a.signal + t.g), "r"(1u) : "memory");
        }
        if (!ok) return;
    }
}

// One projection as a kernel of its own (per-layer launches).
template <int NMAT, int WDT>
__global__ void __launch_bounds__(kGroupThreads, 1)
dense_group_kernel(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
                   const __grid_constant__ CUtensorMap map_x, GroupArgs a)
{
    constexpr int kTmemCols = WDT == 1 ? kGroupTmemCols : kGroup8TmemCols;
    extern __shared__ uint8_t dsm_raw[];
    __shared__ uint64_t full[kGroupMaxStages], empty[kGroupMaxStages], tfull[2], tempty[2];
    __shared__ uint32_t s_tmem;
    __shared__ int s_dead;
    const int tid = threadIdx.x, warp = tid / kWarp, lane = tid % kWarp;
    GroupRing r;
    r.dsm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dsm_raw) + 1023) & ~(uintptr_t)1023);
    r.full = full, r.empty = empty, r.tfull = tfull, r.tempty = tempty, r.dead = &s_dead;
    r.NS = group_stages<NMAT, WDT>(a.np), r.slot = group_stage_bytes<NMAT, WDT>(a.np);
    if (tid == 0) {
        s_dead = r.NS < 1;  // cannot happen with the host's sizing; never run a ring without stages
        group_ring_init(r);
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

    if (warp == 0) {
        if (lane == 0) {
            RingPos pos;
            int issued = 0;
            group_produce<NMAT, WDT>(&map_w0, &map_w1, &map_x, a, r, pos, issued);
            group_drain(r, pos, issued);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            RingPos pos;
            AccPos ap;
            group_mma<NMAT, WDT>(a, r, pos, ap);
        }
    } else {
        AccPos ap;
        group_epilogue<NMAT, WDT>(a, r, ap, warp % 4, lane);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(r.tmem), "r"(kTmemCols) : "memory");
    }
    if (tid == 0 && s_dead) *a.err = 1u;
}

// h_out[b][c] = h[b][c] + r * (weighted sum of the down projection's partial sums); the bf16
// copy is the next layer's gate/up operand
__global__ void __launch_bounds__(256) dense_combine_kernel(FfnArgs a, int S, __nv_bfloat16 *xb)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < a.B * a.H; i += gridDim.x * blockDim.x) {
        const float v = finish_value(a, i / a.H, i % a.H, S);
        a.h_out[i] = v;
        xb[i] = __float2bfloat16_rn(v);
    }
}

}  // namespace stmoe_dev
