// Host runtime and C ABI of the decode-time MoE layer step: weight storage, predictor
// tables, the HBM slot cache with its copy stream and event fences, kernel launches.
#include "../../include/stmoe.h"

#include <atomic>
#include <chrono>
#include <cstdio>
#include <cstring>
#include <deque>
#include <new>
#include <set>
#include <tuple>
#include <utility>
#include <vector>

#include "dense_ffn.cuh"
#include "dense8_group.cuh"
#include "dense_group.cuh"
#include "device_utils.cuh"
#include "ffn.cuh"
#include "predictor.cuh"
#include "router.cuh"
#include "token_dense_kernel.cuh"
#include "token_fused_kernel.cuh"
#include "token_kernel.cuh"

using namespace stmoe_dev;

#define CU_TRY(expr)                                  \
    do {                                              \
        cudaError_t e_ = (expr);                      \
        if (e_ != cudaSuccess) {                      \
            (void)cudaGetLastError();                 \
            return e_ == cudaErrorMemoryAllocation ? STMOE_ERR_OOM : STMOE_ERR_CUDA; \
        }                                             \
    } while (0)
#define ST_TRY(expr)            \
    do {                        \
        int r_ = (expr);        \
        if (r_ != STMOE_OK) return r_; \
    } while (0)

namespace {

constexpr uint32_t kStateMagic = 0x53544D50;
constexpr int kWaitTimeoutMs = 20000;

inline int dtype_bytes(int dt) { return dt == STMOE_F32 ? 4 : dt == STMOE_BF16 ? 2 : 1; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// the down projection's rows are cut into segments of at most 16 KB so that the last block a
// warp claims stays short
int down_splits(int I, int dt)
{
    return (int)((((size_t)I * dtype_bytes(dt)) + STMOE_SEG_BYTES - 1) / STMOE_SEG_BYTES);
}

size_t image_bytes(int H, int I, int dt)
{
    size_t n = 3 * (size_t)H * I * dtype_bytes(dt);
    if (dt == STMOE_FP8_E4M3) n += 2 * (size_t)(2 * I + H);
    return round_up(n, 256);
}

// ---- kernel dispatch -------------------------------------------------------------------
// MTMAX = 1: every work-list entry holds one token.  MTMAX = 4: entries of 1..4 tokens; the
// kernel is instantiated for 4 and clamps (extra token columns recompute the last token).
struct FfnPlan {
    int grid_gate_up = 0, grid_down = 0;
};

// Launch with the programmatic-stream-serialization attribute: the kernel may start before the
// previous kernel in the stream has finished and orders itself with griddepcontrol.wait.
template <typename Arg> void launch_pdl(void (*kernel)(Arg), int grid, int block, cudaStream_t st, const Arg &arg)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid), cfg.blockDim = dim3(block), cfg.dynamicSmemBytes = 0, cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at, cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, arg);
}

template <int DT, int MT> void launch_gate_up(const FfnArgs &a, int grid, cudaStream_t st)
{
    gate_up_kernel<DT, MT><<<grid, kFfnThreads, 0, st>>>(a);
}
template <int DT, int MT> void launch_down(const FfnArgs &a, int grid, cudaStream_t st)
{
    launch_pdl(down_kernel<DT, MT>, grid, kFfnThreads, st, a);
}
template <int DT, int MT> int occupancy_gate_up()
{
    int n = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, gate_up_kernel<DT, MT>, kFfnThreads, 0);
    return n;
}
template <int DT, int MT> int occupancy_down()
{
    int n = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, down_kernel<DT, MT>, kFfnThreads, 0);
    return n;
}

#define DISPATCH_DT_MT(dt, mt, FN, ...)                      \
    do {                                                     \
        if ((dt) == STMOE_F32) {                             \
            if ((mt) == 1) FN<0, 1>(__VA_ARGS__); else FN<0, 4>(__VA_ARGS__); \
        } else if ((dt) == STMOE_BF16) {                     \
            if ((mt) == 1) FN<1, 1>(__VA_ARGS__); else FN<1, 4>(__VA_ARGS__); \
        } else {                                             \
            if ((mt) == 1) FN<2, 1>(__VA_ARGS__); else FN<2, 4>(__VA_ARGS__); \
        }                                                    \
    } while (0)

int occ_gate_up(int dt, int mt)
{
    int n = 0;
#define OCC_G(DT, MT) n = occupancy_gate_up<DT, MT>()
    if (dt == STMOE_F32) { if (mt == 1) OCC_G(0, 1); else OCC_G(0, 4); }
    else if (dt == STMOE_BF16) { if (mt == 1) OCC_G(1, 1); else OCC_G(1, 4); }
    else { if (mt == 1) OCC_G(2, 1); else OCC_G(2, 4); }
#undef OCC_G
    return n;
}
int occ_down(int dt, int mt)
{
    int n = 0;
#define OCC_D(DT, MT) n = occupancy_down<DT, MT>()
    if (dt == STMOE_F32) { if (mt == 1) OCC_D(0, 1); else OCC_D(0, 4); }
    else if (dt == STMOE_BF16) { if (mt == 1) OCC_D(1, 1); else OCC_D(1, 4); }
    else { if (mt == 1) OCC_D(2, 1); else OCC_D(2, 4); }
#undef OCC_D
    return n;
}

template <int DT, int MT> void *token_kernel_ptr(int rdt)
{
    return rdt == STMOE_F32 ? (void *)decode_token_kernel<DT, 0, MT> : (void *)decode_token_kernel<DT, 1, MT>;
}
void *token_kernel(int dt, int rdt, int mt)
{
    if (dt == STMOE_F32) return mt == 1 ? token_kernel_ptr<0, 1>(rdt) : token_kernel_ptr<0, 4>(rdt);
    if (dt == STMOE_BF16) return mt == 1 ? token_kernel_ptr<1, 1>(rdt) : token_kernel_ptr<1, 4>(rdt);
    return mt == 1 ? token_kernel_ptr<2, 1>(rdt) : token_kernel_ptr<2, 4>(rdt);
}
size_t token_smem(int B, int K, int n_shared) { return sizeof(int) * (size_t)(4 + 5 * B * (K + n_shared) + 3 * B * K); }

int sm_count()
{
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

FfnPlan make_plan(int dt, int mt)
{
    FfnPlan p;
    const int sms = sm_count();
    p.grid_gate_up = sms * std::max(1, std::min(occ_gate_up(dt, mt), 1));
    p.grid_down = sms * std::max(1, std::min(occ_down(dt, mt), 1));
    return p;
}

void launch_router_logits(int rdt, const float *h, const void *W, int B, int E, int H, float eps,
                          float *inv_rms, float *logits, cudaStream_t st)
{
    const int grid = (E + kRouterWarps - 1) / kRouterWarps;
    if (rdt == STMOE_F32)
        router_logits_kernel<0><<<grid, kRouterWarps * kWarp, 0, st>>>(h, (const uint8_t *)W, B, E, H, eps,
                                                                      inv_rms, logits);
    else
        router_logits_kernel<1><<<grid, kRouterWarps * kWarp, 0, st>>>(h, (const uint8_t *)W, B, E, H, eps,
                                                                      inv_rms, logits);
}

// ---- device work-list storage ----------------------------------------------------------
struct WorkListMem {
    int *base = nullptr;
    WorkList wl{};
    int alloc(int pairs)
    {
        CU_TRY(cudaMalloc(&base, sizeof(int) * (size_t)(4 + 5 * pairs)));
        bind(base, pairs);
        return STMOE_OK;
    }
    void bind(int *p, int pairs)
    {
        wl.n_groups = p;
        wl.g_expert = p + 4;
        wl.g_start = p + 4 + pairs;
        wl.g_count = p + 4 + 2 * pairs;
        wl.pair_token = p + 4 + 3 * pairs;
        wl.pair_slot = p + 4 + 4 * pairs;
    }
    void release()
    {
        if (base) cudaFree(base);
        base = nullptr;
    }
};

// ---- host-side slot cache (verification, miss loading, prefetch; Sections 4.1, 4.3.4) ---
// Victim order among the slots not protected in the current step: empty slots first, then the key
// with the fewest uses in its history window (W bits per key: routed at its layer's turn i decode
// steps ago), then (by_turn) the key whose layer's next turn is furthest away in the cyclic layer
// walk, then the least recently used on a clock that ticks once per layer step, then the lowest
// slot.  W = 0 without by_turn is plain LRU.  One ordered set per layer (uses, stamp, slot) makes a
// victim a walk over the layers' first unprotected entries; only the keys of the layer in progress
// change their use counts when its history shifts.
struct SlotCache {
    int64_t S = 0, clock = 0;
    int E = 0, L = 0, W = 0, floor = -1, cur_layer = 0;
    bool by_turn = false;
    std::vector<int32_t> slot_of, tag;
    std::vector<int64_t> stamp;
    std::vector<uint32_t> hist;
    std::vector<uint8_t> pf_unused, guard;
    typedef std::tuple<int, int64_t, int32_t> Key;  // (uses, stamp, slot)
    std::vector<std::set<Key>> by_layer;
    std::set<int32_t> empty;
    std::vector<int32_t> guarded;
    int64_t hits = 0, misses = 0, pf_issued = 0, pf_useful = 0, pf_wasted = 0, pf_dropped = 0,
            pf_resident = 0, tag_mismatches = 0;

    void init(int64_t slots, int layers, int experts)
    {
        S = slots, E = experts, L = layers, clock = 0;
        slot_of.assign((size_t)L * E, -1);
        tag.assign((size_t)S, -1);
        stamp.assign((size_t)S, -1);
        hist.assign((size_t)L * E, 0u);
        pf_unused.assign((size_t)S, 0);
        guard.assign((size_t)S, 0);
        by_layer.assign((size_t)L, std::set<Key>());
        empty.clear();
        guarded.clear();
        for (int32_t s = 0; s < S; ++s) empty.insert(s);
    }
    static int popcount(uint32_t v)
    {
        int n = 0;
        for (; v; v &= v - 1) ++n;
        return n;
    }
    Key key_of(int32_t s) const { return Key(popcount(hist[tag[s]]), stamp[s], s); }
    void protect(int32_t s)
    {
        if (!guard[s]) guard[s] = 1, guarded.push_back(s);
    }
    void unprotect_all()
    {
        for (int32_t s : guarded) guard[s] = 0;
        guarded.clear();
    }
    // a new turn of `layer`: its keys' histories shift by one
    void begin_step(int layer)
    {
        cur_layer = layer;
        const uint32_t mask = W >= 32 ? 0xffffffffu : ((1u << W) - 1u);
        for (int e = 0; e < E; ++e) {
            const int32_t key = layer * E + e;
            const uint32_t h = (hist[key] << 1) & mask;
            if (h == hist[key]) continue;
            const int32_t s = slot_of[key];
            if (s >= 0) by_layer[layer].erase(key_of(s));
            hist[key] = h;
            if (s >= 0) by_layer[layer].insert(key_of(s));
        }
    }
    // the routed key in slot s is used now
    void use(int32_t s)
    {
        const int layer = tag[s] / E;
        by_layer[layer].erase(key_of(s));
        if (W > 0) hist[tag[s]] |= 1u;
        stamp[s] = clock;
        by_layer[layer].insert(key_of(s));
    }
    int uses_of(int32_t s) const { return tag[s] < 0 ? -1 : popcount(hist[tag[s]]); }
    int32_t victim() const
    {
        if (!empty.empty()) return *empty.begin();
        bool have = false;
        Key best;
        int best_wait = 0;
        for (int m = 0; m < L; ++m) {
            auto it = by_layer[m].begin();
            while (it != by_layer[m].end() && guard[std::get<2>(*it)]) ++it;
            if (it == by_layer[m].end()) continue;
            int wait = 0;
            if (by_turn) {
                wait = (m - cur_layer) % L;
                if (wait < 0) wait += L;
                if (wait == 0) wait = L;
            }
            const Key &k = *it;
            const bool better = !have || std::get<0>(k) < std::get<0>(best) ||
                                (std::get<0>(k) == std::get<0>(best) &&
                                 (wait > best_wait ||
                                  (wait == best_wait && (std::get<1>(k) < std::get<1>(best) ||
                                                         (std::get<1>(k) == std::get<1>(best) && std::get<2>(k) < std::get<2>(best))))));
            if (better) best = k, best_wait = wait, have = true;
        }
        return have ? std::get<2>(best) : -1;
    }
    void place(int32_t s, int32_t key, bool by_prefetch)
    {
        if (tag[s] >= 0) {
            by_layer[tag[s] / E].erase(key_of(s));
            slot_of[tag[s]] = -1;
            if (pf_unused[s]) ++pf_wasted;
        } else {
            empty.erase(s);
        }
        tag[s] = key, slot_of[key] = s;
        if (!by_prefetch && W > 0) hist[key] |= 1u;
        pf_unused[s] = by_prefetch;
        stamp[s] = clock;
        by_layer[key / E].insert(key_of(s));
    }
};

struct TimedSpan {
    cudaEvent_t a, b;
    int kind;  // 0 transfer, 1 exposed wait, 2 gate/up kernel, 3 down kernel, 4 router kernel
};

}  // namespace

struct stmoe {
    stmoe_config_t cfg{};
    int rdt = 0;          // router dtype
    int KS = 0;           // K + n_shared
    int max_pred = 0;
    int S = 1;            // column splits of the down projection
    unsigned *d_err = nullptr;  // set by a kernel whose bounded wait ran out
    size_t img_bytes = 0;
    int next_layer = 0;
    int64_t host_t = 0;
    bool built = false;
    bool failed = false;  // a layer step broke off after the predictor had run: tables and counters are ahead of next_layer

    uint8_t *d_router = nullptr;    // [L][E][H]
    uint8_t *d_resident = nullptr;  // [L][E] images (resident stacks)
    uint8_t *d_shared = nullptr;    // [L][n_shared] images
    uint8_t *h_store = nullptr;     // pinned [L][E] images (offloaded stacks)
    uint8_t *d_slots = nullptr;     // [S] images
    const uint8_t **d_blob_table = nullptr;  // [L][E+n_shared] (resident) or [E+n_shared] (per step)
    const uint8_t **h_blob_table = nullptr;  // pinned staging of one step's table

    PredState pst{};
    float *d_rpart = nullptr, *d_sspart = nullptr;
    unsigned *d_arrivals = nullptr, *d_tile_done = nullptr;
    float *d_inv = nullptr, *d_logits = nullptr, *d_w = nullptr, *d_act = nullptr, *d_part = nullptr;
    int32_t *d_ids = nullptr;   // [L][B][K] routing of the current decode step
    int32_t *d_queue = nullptr; // [1 + 2E]
    // the routing and the prefetch queue of a layer step, written by the predictor kernel into pinned host
    // memory mapped on the device: [0] stamp of the step | ids | queue; h_ids / h_queue point into it
    int32_t *h_route = nullptr, *d_route = nullptr, *h_ids = nullptr, *h_queue = nullptr;
    int32_t route_seq = 0;
    WorkListMem wlm;
    FfnPlan plan1, plan4;

    cudaStream_t side_stream = nullptr;   // predictor kernels of resident stacks
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    bool side_pending = false;
    // one decode step of a resident stack captured as a CUDA graph, replayed while the
    // caller keeps passing the same buffers
    cudaGraphExec_t graph_exec = nullptr;
    const void *graph_key[9] = {};
    int64_t graph_launches = 0;
    int graph_captures = 0;
    bool graph_off = false;

    // persistent one-kernel decode step of resident stacks (token_kernel.cuh)
    bool persistent = false;
    int persistent_grid = 0;
    float *d_hbuf = nullptr, *d_rpart_all = nullptr, *d_sspart_all = nullptr, *d_act_all = nullptr, *d_part_all = nullptr;
    unsigned *d_tiles_all = nullptr, *d_barrier = nullptr;

    // single-sequence decode step with one streaming phase per layer (token_fused_kernel.cuh)
    bool fused = false;
    uint8_t *d_down_t = nullptr;            // transposed down projections, one per image
    size_t down_t_bytes = 0;
    float *d_zpart = nullptr;
    unsigned long long *d_acc = nullptr;
    int poll_limit = kBarrierSpinLimit;

    // tensor-core path for batched steps of resident bf16 stacks (dense_group.cuh)
    bool dense = false;
    int dense_min_batch = 0;
    CUtensorMap map_gate{}, map_up{}, map_down{}, map_x[4]{}, map_act[4]{};  // [np/16 - 1]
    __nv_bfloat16 *d_xb = nullptr, *d_actb = nullptr;
    float *d_part_dense = nullptr;
    int dense_grid = 0;
    bool dense8 = false;            // fp8 stacks: e4m3 weight tiles x three e5m2 activation planes
    CUtensorMap map8_gate{}, map8_up{}, map8_down{}, map8_x[4]{}, map8_act[4]{};
    uint8_t *d_x8 = nullptr, *d_act8 = nullptr;  // [3][64][H], [3][pairs + 64][I]
    float *d_host_io = nullptr;     // stmoe_decode_token_host: [2][max_batch][H] staging of h_in / h_out
    int32_t *d_host_ids = nullptr;  // and [L][max_batch][K] of the routed ids
    bool dense_persistent = false;  // one cooperative kernel per decode step (token_dense_kernel.cuh)
    unsigned *d_gu_done = nullptr;  // its per-entry gate/up completion counters, [L][E + n_shared]
    int dense_dyn_bytes = 0;

    // on-chip staging of the single-sequence persistent kernel (see ffn.cuh)
    long long stage_down_bytes = 0, stage_pred_bytes = 0;
    int stage_shared = 0;
    int prefetch_min_score = 0;  // queue entries below this summed score are not prefetched
    int host_wait_ms = kWaitTimeoutMs;     // limit of the host's wait for a layer's routing
    int throttle_chunk = 0, throttle_gap_us = 0;  // expert copies in chunks with idle gaps (0: whole images)
    int hook_drop_prefetch = 0, hook_fail_copy = 0, hook_delay_us = 0;  // host-side fault injection (tests)
    SlotCache cache;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_route = nullptr;
    std::vector<cudaEvent_t> slot_ready;  // last copy into each slot
    std::vector<uint8_t> slot_pending;
    std::deque<TimedSpan> spans;
    std::vector<cudaEvent_t> free_events;
    double transfer_ms = 0, exposed_ms = 0, gate_up_ms = 0, down_ms = 0, router_ms = 0;
    int64_t launches = 0, timed_ffn = 0;
    bool time_kernels = false;
    int64_t bytes_demand = 0, bytes_prefetch = 0;
};

namespace {

bool offloaded(const stmoe *s) { return s->cfg.cache_slots > 0; }

int get_event(stmoe *s, cudaEvent_t *ev)
{
    if (!s->free_events.empty()) {
        *ev = s->free_events.back();
        s->free_events.pop_back();
        return STMOE_OK;
    }
    CU_TRY(cudaEventCreate(ev));
    return STMOE_OK;
}

void harvest_spans(stmoe *s, bool all)
{
    while (!s->spans.empty()) {
        TimedSpan &sp = s->spans.front();
        if (all)
            cudaEventSynchronize(sp.b);
        else if (cudaEventQuery(sp.b) != cudaSuccess) {
            (void)cudaGetLastError();
            break;
        }
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, sp.a, sp.b) == cudaSuccess) {
            double *acc[5] = {&s->transfer_ms, &s->exposed_ms, &s->gate_up_ms, &s->down_ms, &s->router_ms};
            *acc[sp.kind] += ms;
        }
        s->free_events.push_back(sp.a);
        if (sp.kind != 2) s->free_events.push_back(sp.b);  // a gate/up span's end event starts the down span
        s->spans.pop_front();
    }
}

uint8_t *image_ptr(stmoe *s, int layer, int expert, bool shared)
{
    const stmoe_config_t &c = s->cfg;
    if (shared) return s->d_shared + ((size_t)layer * c.n_shared + expert) * s->img_bytes;
    if (offloaded(s)) return s->h_store + ((size_t)layer * c.n_experts + expert) * s->img_bytes;
    return s->d_resident + ((size_t)layer * c.n_experts + expert) * s->img_bytes;
}

int launch_predictor(stmoe *s, int layer, int batch, const int32_t *cur, const int32_t *prev,
                     int32_t *pred_ids, int32_t *n_pred, bool want_queue, cudaStream_t st)
{
    const stmoe_config_t &c = s->cfg;
    PredArgs a{};
    a.st = s->pst;
    a.L = c.n_layers, a.E = c.n_experts, a.K = c.top_k, a.P = c.profile_tokens;
    a.mode = c.predictor_mode, a.layer = layer, a.B = batch;
    a.cur = cur, a.prev = prev;
    a.pred_ids = pred_ids, a.n_pred = n_pred, a.max_pred = s->max_pred;
    a.queue = want_queue ? s->d_queue : nullptr;
    if (want_queue && s->d_route) {
        a.host_out = s->d_route, a.host_seq = ++s->route_seq;
        a.host_queue_off = (int)(s->h_queue - s->h_route);
    }
    predictor_step_kernel<<<1, 256, 0, st>>>(a);
    s->launches += 1;
    if (layer == c.n_layers - 1) {
        if (!s->built && s->host_t == c.profile_tokens - 1) {
            const int rows = (c.n_layers - 1) * c.n_experts;
            if (rows > 0)
                cct_build_kernel<<<(rows + 7) / 8, 256, 0, st>>>(s->pst, c.n_layers, c.n_experts, c.top_k);
            s->launches += rows > 0;
            s->built = true;
        }
        s->host_t += 1;
    }
    CU_TRY(cudaGetLastError());
    return STMOE_OK;
}

// Bounded idle time on a stream (copy throttle, injected delays): spins on the global timer.
__global__ void delay_kernel(long long ns)
{
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
    for (int i = 0; i < (1 << 22); ++i) {
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
        if ((long long)(t - t0) >= ns) break;
        __nanosleep(200);
    }
}

// One expert image host -> slot on the copy stream, whole or in throttled chunks.
int copy_image(stmoe *s, int32_t slot, const uint8_t *src)
{
    if (s->hook_fail_copy > 0 && --s->hook_fail_copy == 0) return STMOE_ERR_CUDA;  // injected failure
    if (s->hook_delay_us > 0) {
        delay_kernel<<<1, 1, 0, s->copy_stream>>>(std::min<long long>(s->hook_delay_us, 10000) * 1000ll);
        s->hook_delay_us = 0;
    }
    uint8_t *dst = s->d_slots + (size_t)slot * s->img_bytes;
    if (s->throttle_chunk <= 0) {
        CU_TRY(cudaMemcpyAsync(dst, src, s->img_bytes, cudaMemcpyHostToDevice, s->copy_stream));
    } else {
        for (size_t o = 0; o < s->img_bytes; o += (size_t)s->throttle_chunk) {
            const size_t n = std::min(s->img_bytes - o, (size_t)s->throttle_chunk);
            CU_TRY(cudaMemcpyAsync(dst + o, src + o, n, cudaMemcpyHostToDevice, s->copy_stream));
            if (s->throttle_gap_us > 0) delay_kernel<<<1, 1, 0, s->copy_stream>>>((long long)s->throttle_gap_us * 1000ll);
        }
    }
    CU_TRY(cudaEventRecord(s->slot_ready[slot], s->copy_stream));
    s->slot_pending[slot] = 1;
    return STMOE_OK;
}

// Verification, miss loading and prefetch for one layer step of an offloaded stack.
int cache_step(stmoe *s, int layer, int batch, cudaStream_t st)
{
    const stmoe_config_t &c = s->cfg;
    const int E = c.n_experts, K = c.top_k, L = c.n_layers;
    const int next = (layer + 1) % L;
    SlotCache &ch = s->cache;

    // this layer's routing and the prefetch queue: the predictor kernel has been enqueued and stamps
    // the mapped host block when they are there (bounded wait; no copy, no event)
    {
        const auto t0 = std::chrono::steady_clock::now();
        volatile int32_t *stamp = s->h_route;
        for (unsigned spins = 0; *stamp != s->route_seq; ++spins) {
            if ((spins & 1023u) == 1023u) {
                const cudaError_t q = cudaStreamQuery(st);
                if (q != cudaSuccess && q != cudaErrorNotReady) {
                    (void)cudaGetLastError();
                    return STMOE_ERR_CUDA;
                }
                if (std::chrono::steady_clock::now() - t0 > std::chrono::milliseconds(s->host_wait_ms))
                    return STMOE_ERR_TIMEOUT;
            }
        }
        std::atomic_thread_fence(std::memory_order_acquire);
    }
    harvest_spans(s, false);

    std::vector<uint8_t> routed(E, 0);
    for (int i = 0; i < batch * K; ++i) routed[s->h_ids[i]] = 1;

    // verify: hits and demand loads (ascending expert id)
    ch.begin_step(layer);
    ch.unprotect_all();
    for (int e = 0; e < E; ++e) {
        if (!routed[e]) continue;
        const int32_t key = layer * E + e, sl = ch.slot_of[key];
        if (sl >= 0 && ch.tag[sl] != key) {  // the slot does not hold what the table says: forget the entry, load again
            ch.slot_of[key] = -1;
            ++ch.tag_mismatches;
        } else if (sl >= 0) {
            ch.protect(sl);
        }
    }
    std::vector<cudaEvent_t> wait_on;
    bool any_copy = false;
    cudaEvent_t span_a = nullptr, span_b = nullptr;
    auto copy_into = [&](int32_t slot, int lyr, int e) -> int {
        if (!any_copy) {
            ST_TRY(get_event(s, &span_a));
            ST_TRY(get_event(s, &span_b));
            CU_TRY(cudaEventRecord(span_a, s->copy_stream));
            any_copy = true;
        }
        return copy_image(s, slot, image_ptr(s, lyr, e, false));
    };
    for (int e = 0; e < E; ++e) {
        if (!routed[e]) continue;
        const int32_t key = layer * E + e;
        int32_t slot = ch.slot_of[key];
        if (slot >= 0) {
            ++ch.hits;
            if (ch.pf_unused[slot]) ++ch.pf_useful, ch.pf_unused[slot] = 0;
            ch.use(slot);
        } else {
            slot = ch.victim();
            if (slot < 0) return STMOE_ERR_STATE;
            ++ch.misses;
            ch.place(slot, key, false);
            ch.protect(slot);
            ST_TRY(copy_into(slot, layer, e));
            s->bytes_demand += (int64_t)s->img_bytes;
        }
        if (s->slot_pending[slot]) {
            if (cudaEventQuery(s->slot_ready[slot]) != cudaSuccess) {
                (void)cudaGetLastError();
                wait_on.push_back(s->slot_ready[slot]);
            }
            s->slot_pending[slot] = 0;  // later steps on this stream are ordered behind the wait
        }
        s->h_blob_table[e] = s->d_slots + (size_t)slot * s->img_bytes;
    }
    for (int i = 0; i < c.n_shared; ++i) s->h_blob_table[E + i] = image_ptr(s, layer, i, true);
    CU_TRY(cudaMemcpyAsync(s->d_blob_table, s->h_blob_table, sizeof(void *) * (E + c.n_shared),
                           cudaMemcpyHostToDevice, st));
    if (!wait_on.empty()) {
        // event-fenced handoff: the FFN kernels of this step start only after the copies into
        // the slots they read have landed; the time they wait is the exposed transfer time
        TimedSpan w{};
        w.kind = 1;
        ST_TRY(get_event(s, &w.a));
        ST_TRY(get_event(s, &w.b));
        CU_TRY(cudaEventRecord(w.a, st));
        for (cudaEvent_t e : wait_on) CU_TRY(cudaStreamWaitEvent(st, e, 0));
        CU_TRY(cudaEventRecord(w.b, st));
        s->spans.push_back(w);
    }

    // prefetch the queued experts of the next layer (priority order)
    int nq = s->h_queue[0];
    while (nq > 0 && s->h_queue[1 + E + nq - 1] < s->prefetch_min_score) --nq;  // the queue is in score order
    for (int i = 0; i < nq; ++i) {
        const int32_t sl = ch.slot_of[(size_t)next * E + s->h_queue[1 + i]];
        if (sl >= 0) ch.protect(sl);
    }
    int issued = 0;
    for (int i = 0; i < nq; ++i) {
        const int f = s->h_queue[1 + i];
        const int32_t key = next * E + f;
        if (ch.slot_of[key] >= 0) {
            ++ch.pf_resident;
            continue;
        }
        int32_t slot = (c.prefetch_limit > 0 && issued >= c.prefetch_limit) ? -1 : ch.victim();
        if (slot >= 0 && ch.floor >= 0 && ch.uses_of(slot) > ch.floor) slot = -1;  // only slots without recent use
        if (slot >= 0 && s->hook_drop_prefetch > 0) --s->hook_drop_prefetch, slot = -1;  // injected: a lost request
        if (slot < 0) {
            ++ch.pf_dropped;
            continue;
        }
        ch.place(slot, key, true);
        ch.protect(slot);
        ++ch.pf_issued, ++issued;
        ST_TRY(copy_into(slot, next, f));
        s->bytes_prefetch += (int64_t)s->img_bytes;
    }
    if (any_copy) {
        CU_TRY(cudaEventRecord(span_b, s->copy_stream));
        s->spans.push_back(TimedSpan{span_a, span_b, 0});
    }
    ch.clock += 1;
    return STMOE_OK;
}

// ---- tensor-core path (dense_group.cuh) ---------------------------------------------------
constexpr int kDenseMinBatch = 2;   // bf16 stacks: measured ahead of the CUDA-core kernels from two sequences on
constexpr int kDense8MinBatch = 2;  // fp8 stacks
constexpr int kDenseMaxSplits = 4;
constexpr int kTokenDenseDynBytes = 220 * 1024;

bool use_dense(const stmoe *s, int batch) { return (s->dense || s->dense8) && batch >= s->dense_min_batch; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 tensor of `rank` dimensions (dims[0] innermost, strides in bytes for dims 1..), boxes of
// 64 columns x box_rows rows (x 1 image), 128-byte swizzle, zero fill outside
int encode_map(EncodeTiledFn fn, CUtensorMap *m, void *base, int rank, const cuuint64_t *dims,
               const cuuint64_t *strides, int box_rows, CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
               int box_cols = kDenseKStep)
{
    cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(m, dt, (cuuint32_t)rank, base, dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS
               ? STMOE_OK
               : STMOE_ERR_CUDA;
}

void *token_dense_kernel(int rdt, bool w8);
// first image the tensor maps of the tensor-core path cover
uint8_t *dense_store(const stmoe *s) { return offloaded(s) ? s->d_slots : s->d_resident; }

int dense_setup(stmoe *s)
{
    const stmoe_config_t &c = s->cfg;
    const int L = c.n_layers, E = c.n_experts, B = c.max_batch, H = c.hidden, I = c.inter;
    int dev = 0, major = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (major != 10) return STMOE_OK;  // tcgen05 kernels need sm_100: stay on the CUDA-core path
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qr) != cudaSuccess || !sym) {
        (void)cudaGetLastError();
        return STMOE_OK;
    }
    EncodeTiledFn enc = (EncodeTiledFn)sym;
    const size_t pairs = (size_t)B * s->KS;
    CU_TRY(cudaMalloc(&s->d_xb, sizeof(__nv_bfloat16) * (size_t)kDenseMaxTokens * H));
    CU_TRY(cudaMemset(s->d_xb, 0, sizeof(__nv_bfloat16) * (size_t)kDenseMaxTokens * H));
    CU_TRY(cudaMalloc(&s->d_actb, sizeof(__nv_bfloat16) * (pairs + kDenseMaxTokens) * I));
    CU_TRY(cudaMemset(s->d_actb, 0, sizeof(__nv_bfloat16) * (pairs + kDenseMaxTokens) * I));
    CU_TRY(cudaMalloc(&s->d_part_dense, sizeof(float) * pairs * kDenseMaxSplits * H));
    // the images the maps cover: the whole resident stack, or the slot store of an offloaded one
    uint8_t *store = dense_store(s);
    const cuuint64_t n_img = offloaded(s) ? (cuuint64_t)c.cache_slots : (cuuint64_t)L * (E + c.n_shared);
    const cuuint64_t gd[3] = {(cuuint64_t)H, (cuuint64_t)I, n_img}, gs[2] = {(cuuint64_t)H * 2, s->img_bytes};
    const cuuint64_t dd[3] = {(cuuint64_t)I, (cuuint64_t)H, n_img}, ds[2] = {(cuuint64_t)I * 2, s->img_bytes};
    ST_TRY(encode_map(enc, &s->map_gate, store, 3, gd, gs, kDenseRows));
    ST_TRY(encode_map(enc, &s->map_up, store + (size_t)I * H * 2, 3, gd, gs, kDenseRows));
    ST_TRY(encode_map(enc, &s->map_down, store + 2 * (size_t)I * H * 2, 3, dd, ds, kDenseRows));
    for (int i = 0; i < 4; ++i) {
        const cuuint64_t xd[2] = {(cuuint64_t)H, (cuuint64_t)kDenseMaxTokens}, xs[1] = {(cuuint64_t)H * 2};
        const cuuint64_t ad[2] = {(cuuint64_t)I, (cuuint64_t)(pairs + kDenseMaxTokens)}, as[1] = {(cuuint64_t)I * 2};
        ST_TRY(encode_map(enc, &s->map_x[i], s->d_xb, 2, xd, xs, 16 * (i + 1)));
        ST_TRY(encode_map(enc, &s->map_act[i], s->d_actb, 2, ad, as, 16 * (i + 1)));
    }
    CU_TRY(cudaFuncSetAttribute(dense_group_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGroupSmemBytes));
    CU_TRY(cudaFuncSetAttribute(dense_group_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGroupSmemBytes));
    s->dense_grid = sm_count();
    s->dense_min_batch = kDenseMinBatch;
    s->dense = true;
    if (s->persistent) {  // cooperative launches work and the per-layer buffers exist
        void *k = token_dense_kernel(s->rdt, false);
        const int np = (B + 15) / 16 * 16;
        const int slot = std::max(group_stage_bytes<1, 1>(np), group_stage_bytes<2, 1>(np));
        const int need = (int)token_smem(B, c.top_k, c.n_shared) + 1024 + slot;  // at least one stage
        int occ = 0;
        if (need <= kTokenDenseDynBytes &&
            cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kTokenDenseDynBytes) == cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k, kFfnThreads, kTokenDenseDynBytes) == cudaSuccess &&
            occ >= 1 &&
            cudaMalloc(&s->d_gu_done, sizeof(unsigned) * (size_t)L * (E + c.n_shared)) == cudaSuccess) {
            s->dense_persistent = true;
            s->dense_dyn_bytes = kTokenDenseDynBytes;
        }
        (void)cudaGetLastError();
    }
    return STMOE_OK;
}

// gate/up, down and the weighted sum of one layer step on the tensor-core kernels; the work
// list (one entry per expert) and inv_rms come from the router kernel launched before
int dense_down_splits(const stmoe *s, int batch, int *seg);

// fp8 stacks: tensor maps over the e4m3 images (128 x 128-byte boxes) and over the e5m2 planes of
// the activations (a plane after the other in the row dimension)
int dense8_setup(stmoe *s)
{
    const stmoe_config_t &c = s->cfg;
    const int L = c.n_layers, E = c.n_experts, B = c.max_batch, H = c.hidden, I = c.inter;
    int dev = 0, major = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (major != 10) return STMOE_OK;
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qr) != cudaSuccess || !sym) {
        (void)cudaGetLastError();
        return STMOE_OK;
    }
    EncodeTiledFn enc = (EncodeTiledFn)sym;
    const size_t pairs = (size_t)B * s->KS, act_rows = pairs + kDenseMaxTokens;
    CU_TRY(cudaMalloc(&s->d_x8, 3 * (size_t)kDenseMaxTokens * H));
    CU_TRY(cudaMemset(s->d_x8, 0, 3 * (size_t)kDenseMaxTokens * H));
    CU_TRY(cudaMalloc(&s->d_act8, 3 * act_rows * I));
    CU_TRY(cudaMemset(s->d_act8, 0, 3 * act_rows * I));
    CU_TRY(cudaMalloc(&s->d_part_dense, sizeof(float) * pairs * kDenseMaxSplits * H));
    uint8_t *store = dense_store(s);
    const cuuint64_t n_img = offloaded(s) ? (cuuint64_t)c.cache_slots : (cuuint64_t)L * (E + c.n_shared);
    const cuuint64_t gd[3] = {(cuuint64_t)H, (cuuint64_t)I, n_img}, gs[2] = {(cuuint64_t)H, s->img_bytes};
    const cuuint64_t dd[3] = {(cuuint64_t)I, (cuuint64_t)H, n_img}, ds[2] = {(cuuint64_t)I, s->img_bytes};
    const CUtensorMapDataType u8 = CU_TENSOR_MAP_DATA_TYPE_UINT8;
    constexpr int kCols = group_box_cols<2>();
    ST_TRY(encode_map(enc, &s->map8_gate, store, 3, gd, gs, kDenseRows, u8, kCols));
    ST_TRY(encode_map(enc, &s->map8_up, store + (size_t)I * H, 3, gd, gs, kDenseRows, u8, kCols));
    ST_TRY(encode_map(enc, &s->map8_down, store + 2 * (size_t)I * H, 3, dd, ds, kDenseRows, u8, kCols));
    for (int i = 0; i < 4; ++i) {
        const cuuint64_t xd[2] = {(cuuint64_t)H, (cuuint64_t)(3 * kDenseMaxTokens)}, xs[1] = {(cuuint64_t)H};
        const cuuint64_t ad[2] = {(cuuint64_t)I, (cuuint64_t)(3 * act_rows)}, as[1] = {(cuuint64_t)I};
        ST_TRY(encode_map(enc, &s->map8_x[i], s->d_x8, 2, xd, xs, 16 * (i + 1), u8, kCols));
        ST_TRY(encode_map(enc, &s->map8_act[i], s->d_act8, 2, ad, as, 16 * (i + 1), u8, kCols));
    }
    CU_TRY(cudaFuncSetAttribute(dense_group_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGroupSmemBytes));
    CU_TRY(cudaFuncSetAttribute(dense_group_kernel<1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGroupSmemBytes));
    s->dense_grid = sm_count();
    s->dense_min_batch = kDense8MinBatch;
    s->dense8 = true;
    if (s->persistent) {  // cooperative launches work and the per-layer buffers exist
        void *k = token_dense_kernel(s->rdt, true);
        const int np = (B + 15) / 16 * 16;
        const int slot = std::max(group_stage_bytes<1, 2>(np), group_stage_bytes<2, 2>(np));
        const int need = (int)token_smem(B, c.top_k, c.n_shared) + 1024 + slot;  // at least one stage
        int occ = 0;
        if (need <= kTokenDenseDynBytes &&
            cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kTokenDenseDynBytes) == cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k, kFfnThreads, kTokenDenseDynBytes) == cudaSuccess &&
            occ >= 1 &&
            cudaMalloc(&s->d_gu_done, sizeof(unsigned) * (size_t)L * (E + c.n_shared)) == cudaSuccess) {
            s->dense_persistent = true;
            s->dense_dyn_bytes = kTokenDenseDynBytes;
        }
        (void)cudaGetLastError();
    }
    return STMOE_OK;
}

int dense8_ffn(stmoe *s, int layer, int batch, bool chained, const FfnArgs &fa, cudaStream_t st)
{
    const stmoe_config_t &c = s->cfg;
    const int E = c.n_experts, H = c.hidden, I = c.inter, np = (batch + 15) / 16 * 16;
    cudaEvent_t e0 = nullptr, e1 = nullptr, e2 = nullptr;
    const bool timed = s->time_kernels;
    if (timed) {
        ST_TRY(get_event(s, &e0));
        ST_TRY(get_event(s, &e1));
        ST_TRY(get_event(s, &e2));
        CU_TRY(cudaEventRecord(e0, st));
    }
    if (!chained) {
        dense8_cast_kernel<<<std::min(s->dense_grid, (batch * H + 255) / 256), 256, 0, st>>>(fa.h, batch * H, H, s->d_x8);
        s->launches += 1;
    }
    GroupArgs g{};
    g.wl = fa.wl, g.E = E, g.img_routed0 = layer * E, g.img_shared0 = c.n_layers * E + layer * c.n_shared;
    g.np = np, g.KS = s->KS, g.inv_rms = fa.inv_rms, g.part = s->d_part_dense, g.err = s->d_err;
    g.store = dense_store(s), g.img_bytes = s->img_bytes, g.blob = offloaded(s) ? fa.blob : nullptr;
    g.act8 = s->d_act8, g.act_rows = batch * s->KS + kDenseMaxTokens;
    constexpr int kGu = group_kstage<2, 2>(), kDn = group_kstage<1, 2>();
    g.rows = I, g.kd = H, g.splits = 1, g.seg = (H + kGu - 1) / kGu * kGu;
    g.scale_off = 0, g.x_rows = kDenseMaxTokens;
    dense_group_kernel<2, 2><<<s->dense_grid, kGroupThreads, kGroupSmemBytes, st>>>(s->map8_gate, s->map8_up,
                                                                                    s->map8_x[np / 16 - 1], g);
    if (timed) CU_TRY(cudaEventRecord(e1, st));
    int seg = 0;
    int splits = dense_down_splits(s, batch, &seg);
    seg = (seg + kDn - 1) / kDn * kDn;
    splits = (I + seg - 1) / seg;
    g.rows = H, g.kd = I, g.splits = splits, g.seg = seg;
    g.scale_off = 2 * I, g.x_rows = g.act_rows;
    dense_group_kernel<1, 2><<<s->dense_grid, kGroupThreads, kGroupSmemBytes, st>>>(s->map8_down, s->map8_down,
                                                                                    s->map8_act[np / 16 - 1], g);
    FfnArgs fc = fa;
    fc.part = s->d_part_dense;
    dense8_combine_kernel<<<std::min(8 * s->dense_grid, (batch * H + 255) / 256), 256, 0, st>>>(fc, splits, s->d_x8);
    if (timed) {
        CU_TRY(cudaEventRecord(e2, st));
        s->spans.push_back(TimedSpan{e0, e1, 2});
        s->spans.push_back(TimedSpan{e1, e2, 3});
        s->timed_ffn += 1;
    }
    s->launches += 3;
    CU_TRY(cudaGetLastError());
    return STMOE_OK;
}

// chained: h_in is the output of the previous layer's dense_ffn, whose bf16 copy is still in d_xb
int dense_ffn(stmoe *s, int layer, int batch, bool chained, const FfnArgs &fa, cudaStream_t st)
{
    const stmoe_config_t &c = s->cfg;
    const int E = c.n_experts, H = c.hidden, I = c.inter, np = (batch + 15) / 16 * 16;
    cudaEvent_t e0 = nullptr, e1 = nullptr, e2 = nullptr;
    const bool timed = s->time_kernels;
    if (timed) {
        ST_TRY(get_event(s, &e0));
        ST_TRY(get_event(s, &e1));
        ST_TRY(get_event(s, &e2));
        CU_TRY(cudaEventRecord(e0, st));
    }
    if (!chained) {
        dense_cast_kernel<<<std::min(s->dense_grid, (batch * H + 255) / 256), 256, 0, st>>>(fa.h, nullptr, batch, batch, H, s->d_xb);
        s->launches += 1;
    }
    GroupArgs g{};
    g.wl = fa.wl, g.E = E, g.img_routed0 = layer * E, g.img_shared0 = c.n_layers * E + layer * c.n_shared;
    g.np = np, g.KS = s->KS, g.inv_rms = fa.inv_rms, g.act = s->d_actb, g.part = s->d_part_dense, g.err = s->d_err;
    g.store = dense_store(s), g.img_bytes = s->img_bytes, g.blob = offloaded(s) ? fa.blob : nullptr;
    g.rows = I, g.kd = H, g.splits = 1, g.seg = (H + group_kstage<2, 1>() - 1) / group_kstage<2, 1>() * group_kstage<2, 1>();
    dense_group_kernel<2, 1><<<s->dense_grid, kGroupThreads, kGroupSmemBytes, st>>>(s->map_gate, s->map_up,
                                                                                      s->map_x[np / 16 - 1], g);
    if (timed) CU_TRY(cudaEventRecord(e1, st));
    // down: split the reduction dimension until there are a few tasks per SM
    int seg = 0;
    const int splits = dense_down_splits(s, batch, &seg);
    const int tiles = (H + kDenseRows - 1) / kDenseRows;
    (void)tiles;
    g.rows = H, g.kd = I, g.splits = splits, g.seg = seg;
    dense_group_kernel<1, 1><<<s->dense_grid, kGroupThreads, kGroupSmemBytes, st>>>(s->map_down, s->map_down,
                                                                                      s->map_act[np / 16 - 1], g);
    FfnArgs fc = fa;
    fc.part = s->d_part_dense;
    dense_combine_kernel<<<std::min(8 * s->dense_grid, (batch * H + 255) / 256), 256, 0, st>>>(fc, splits, s->d_xb);
    if (timed) {
        CU_TRY(cudaEventRecord(e2, st));
        s->spans.push_back(TimedSpan{e0, e1, 2});
        s->spans.push_back(TimedSpan{e1, e2, 3});
        s->timed_ffn += 1;
    }
    s->launches += 3;
    CU_TRY(cudaGetLastError());
    return STMOE_OK;
}

int run_ffn(stmoe *s, int dt, int mt, const FfnPlan &plan, const FfnArgs &fa, cudaStream_t st)
{
    cudaEvent_t e0 = nullptr, e1 = nullptr, e2 = nullptr;
    const bool timed = s && s->time_kernels;
    if (timed) {
        ST_TRY(get_event(s, &e0));
        ST_TRY(get_event(s, &e1));
        ST_TRY(get_event(s, &e2));
        CU_TRY(cudaEventRecord(e0, st));
    }
    DISPATCH_DT_MT(dt, mt, launch_gate_up, fa, plan.grid_gate_up, st);
    if (timed) CU_TRY(cudaEventRecord(e1, st));
    DISPATCH_DT_MT(dt, mt, launch_down, fa, plan.grid_down, st);
    if (timed) {
        CU_TRY(cudaEventRecord(e2, st));
        s->spans.push_back(TimedSpan{e0, e1, 2});
        s->spans.push_back(TimedSpan{e1, e2, 3});
        s->timed_ffn += 1;
    }
    if (s) s->launches += 2;
    CU_TRY(cudaGetLastError());
    return STMOE_OK;
}

int layer_step(stmoe *s, int layer, int batch, const float *h_in, float *h_out, int32_t *routed_ids,
               float *routed_w, int32_t *predicted_ids, int32_t *n_predicted, uint32_t *flags,
               cudaStream_t st, bool chained = false)
{
    const stmoe_config_t &c = s->cfg;
    const int E = c.n_experts, K = c.top_k, H = c.hidden;
    const bool dense = use_dense(s, batch);
    const int mt = batch == 1 ? 1 : dense ? kDenseMaxTokens : 4;
    int32_t *ids = s->d_ids + (size_t)layer * c.max_batch * K;
    const int32_t *prev = layer > 0 ? s->d_ids + (size_t)(layer - 1) * c.max_batch * K : nullptr;

    cudaEvent_t er0 = nullptr, er1 = nullptr;
    if (s->time_kernels) {
        ST_TRY(get_event(s, &er0));
        ST_TRY(get_event(s, &er1));
        CU_TRY(cudaEventRecord(er0, st));
    }
    RouterArgs ra{};
    ra.h = h_in, ra.W = s->d_router + (size_t)layer * E * H * dtype_bytes(s->rdt), ra.H = H, ra.eps = c.rms_eps;
    ra.part = s->d_rpart, ra.ss_part = s->d_sspart, ra.arrivals = s->d_arrivals, ra.inv_rms = s->d_inv;
    TopkArgs &ta = ra.tk;
    ta.B = batch, ta.E = E, ta.K = K, ta.n_shared = c.n_shared, ta.mt = mt;
    ta.renorm = (c.flags & STMOE_FLAG_RENORM_TOPK) ? 1 : 0;
    ta.ids = ids, ta.w = s->d_w;
    ta.ids_out = routed_ids, ta.w_out = routed_w, ta.flags_out = flags;
    ta.near_tie_counter = s->pst.stats + 4;
    ta.wl = s->wlm.wl;
    {
        const int C = s->rdt == STMOE_F32 ? router_chunks<0>(H, batch) : router_chunks<1>(H, batch);
        const int threads = batch > 8 ? 512 : 256, nw = threads / kWarp;
        const int grid = std::min((E * C + nw - 1) / nw, 2 * s->plan1.grid_gate_up);
        if (s->rdt == STMOE_F32) {
            if (layer > 0 && !offloaded(s))
                launch_pdl(router_fused_kernel<0>, grid, threads, st, ra);
            else
                router_fused_kernel<0><<<grid, threads, 0, st>>>(ra);
        } else {
            if (layer > 0 && !offloaded(s))
                launch_pdl(router_fused_kernel<1>, grid, threads, st, ra);
            else
                router_fused_kernel<1><<<grid, threads, 0, st>>>(ra);
        }
    }
    CU_TRY(cudaGetLastError());
    if (s->time_kernels) {
        CU_TRY(cudaEventRecord(er1, st));
        s->spans.push_back(TimedSpan{er0, er1, 4});
    }
    if (offloaded(s))  // the host needs the prefetch queue before it can issue copies
        ST_TRY(launch_predictor(s, layer, batch, ids, prev, predicted_ids, n_predicted, true, st));

    FfnArgs fa{};
    fa.h = h_in, fa.inv_rms = s->d_inv, fa.wl = s->wlm.wl;
    fa.act = s->d_act, fa.part = s->d_part, fa.H = H, fa.I = c.inter, fa.E = E, fa.S = s->S;
    fa.w = s->d_w, fa.h_out = h_out, fa.tile_done = s->d_tile_done;
    fa.B = batch, fa.K = K, fa.n_shared = c.n_shared, fa.residual_scale = c.residual_scale;
    if (offloaded(s)) {
        ST_TRY(cache_step(s, layer, batch, st));
        fa.blob = s->d_blob_table;
    } else {
        fa.blob = s->d_blob_table + (size_t)layer * (E + c.n_shared);
    }
    s->launches += 1;
    if (dense && s->dense8)
        ST_TRY(dense8_ffn(s, layer, batch, chained, fa, st));
    else if (dense)
        ST_TRY(dense_ffn(s, layer, batch, chained, fa, st));
    else
        ST_TRY(run_ffn(s, c.weight_dtype, mt, mt == 1 ? s->plan1 : s->plan4, fa, st));
    if (!offloaded(s)) {
        // resident: nothing in the step depends on the predictor, so it runs on a side stream
        // once the FFN kernels (which fill every SM) are done, beside the next layer's router
        CU_TRY(cudaEventRecord(s->ev_fork, st));
        CU_TRY(cudaStreamWaitEvent(s->side_stream, s->ev_fork, 0));
        ST_TRY(launch_predictor(s, layer, batch, ids, prev, predicted_ids, n_predicted, false, s->side_stream));
        s->side_pending = true;
    }
    return STMOE_OK;
}

int join_side(stmoe *s, cudaStream_t st)
{
    if (!s->side_pending) return STMOE_OK;
    CU_TRY(cudaEventRecord(s->ev_join, s->side_stream));
    CU_TRY(cudaStreamWaitEvent(st, s->ev_join, 0));
    s->side_pending = false;
    return STMOE_OK;
}

int token_eager(stmoe *s, int batch, const float *h_in, float *h_out, int32_t *routed_ids, float *routed_w,
                int32_t *predicted_ids, int32_t *n_predicted, uint32_t *flags, cudaStream_t st)
{
    const int K = s->cfg.top_k;
    for (int l = 0; l < s->cfg.n_layers; ++l) {
        const size_t o = (size_t)l * batch;
        ST_TRY(layer_step(s, l, batch, l == 0 ? h_in : h_out, h_out, routed_ids ? routed_ids + o * K : nullptr,
                          routed_w ? routed_w + o * K : nullptr,
                          predicted_ids ? predicted_ids + o * s->max_pred : nullptr,
                          n_predicted ? n_predicted + o : nullptr, flags ? flags + o : nullptr, st, l > 0));
    }
    return join_side(s, st);
}

int token_persistent(stmoe *s, int batch, const float *h_in, float *h_out, int32_t *routed_ids, float *routed_w,
                     int32_t *predicted_ids, int32_t *n_predicted, uint32_t *flags, cudaStream_t st)
{
    const stmoe_config_t &c = s->cfg;
    TokenArgs a{};
    a.L = c.n_layers, a.B = batch, a.E = c.n_experts, a.K = c.top_k, a.n_shared = c.n_shared;
    a.H = c.hidden, a.I = c.inter, a.S = s->S, a.mt = batch == 1 ? 1 : 4;
    a.renorm = (c.flags & STMOE_FLAG_RENORM_TOPK) ? 1 : 0;
    a.eps = c.rms_eps, a.residual_scale = c.residual_scale;
    a.h_in = h_in, a.h_out = h_out, a.hbuf = s->d_hbuf;
    a.router = s->d_router, a.blob = s->d_blob_table;
    a.rpart = s->d_rpart_all, a.sspart = s->d_sspart_all, a.act = s->d_act_all, a.part = s->d_part_all;
    a.tile_done = s->d_tiles_all;
    a.ids_all = s->d_ids, a.Bmax = c.max_batch;
    a.ids_out = routed_ids, a.w_out = routed_w, a.flags_out = flags;
    a.pred_ids = predicted_ids, a.n_pred = n_predicted, a.max_pred = s->max_pred;
    a.pst = s->pst, a.P = c.profile_tokens, a.mode = c.predictor_mode;
    a.barrier = s->d_barrier, a.err = s->d_err;
    a.store = s->d_resident, a.img_bytes = s->img_bytes;
    a.stage_down_bytes = s->stage_down_bytes, a.stage_pred_bytes = s->stage_pred_bytes, a.stage_shared = s->stage_shared;
    CU_TRY(cudaMemsetAsync(s->d_barrier, 0, 4, st));
    void *args[] = {&a};
    CU_TRY(cudaLaunchCooperativeKernel(token_kernel(c.weight_dtype, s->rdt, a.mt), dim3(s->persistent_grid),
                                       dim3(kFfnThreads), args, token_smem(batch, c.top_k, c.n_shared), st));
    s->launches += 1;
    if (!s->built && s->host_t == c.profile_tokens - 1) {
        const int rows = (c.n_layers - 1) * c.n_experts;
        if (rows > 0) cct_build_kernel<<<(rows + 7) / 8, 256, 0, st>>>(s->pst, c.n_layers, c.n_experts, c.top_k);
        s->launches += rows > 0;
        s->built = true;
        CU_TRY(cudaGetLastError());
    }
    s->host_t += 1;
    return STMOE_OK;
}

void *token_fused_kernel(const stmoe_config_t &c)
{
    const int dt = c.weight_dtype;
    const int ch = fused_chunks(c.hidden, 16 / dtype_bytes(dt), c.inter, c.top_k, sm_count());
    if (dt == STMOE_F32) return ch == 2 ? (void *)decode_token_fused_kernel<0, 0, 2> : (void *)decode_token_fused_kernel<0, 0, 1>;
    if (dt == STMOE_BF16) return ch == 2 ? (void *)decode_token_fused_kernel<1, 1, 2> : (void *)decode_token_fused_kernel<1, 1, 1>;
    const int rows = fused_rows(c.hidden, 16 / dtype_bytes(dt), c.inter, c.top_k, sm_count(), ch);
    return rows == 4 ? (void *)decode_token_fused_kernel<2, 1, 1, 4> : (void *)decode_token_fused_kernel<2, 1, 1, 2>;
}

int token_fused(stmoe *s, const float *h_in, float *h_out, int32_t *routed_ids, float *routed_w,
                int32_t *predicted_ids, int32_t *n_predicted, uint32_t *flags, cudaStream_t st)
{
    const stmoe_config_t &c = s->cfg;
    FusedArgs f{};
    TokenArgs &a = f.t;
    a.L = c.n_layers, a.B = 1, a.E = c.n_experts, a.K = c.top_k, a.n_shared = c.n_shared;
    a.H = c.hidden, a.I = c.inter, a.S = 1, a.mt = 1;
    a.renorm = (c.flags & STMOE_FLAG_RENORM_TOPK) ? 1 : 0;
    a.eps = c.rms_eps, a.residual_scale = c.residual_scale;
    a.h_in = h_in, a.h_out = h_out;
    a.router = s->d_router;
    a.ids_all = s->d_ids, a.Bmax = c.max_batch;
    a.ids_out = routed_ids, a.w_out = routed_w, a.flags_out = flags;
    a.pred_ids = predicted_ids, a.n_pred = n_predicted, a.max_pred = s->max_pred;
    a.pst = s->pst, a.P = c.profile_tokens, a.mode = c.predictor_mode;
    a.barrier = s->d_barrier, a.err = s->d_err;
    a.store = s->d_resident, a.img_bytes = s->img_bytes;
    f.down_t = s->d_down_t, f.down_t_bytes = s->down_t_bytes;
    f.zpart = s->d_zpart, f.acc = s->d_acc, f.poll_limit = s->poll_limit;
    CU_TRY(cudaMemsetAsync(s->d_barrier, 0, 4, st));
    CU_TRY(cudaMemsetAsync(s->d_acc, 0, 8 * (size_t)c.n_layers * c.hidden, st));
    void *args[] = {&f};
    CU_TRY(cudaLaunchCooperativeKernel(token_fused_kernel(c), dim3(s->persistent_grid), dim3(kFfnThreads),
                                       args, (size_t)fused_smem_bytes(c.hidden), st));
    s->launches += 1;
    if (!s->built && s->host_t == c.profile_tokens - 1) {
        const int rows = (c.n_layers - 1) * c.n_experts;
        if (rows > 0) cct_build_kernel<<<(rows + 7) / 8, 256, 0, st>>>(s->pst, c.n_layers, c.n_experts, c.top_k);
        s->launches += rows > 0;
        s->built = true;
        CU_TRY(cudaGetLastError());
    }
    s->host_t += 1;
    return STMOE_OK;
}

void *token_dense_kernel(int rdt, bool w8)
{
    if (w8) return rdt == STMOE_F32 ? (void *)decode_token_dense_kernel<0, 2> : (void *)decode_token_dense_kernel<1, 2>;
    return rdt == STMOE_F32 ? (void *)decode_token_dense_kernel<0, 1> : (void *)decode_token_dense_kernel<1, 1>;
}

int dense_down_splits(const stmoe *s, int batch, int *seg)
{
    const stmoe_config_t &c = s->cfg;
    const int entries = std::min(c.n_experts, batch * c.top_k) + c.n_shared, tiles = (c.hidden + kDenseRows - 1) / kDenseRows;
    int splits = std::max(1, std::min(kDenseMaxSplits, (4 * s->dense_grid + entries * tiles - 1) / (entries * tiles)));
    *seg = ((c.inter + splits - 1) / splits + group_kstage<1, 1>() - 1) / group_kstage<1, 1>() * group_kstage<1, 1>();
    return (c.inter + *seg - 1) / *seg;  // no empty split
}

int token_dense(stmoe *s, int batch, const float *h_in, float *h_out, int32_t *routed_ids, float *routed_w,
                int32_t *predicted_ids, int32_t *n_predicted, uint32_t *flags, cudaStream_t st)
{
    const stmoe_config_t &c = s->cfg;
    TokenDenseArgs d{};
    TokenArgs &a = d.t;
    a.L = c.n_layers, a.B = batch, a.E = c.n_experts, a.K = c.top_k, a.n_shared = c.n_shared;
    a.H = c.hidden, a.I = c.inter, a.S = 1, a.mt = kDenseMaxTokens;
    a.renorm = (c.flags & STMOE_FLAG_RENORM_TOPK) ? 1 : 0;
    a.eps = c.rms_eps, a.residual_scale = c.residual_scale;
    a.h_in = h_in, a.h_out = h_out, a.hbuf = s->d_hbuf;
    a.router = s->d_router;
    a.rpart = s->d_rpart_all, a.sspart = s->d_sspart_all;
    a.ids_all = s->d_ids, a.Bmax = c.max_batch;
    a.ids_out = routed_ids, a.w_out = routed_w, a.flags_out = flags;
    a.pred_ids = predicted_ids, a.n_pred = n_predicted, a.max_pred = s->max_pred;
    a.pst = s->pst, a.P = c.profile_tokens, a.mode = c.predictor_mode;
    a.barrier = s->d_barrier, a.err = s->d_err;
    d.splits = dense_down_splits(s, batch, &d.seg);
    d.img_shared_base = c.n_layers * c.n_experts;
    d.dyn_bytes = s->dense_dyn_bytes;
    const bool w8 = s->dense8;
    d.xb = w8 ? (void *)s->d_x8 : (void *)s->d_xb, d.actb = w8 ? (void *)s->d_act8 : (void *)s->d_actb;
    d.part = s->d_part_dense, d.store = s->d_resident, d.img_bytes = s->img_bytes, d.gu_done = s->d_gu_done;
    if (w8) {  // a split is a whole number of the fp8 format's stages
        d.seg = (d.seg + group_kstage<1, 2>() - 1) / group_kstage<1, 2>() * group_kstage<1, 2>();
        d.splits = (c.inter + d.seg - 1) / d.seg;
    }
    const int np = (batch + 15) / 16 * 16;
    CU_TRY(cudaMemsetAsync(s->d_barrier, 0, 4, st));
    void *args_bf16[] = {&s->map_gate, &s->map_up, &s->map_down, &s->map_x[np / 16 - 1], &s->map_act[np / 16 - 1], &d};
    void *args_fp8[] = {&s->map8_gate, &s->map8_up, &s->map8_down, &s->map8_x[np / 16 - 1], &s->map8_act[np / 16 - 1], &d};
    void **args = w8 ? args_fp8 : args_bf16;
    void *k = token_dense_kernel(s->rdt, w8);
    CU_TRY(cudaLaunchCooperativeKernel(k, dim3(s->dense_grid), dim3(kFfnThreads), args, (size_t)s->dense_dyn_bytes, st));
    s->launches += 1;
    if (!s->built && s->host_t == c.profile_tokens - 1) {
        const int rows = (c.n_layers - 1) * c.n_experts;
        if (rows > 0) cct_build_kernel<<<(rows + 7) / 8, 256, 0, st>>>(s->pst, c.n_layers, c.n_experts, c.top_k);
        s->launches += rows > 0;
        s->built = true;
        CU_TRY(cudaGetLastError());
    }
    s->host_t += 1;
    return STMOE_OK;
}

size_t state_bytes(const stmoe_config_t &c)
{
    const size_t pairs = c.n_layers > 1 ? c.n_layers - 1 : 0;
    return 40 + pairs * c.n_experts * c.n_experts * 4 + 2 * pairs * c.n_experts * c.top_k +
           (size_t)c.max_batch * c.n_layers * c.top_k * 2;
}

}  // namespace

// ============================================================================== C ABI
extern "C" {

const char *stmoe_strerror(int code)
{
    switch (code) {
    case STMOE_OK: return "ok";
    case STMOE_ERR_BAD_ARG: return "bad argument";
    case STMOE_ERR_OOM: return "out of memory";
    case STMOE_ERR_CUDA: return "CUDA error";
    case STMOE_ERR_TIMEOUT: return "timed out waiting for the device";
    case STMOE_ERR_STATE: return "call out of order or inconsistent state";
    case STMOE_ERR_UNIMPLEMENTED: return "not implemented";
    case STMOE_ERR_TOO_LARGE: return "problem exceeds the capacity of the built-in scratch area";
    default: return "unknown error";
    }
}

int stmoe_destroy(stmoe_t *s)
{
    if (!s) return STMOE_OK;
    cudaDeviceSynchronize();
    harvest_spans(s, true);
    for (cudaEvent_t e : s->free_events) cudaEventDestroy(e);
    for (cudaEvent_t e : s->slot_ready) cudaEventDestroy(e);
    if (s->ev_route) cudaEventDestroy(s->ev_route);
    if (s->graph_exec) cudaGraphExecDestroy(s->graph_exec);
    if (s->ev_fork) cudaEventDestroy(s->ev_fork);
    if (s->ev_join) cudaEventDestroy(s->ev_join);
    if (s->side_stream) cudaStreamDestroy(s->side_stream);
    if (s->copy_stream) cudaStreamDestroy(s->copy_stream);
    void *dev[] = {s->d_router, s->d_resident, s->d_shared, s->d_slots, (void *)s->d_blob_table,
                   s->pst.Co, s->pst.cct_id, s->pst.cct_conf, s->pst.HT, s->pst.t, s->pst.pred_mask,
                   s->pst.pred_valid, s->pst.stats, s->d_rpart, s->d_sspart, s->d_arrivals, s->d_tile_done, s->d_hbuf, s->d_rpart_all, s->d_sspart_all,
                   s->d_act_all, s->d_part_all, s->d_tiles_all, s->d_barrier, s->d_err, s->d_inv, s->d_logits, s->d_w, s->d_act, s->d_part,
                   s->d_ids, s->d_queue, s->d_xb, s->d_actb, s->d_part_dense, s->d_x8, s->d_act8, s->d_host_io, s->d_host_ids, s->d_gu_done,
                   s->d_down_t, s->d_zpart, s->d_acc};
    if (s->d_shared && s->d_resident && s->d_shared > s->d_resident) dev[2] = nullptr;  // one allocation
    for (void *p : dev)
        if (p) cudaFree(p);
    s->wlm.release();
    void *host[] = {s->h_store, (void *)s->h_blob_table, s->h_route};
    for (void *p : host)
        if (p) cudaFreeHost(p);
    (void)cudaGetLastError();
    delete s;
    return STMOE_OK;
}

int stmoe_create(const stmoe_config_t *cfg, stmoe_t **out)
{
    if (!out) return STMOE_ERR_BAD_ARG;
    *out = nullptr;
    if (!cfg) return STMOE_ERR_BAD_ARG;
    const stmoe_config_t &c = *cfg;
    if (c.n_layers < 1 || c.n_experts < 1 || c.n_experts > kMaxExperts || c.top_k < 1 || c.top_k > kMaxTopK ||
        c.top_k > c.n_experts || c.n_shared < 0 || c.n_shared > 8 || c.hidden < 16 || c.hidden % 16 ||
        c.inter < 16 || c.inter % 16 || c.max_batch < 1 || c.max_batch > kMaxBatch ||
        c.weight_dtype < STMOE_F32 || c.weight_dtype > STMOE_FP8_E4M3 || c.cache_slots < 0 ||
        c.profile_tokens < 0 || c.predictor_mode < 0 || c.predictor_mode > 3 || c.prefetch_limit < 0 ||
        (c.cache_slots > 0 && c.cache_slots < (int64_t)c.max_batch * c.top_k) ||
        c.cache_slots > (int64_t)c.n_layers * c.n_experts)
        return STMOE_ERR_BAD_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
        (void)cudaGetLastError();
        return STMOE_ERR_CUDA;
    }
    stmoe *s = new (std::nothrow) stmoe();
    if (!s) return STMOE_ERR_OOM;
    s->cfg = c;
    s->rdt = c.weight_dtype == STMOE_F32 ? STMOE_F32 : STMOE_BF16;
    s->KS = c.top_k + c.n_shared;
    s->max_pred = std::min(c.n_experts, c.top_k * c.top_k + c.top_k);
    s->img_bytes = image_bytes(c.hidden, c.inter, c.weight_dtype);
    s->S = down_splits(c.inter, c.weight_dtype);
    const int L = c.n_layers, E = c.n_experts, K = c.top_k, B = c.max_batch, H = c.hidden, I = c.inter;
    const size_t pairs = L > 1 ? L - 1 : 0;

    auto fail = [&](int code) {
        stmoe_destroy(s);
        return code;
    };
#define CR_TRY(expr)                                                                       \
    do {                                                                                   \
        cudaError_t e_ = (expr);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            (void)cudaGetLastError();                                                      \
            return fail(e_ == cudaErrorMemoryAllocation ? STMOE_ERR_OOM : STMOE_ERR_CUDA); \
        }                                                                                  \
    } while (0)

    CR_TRY(cudaMalloc(&s->d_router, (size_t)L * E * H * dtype_bytes(s->rdt)));
    CR_TRY(cudaStreamCreateWithFlags(&s->side_stream, cudaStreamNonBlocking));
    CR_TRY(cudaEventCreateWithFlags(&s->ev_fork, cudaEventDisableTiming));
    CR_TRY(cudaEventCreateWithFlags(&s->ev_join, cudaEventDisableTiming));
    if (c.n_shared && c.cache_slots > 0) CR_TRY(cudaMalloc(&s->d_shared, (size_t)L * c.n_shared * s->img_bytes));
    if (c.cache_slots > 0) {
        CR_TRY(cudaHostAlloc(&s->h_store, (size_t)L * E * s->img_bytes, cudaHostAllocDefault));
        CR_TRY(cudaMalloc(&s->d_slots, (size_t)c.cache_slots * s->img_bytes));
        CR_TRY(cudaMalloc(&s->d_blob_table, sizeof(void *) * (E + c.n_shared)));
        CR_TRY(cudaHostAlloc(&s->h_blob_table, sizeof(void *) * (E + c.n_shared), cudaHostAllocDefault));
        CR_TRY(cudaHostAlloc(&s->h_route, sizeof(int32_t) * (1 + (size_t)B * K + 1 + 2 * E), cudaHostAllocMapped));
        memset(s->h_route, 0, sizeof(int32_t) * (1 + (size_t)B * K + 1 + 2 * E));
        CR_TRY(cudaHostGetDevicePointer((void **)&s->d_route, s->h_route, 0));
        s->h_ids = s->h_route + 1, s->h_queue = s->h_route + 1 + (size_t)B * K;
        CR_TRY(cudaStreamCreateWithFlags(&s->copy_stream, cudaStreamNonBlocking));
        CR_TRY(cudaEventCreateWithFlags(&s->ev_route, cudaEventDisableTiming));
        s->cache.init(c.cache_slots, L, E);
        // A decode step that can touch more (layer, expert) keys than there are slots walks the
        // cache in a cycle: use counts and the turn order decide there; otherwise plain LRU.
        if ((int64_t)L * std::min(E, B * K) > c.cache_slots) s->cache.W = 16, s->cache.by_turn = true;
        s->slot_ready.resize((size_t)c.cache_slots);
        s->slot_pending.assign((size_t)c.cache_slots, 0);
        for (auto &e : s->slot_ready) CR_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    } else {
        // routed images [L][E], then the shared ones [L][n_shared], in one allocation: one
        // tensor map with the image index as its outermost coordinate covers both
        CR_TRY(cudaMalloc(&s->d_resident, (size_t)L * (E + c.n_shared) * s->img_bytes));
        if (c.n_shared) s->d_shared = s->d_resident + (size_t)L * E * s->img_bytes;
        std::vector<const uint8_t *> tab((size_t)L * (E + c.n_shared));
        for (int l = 0; l < L; ++l) {
            for (int e = 0; e < E; ++e) tab[(size_t)l * (E + c.n_shared) + e] = image_ptr(s, l, e, false);
            for (int i = 0; i < c.n_shared; ++i) tab[(size_t)l * (E + c.n_shared) + E + i] = image_ptr(s, l, i, true);
        }
        CR_TRY(cudaMalloc(&s->d_blob_table, sizeof(void *) * tab.size()));
        CR_TRY(cudaMemcpy(s->d_blob_table, tab.data(), sizeof(void *) * tab.size(), cudaMemcpyHostToDevice));
    }
    s->pst.threshold = kThreshold;
    s->pst.live_counts = 0;
    CR_TRY(cudaMalloc(&s->pst.Co, std::max<size_t>(pairs * E * E * 4, 4)));
    CR_TRY(cudaMalloc(&s->pst.cct_id, std::max<size_t>(pairs * E * K, 4)));
    CR_TRY(cudaMalloc(&s->pst.cct_conf, std::max<size_t>(pairs * E * K, 4)));
    CR_TRY(cudaMalloc(&s->pst.HT, (size_t)B * L * K * 2));
    CR_TRY(cudaMalloc(&s->pst.t, 16));
    CR_TRY(cudaMalloc(&s->pst.pred_mask, (size_t)B * 8 * 4));
    CR_TRY(cudaMalloc(&s->pst.pred_valid, (size_t)B * 4));
    CR_TRY(cudaMalloc(&s->pst.stats, 8 * 8));
    CR_TRY(cudaMemset(s->pst.Co, 0, std::max<size_t>(pairs * E * E * 4, 4)));
    CR_TRY(cudaMemset(s->pst.cct_id, 0, std::max<size_t>(pairs * E * K, 4)));
    CR_TRY(cudaMemset(s->pst.cct_conf, 0, std::max<size_t>(pairs * E * K, 4)));
    CR_TRY(cudaMemset(s->pst.HT, 0xff, (size_t)B * L * K * 2));
    CR_TRY(cudaMemset(s->pst.t, 0, 16));
    CR_TRY(cudaMemset(s->pst.pred_mask, 0, (size_t)B * 8 * 4));
    CR_TRY(cudaMemset(s->pst.pred_valid, 0, (size_t)B * 4));
    CR_TRY(cudaMemset(s->pst.stats, 0, 8 * 8));
    CR_TRY(cudaMalloc(&s->d_err, 16));
    CR_TRY(cudaMemset(s->d_err, 0, 16));
    CR_TRY(cudaMalloc(&s->d_inv, sizeof(float) * B));
    CR_TRY(cudaMalloc(&s->d_logits, sizeof(float) * B * E));
    {
        const int C = s->rdt == STMOE_F32 ? router_chunks<0>(H, 2) : router_chunks<1>(H, 2);  // the finer chunking
        CR_TRY(cudaMalloc(&s->d_rpart, sizeof(float) * (size_t)C * B * E));
        CR_TRY(cudaMalloc(&s->d_sspart, sizeof(float) * (size_t)C * B));
        CR_TRY(cudaMalloc(&s->d_arrivals, 16));
        CR_TRY(cudaMemset(s->d_arrivals, 0, 16));
        CR_TRY(cudaMalloc(&s->d_tile_done, sizeof(unsigned) * ((H + kTileRows - 1) / kTileRows)));
        CR_TRY(cudaMemset(s->d_tile_done, 0, sizeof(unsigned) * ((H + kTileRows - 1) / kTileRows)));
    }
    CR_TRY(cudaMalloc(&s->d_w, sizeof(float) * B * K));
    CR_TRY(cudaMalloc(&s->d_act, sizeof(float) * (size_t)B * s->KS * I));
    CR_TRY(cudaMalloc(&s->d_part, sizeof(float) * (size_t)B * s->KS * s->S * H));
    CR_TRY(cudaMalloc(&s->d_ids, sizeof(int32_t) * (size_t)L * B * K));
    CR_TRY(cudaMalloc(&s->d_queue, sizeof(int32_t) * (1 + 2 * E)));
    CR_TRY(cudaMemset(s->d_queue, 0, sizeof(int32_t) * (1 + 2 * E)));
    if (s->wlm.alloc(B * s->KS) != STMOE_OK) return fail(STMOE_ERR_OOM);
    s->plan1 = make_plan(c.weight_dtype, 1);
    s->plan4 = make_plan(c.weight_dtype, 4);
    if (c.cache_slots == 0 && !(c.flags & STMOE_FLAG_NO_PERSISTENT)) {
        int dev = 0, coop = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        const size_t smem = token_smem(B, K, c.n_shared);
        bool ok = coop != 0 && smem <= 160 * 1024;
        for (int mt = 1; ok && mt <= 4; mt += 3) {
            void *k = token_kernel(c.weight_dtype, s->rdt, mt);
            int occ = 0;
            ok = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess &&
                 cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k, kFfnThreads, smem) == cudaSuccess && occ >= 1;
        }
        (void)cudaGetLastError();
        if (ok) {
            const size_t C = s->rdt == STMOE_F32 ? router_chunks<0>(H, 2) : router_chunks<1>(H, 2), tiles = (H + kTileRows - 1) / kTileRows, pairs = (size_t)B * s->KS;
            CR_TRY(cudaMalloc(&s->d_hbuf, sizeof(float) * (size_t)(L + 1) * B * H));
            CR_TRY(cudaMalloc(&s->d_rpart_all, sizeof(float) * L * C * B * E));
            CR_TRY(cudaMalloc(&s->d_sspart_all, sizeof(float) * L * C * B));
            CR_TRY(cudaMalloc(&s->d_act_all, sizeof(float) * L * pairs * I));
            CR_TRY(cudaMalloc(&s->d_part_all, sizeof(float) * L * pairs * s->S * H));
            CR_TRY(cudaMalloc(&s->d_tiles_all, sizeof(unsigned) * L * tiles));
            CR_TRY(cudaMemset(s->d_tiles_all, 0, sizeof(unsigned) * L * tiles));
            CR_TRY(cudaMalloc(&s->d_barrier, 16));
            s->persistent = true;
            s->persistent_grid = sm_count();
        }
    }
    if (s->persistent && !(c.flags & STMOE_FLAG_NO_FUSED) &&
        fused_shape_ok(H, 16 / dtype_bytes(c.weight_dtype))) {
        // a second, transposed copy of every down projection; if it does not fit the stack stays
        // on the three-phase kernel
        const size_t n_img = (size_t)L * (E + c.n_shared);
        s->down_t_bytes = (size_t)H * I * dtype_bytes(c.weight_dtype);
        int occ = 0;
        void *k = token_fused_kernel(c);
        if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, fused_smem_bytes(H)) == cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k, kFfnThreads, fused_smem_bytes(H)) == cudaSuccess && occ >= 1 &&
            cudaMalloc(&s->d_down_t, n_img * s->down_t_bytes) == cudaSuccess &&
            cudaMalloc(&s->d_zpart, sizeof(float) * (size_t)L * E) == cudaSuccess &&
            cudaMalloc(&s->d_acc, 8 * (size_t)L * H) == cudaSuccess) {
            s->fused = true;
        } else {
            (void)cudaGetLastError();
            if (s->d_down_t) cudaFree(s->d_down_t);
            if (s->d_zpart) cudaFree(s->d_zpart);
            if (s->d_acc) cudaFree(s->d_acc);
            s->d_down_t = nullptr, s->d_zpart = nullptr, s->d_acc = nullptr;
        }
    }
    // tensor-core FFN: resident stacks, and offloaded ones whose images all live in the slot store
    // (shared experts of an offloaded stack sit in an allocation of their own, outside the maps)
    const bool dense_ok = (c.cache_slots == 0 || c.n_shared == 0) && !(c.flags & STMOE_FLAG_NO_DENSE) && B >= 2;
    if (dense_ok && c.weight_dtype == STMOE_BF16) {
        const int rc = dense_setup(s);
        if (rc != STMOE_OK) return fail(rc);
    }
    if (dense_ok && c.weight_dtype == STMOE_FP8_E4M3) {
        const int rc = dense8_setup(s);
        if (rc != STMOE_OK) return fail(rc);
    }
    if (c.profile_tokens == 0 && L > 1) {
        const int rows = (L - 1) * E;
        cct_build_kernel<<<(rows + 7) / 8, 256>>>(s->pst, L, E, K);
        CR_TRY(cudaGetLastError());
    }
    s->built = c.profile_tokens == 0;
    CR_TRY(cudaDeviceSynchronize());
#undef CR_TRY
    *out = s;
    return STMOE_OK;
}

int stmoe_max_predicted(const stmoe_t *s) { return s ? s->max_pred : STMOE_ERR_BAD_ARG; }

int stmoe_set_kernel_timing(stmoe_t *s, int on)
{
    if (!s) return STMOE_ERR_BAD_ARG;
    s->time_kernels = on != 0;
    return STMOE_OK;
}

int stmoe_set_prefetch_min_score(stmoe_t *s, int min_score)
{
    if (!s || min_score < 0 || s->next_layer != 0) return STMOE_ERR_BAD_ARG;
    s->prefetch_min_score = min_score;
    return STMOE_OK;
}

int stmoe_selftest_bounded_wait(stmoe_t *s, int which, int poll_limit, void *cuda_stream)
{
    if (!s || which < 0 || which > 4 || poll_limit < 1 || poll_limit > (1 << 16)) return STMOE_ERR_BAD_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!s->d_barrier) CU_TRY(cudaMalloc(&s->d_barrier, 16));
    CU_TRY(cudaMemsetAsync(s->d_barrier, 0, 4, st));
    bounded_wait_selftest_kernel<<<2, 64, 0, st>>>(s->d_barrier, s->d_err, which, poll_limit);
    CU_TRY(cudaGetLastError());
    return STMOE_OK;
}

int stmoe_set_predict_threshold(stmoe_t *s, int threshold)
{
    if (!s || threshold < 1 || threshold > 255 || s->next_layer != 0) return STMOE_ERR_BAD_ARG;
    s->pst.threshold = threshold;
    if (s->graph_exec) cudaGraphExecDestroy(s->graph_exec), s->graph_exec = nullptr;  // captured kernels hold the old value
    memset(s->graph_key, 0, sizeof(s->graph_key));
    return STMOE_OK;
}

int stmoe_set_cache_policy(stmoe_t *s, int history_window, int by_turn, int prefetch_floor)
{
    if (!s || !offloaded(s) || history_window < 0 || history_window > 32 || prefetch_floor < -1 || s->next_layer != 0 ||
        s->cache.clock != 0 || (prefetch_floor >= 0 && history_window == 0))
        return STMOE_ERR_BAD_ARG;
    s->cache.W = history_window, s->cache.by_turn = by_turn != 0, s->cache.floor = prefetch_floor;
    return STMOE_OK;
}

int stmoe_set_copy_throttle(stmoe_t *s, int64_t chunk_bytes, int gap_us)
{
    if (!s || !offloaded(s) || chunk_bytes < 0 || chunk_bytes > (1ll << 30) || gap_us < 0 || gap_us > 10000 ||
        s->next_layer != 0)
        return STMOE_ERR_BAD_ARG;
    s->throttle_chunk = (int)chunk_bytes, s->throttle_gap_us = gap_us;
    return STMOE_OK;
}

int stmoe_test_hook(stmoe_t *s, int what, int64_t value)
{
    if (!s || value < 0 || s->next_layer != 0) return STMOE_ERR_BAD_ARG;
    if (what != STMOE_HOOK_POLL_LIMIT && !offloaded(s)) return STMOE_ERR_BAD_ARG;
    switch (what) {
    case STMOE_HOOK_DROP_PREFETCH: s->hook_drop_prefetch = (int)value; return STMOE_OK;
    case STMOE_HOOK_FAIL_COPY: s->hook_fail_copy = (int)value; return STMOE_OK;
    case STMOE_HOOK_DELAY_COPY_US: s->hook_delay_us = (int)std::min<int64_t>(value, 10000); return STMOE_OK;
    case STMOE_HOOK_CORRUPT_TAG:
        if (value >= s->cfg.cache_slots || s->cache.tag[(size_t)value] < 0) return STMOE_ERR_BAD_ARG;
        // the slot now claims another expert of the same layer (the table entry of the true key stays)
        {
            SlotCache &ch = s->cache;
            const int32_t sl = (int32_t)value, key = ch.tag[sl], layer = key / ch.E;
            ch.by_layer[layer].erase(ch.key_of(sl));
            ch.tag[sl] = layer * ch.E + (key % ch.E + 1) % ch.E;
            ch.by_layer[layer].insert(ch.key_of(sl));
        }
        return STMOE_OK;
    case STMOE_HOOK_HOST_WAIT_MS: s->host_wait_ms = (int)std::min<int64_t>(value, kWaitTimeoutMs); return STMOE_OK;
    case STMOE_HOOK_POLL_LIMIT: s->poll_limit = (int)std::min<int64_t>(std::max<int64_t>(value, 1), kBarrierSpinLimit); return STMOE_OK;
    default: return STMOE_ERR_BAD_ARG;
    }
}

int stmoe_set_onchip_staging(stmoe_t *s, int64_t known_bytes, int64_t predicted_bytes)
{
    if (!s || known_bytes < 0 || predicted_bytes < 0 || s->next_layer != 0) return STMOE_ERR_BAD_ARG;
    s->stage_shared = known_bytes > 0;
    s->stage_down_bytes = known_bytes;
    s->stage_pred_bytes = predicted_bytes;
    return STMOE_OK;
}

int stmoe_set_replacement_rule(stmoe_t *s, int live_counts)
{
    if (!s || s->next_layer != 0) return STMOE_ERR_BAD_ARG;
    s->pst.live_counts = live_counts != 0;
    if (s->graph_exec) cudaGraphExecDestroy(s->graph_exec), s->graph_exec = nullptr;  // captured kernels hold the old value
    memset(s->graph_key, 0, sizeof(s->graph_key));
    return STMOE_OK;
}

int stmoe_set_dense_min_batch(stmoe_t *s, int min_batch)
{
    if (!s || !(s->dense || s->dense8) || min_batch < 2 || s->next_layer != 0) return STMOE_ERR_BAD_ARG;
    s->dense_min_batch = min_batch;
    // a captured decode step holds the kernels of the path chosen at capture time: drop it so
    // the next step is captured again with the new threshold
    if (s->graph_exec) cudaGraphExecDestroy(s->graph_exec), s->graph_exec = nullptr;
    memset(s->graph_key, 0, sizeof(s->graph_key));
    return STMOE_OK;
}

int stmoe_load_router(stmoe_t *s, int layer, const void *w)
{
    if (!s || !w || layer < 0 || layer >= s->cfg.n_layers) return STMOE_ERR_BAD_ARG;
    const size_t n = (size_t)s->cfg.n_experts * s->cfg.hidden * dtype_bytes(s->rdt);
    CU_TRY(cudaMemcpy(s->d_router + (size_t)layer * n, w, n, cudaMemcpyDefault));
    return STMOE_OK;
}

int stmoe_load_experts(stmoe_t *s, int layer, int first_expert, int count, const void *gate, const void *up,
                       const void *down, const void *scales, int is_shared)
{
    if (!s || !gate || !up || !down || layer < 0 || layer >= s->cfg.n_layers || first_expert < 0 || count < 1)
        return STMOE_ERR_BAD_ARG;
    const stmoe_config_t &c = s->cfg;
    if (first_expert + count > (is_shared ? c.n_shared : c.n_experts)) return STMOE_ERR_BAD_ARG;
    if ((c.weight_dtype == STMOE_FP8_E4M3) != (scales != nullptr)) return STMOE_ERR_BAD_ARG;
    const int wb = dtype_bytes(c.weight_dtype);
    const size_t mat = (size_t)c.hidden * c.inter * wb, sc = 2 * (size_t)(2 * c.inter + c.hidden);
    for (int i = 0; i < count; ++i) {
        uint8_t *img = image_ptr(s, layer, first_expert + i, is_shared != 0);
        CU_TRY(cudaMemcpy(img + image_gate(c.hidden, c.inter, wb), (const uint8_t *)gate + i * mat, mat, cudaMemcpyDefault));
        CU_TRY(cudaMemcpy(img + image_up(c.hidden, c.inter, wb), (const uint8_t *)up + i * mat, mat, cudaMemcpyDefault));
        CU_TRY(cudaMemcpy(img + image_down(c.hidden, c.inter, wb), (const uint8_t *)down + i * mat, mat, cudaMemcpyDefault));
        if (scales)
            CU_TRY(cudaMemcpy(img + image_scales(c.hidden, c.inter, wb), (const uint8_t *)scales + i * sc, sc, cudaMemcpyDefault));
        if (s->fused) {  // W_d [H][I] -> [I][H] for the row-triple kernel
            const size_t idx = is_shared ? (size_t)c.n_layers * c.n_experts + (size_t)layer * c.n_shared + first_expert + i
                                         : (size_t)layer * c.n_experts + first_expert + i;
            const uint8_t *in = img + image_down(c.hidden, c.inter, wb);
            uint8_t *out = s->d_down_t + idx * s->down_t_bytes;
            const dim3 grid((c.inter + 31) / 32, (c.hidden + 31) / 32), block(32, 8);
            if (wb == 4) transpose_kernel<uint32_t><<<grid, block>>>((const uint32_t *)in, (uint32_t *)out, c.hidden, c.inter);
            else if (wb == 2) transpose_kernel<uint16_t><<<grid, block>>>((const uint16_t *)in, (uint16_t *)out, c.hidden, c.inter);
            else transpose_kernel<uint8_t><<<grid, block>>>(in, out, c.hidden, c.inter);
            CU_TRY(cudaGetLastError());
        }
    }
    if (s->fused) CU_TRY(cudaDeviceSynchronize());
    return STMOE_OK;
}

int stmoe_decode_step(stmoe_t *s, int layer, int batch, const float *h_in, float *h_out, int32_t *routed_ids,
                      float *routed_w, int32_t *predicted_ids, int32_t *n_predicted, uint32_t *flags,
                      void *cuda_stream)
{
    if (!s || !h_in || !h_out || batch < 1 || batch > s->cfg.max_batch || layer < 0 || layer >= s->cfg.n_layers)
        return STMOE_ERR_BAD_ARG;
    if (s->failed || layer != s->next_layer) return STMOE_ERR_STATE;
    int rc = layer_step(s, layer, batch, h_in, h_out, routed_ids, routed_w, predicted_ids, n_predicted,
                        flags, (cudaStream_t)cuda_stream);
    if (rc == STMOE_OK) rc = join_side(s, (cudaStream_t)cuda_stream);
    if (rc == STMOE_OK) s->next_layer = (layer + 1) % s->cfg.n_layers;
    else s->failed = true;  // Algorithm 3 and the history overwrite of this step may already have run
    return rc;
}

int stmoe_decode_token(stmoe_t *s, int batch, const float *h_in, float *h_out, int32_t *routed_ids,
                       float *routed_w, int32_t *predicted_ids, int32_t *n_predicted, uint32_t *flags,
                       void *cuda_stream)
{
    if (!s || !h_in || !h_out || batch < 1 || batch > s->cfg.max_batch) return STMOE_ERR_BAD_ARG;
    if (s->failed || s->next_layer != 0) return STMOE_ERR_STATE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const stmoe_config_t &c = s->cfg;
    const bool build_due = !s->built && s->host_t == c.profile_tokens - 1;
    if (s->dense_persistent && !s->time_kernels && use_dense(s, batch))
        return token_dense(s, batch, h_in, h_out, routed_ids, routed_w, predicted_ids, n_predicted, flags, st);
    if (s->fused && batch == 1 && !s->time_kernels)
        return token_fused(s, h_in, h_out, routed_ids, routed_w, predicted_ids, n_predicted, flags, st);
    if (s->persistent && !s->time_kernels && !use_dense(s, batch))
        return token_persistent(s, batch, h_in, h_out, routed_ids, routed_w, predicted_ids, n_predicted, flags, st);
    if (offloaded(s) || s->time_kernels || s->graph_off || build_due) {
        const int rc = token_eager(s, batch, h_in, h_out, routed_ids, routed_w, predicted_ids, n_predicted, flags, st);
        if (rc != STMOE_OK) s->failed = true;
        return rc;
    }

    const void *key[9] = {(const void *)(intptr_t)batch, h_in, h_out, routed_ids, routed_w, predicted_ids,
                          n_predicted, flags, st};
    if (s->graph_exec && memcmp(key, s->graph_key, sizeof(key)) == 0) {
        CU_TRY(cudaGraphLaunch(s->graph_exec, st));
        s->host_t += 1;
        s->launches += s->graph_launches;
        return STMOE_OK;
    }
    if (s->graph_captures >= 16) {  // the caller keeps changing buffers: stop re-capturing
        s->graph_off = true;
        return token_eager(s, batch, h_in, h_out, routed_ids, routed_w, predicted_ids, n_predicted, flags, st);
    }
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        (void)cudaGetLastError();  // e.g. the legacy default stream cannot be captured
        s->graph_off = true;
        return token_eager(s, batch, h_in, h_out, routed_ids, routed_w, predicted_ids, n_predicted, flags, st);
    }
    const int64_t before = s->launches;
    const int rc = token_eager(s, batch, h_in, h_out, routed_ids, routed_w, predicted_ids, n_predicted, flags, st);
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(st, &graph);
    if (rc != STMOE_OK || ce != cudaSuccess || !graph) {
        (void)cudaGetLastError();
        if (graph) cudaGraphDestroy(graph);
        s->graph_off = true;
        return rc != STMOE_OK ? rc : STMOE_ERR_CUDA;
    }
    if (s->graph_exec) cudaGraphExecDestroy(s->graph_exec), s->graph_exec = nullptr;
    const cudaError_t ie = cudaGraphInstantiate(&s->graph_exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ie != cudaSuccess) {
        (void)cudaGetLastError();
        s->graph_exec = nullptr, s->graph_off = true;
        return STMOE_ERR_CUDA;
    }
    memcpy(s->graph_key, key, sizeof(key));
    s->graph_launches = s->launches - before;
    s->graph_captures += 1;
    CU_TRY(cudaGraphLaunch(s->graph_exec, st));
    return STMOE_OK;
}

int stmoe_decode_token_host(stmoe_t *s, int batch, const float *h_in_host, float *h_out_host,
                            int32_t *routed_ids_host, void *cuda_stream)
{
    if (!s || !h_in_host || !h_out_host || batch < 1 || batch > s->cfg.max_batch) return STMOE_ERR_BAD_ARG;
    const stmoe_config_t &c = s->cfg;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t hb = sizeof(float) * (size_t)batch * c.hidden, plane = (size_t)c.max_batch * c.hidden;
    if (!s->d_host_io) {
        CU_TRY(cudaMalloc(&s->d_host_io, sizeof(float) * 2 * plane));
        CU_TRY(cudaMalloc(&s->d_host_ids, sizeof(int32_t) * (size_t)c.n_layers * c.max_batch * c.top_k));
    }
    float *d_in = s->d_host_io, *d_out = s->d_host_io + plane;
    CU_TRY(cudaMemcpyAsync(d_in, h_in_host, hb, cudaMemcpyHostToDevice, st));
    const int rc = stmoe_decode_token(s, batch, d_in, d_out, routed_ids_host ? s->d_host_ids : nullptr, nullptr, nullptr,
                                      nullptr, nullptr, cuda_stream);
    if (rc != STMOE_OK) return rc;
    CU_TRY(cudaMemcpyAsync(h_out_host, d_out, hb, cudaMemcpyDeviceToHost, st));
    if (routed_ids_host)
        CU_TRY(cudaMemcpyAsync(routed_ids_host, s->d_host_ids, sizeof(int32_t) * (size_t)c.n_layers * batch * c.top_k,
                               cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    return STMOE_OK;
}

int stmoe_stats(stmoe_t *s, stmoe_stats_t *out)
{
    if (!s || !out) return STMOE_ERR_BAD_ARG;
    CU_TRY(cudaDeviceSynchronize());
    harvest_spans(s, true);
    if (s->d_err) {
        unsigned err = 0;
        CU_TRY(cudaMemcpy(&err, s->d_err, 4, cudaMemcpyDeviceToHost));
        if (err) return STMOE_ERR_TIMEOUT;
    }
    unsigned long long st[8];
    long long t[2];
    CU_TRY(cudaMemcpy(st, s->pst.stats, sizeof(st), cudaMemcpyDeviceToHost));
    CU_TRY(cudaMemcpy(t, s->pst.t, sizeof(t), cudaMemcpyDeviceToHost));
    memset(out, 0, sizeof(*out));
    out->decode_steps = t[0];
    out->runtime_steps = (int64_t)st[0], out->routed = (int64_t)st[1];
    out->predicted = (int64_t)st[2], out->hits = (int64_t)st[3], out->near_ties = (int64_t)st[4];
    const SlotCache &ch = s->cache;
    out->cache_hits = ch.hits, out->cache_misses = ch.misses;
    out->prefetch_issued = ch.pf_issued, out->prefetch_useful = ch.pf_useful;
    out->prefetch_wasted = ch.pf_wasted, out->prefetch_dropped = ch.pf_dropped;
    out->prefetch_resident = ch.pf_resident;
    out->recovered_faults = ch.tag_mismatches;
    out->h2d_bytes_demand = s->bytes_demand, out->h2d_bytes_prefetch = s->bytes_prefetch;
    out->transfer_ms = s->transfer_ms, out->exposed_ms = s->exposed_ms;
    out->kernel_launches = s->launches, out->timed_ffn_launches = s->timed_ffn;
    out->gate_up_ms = s->gate_up_ms, out->down_ms = s->down_ms, out->router_ms = s->router_ms;
    return STMOE_OK;
}

int stmoe_export_state(stmoe_t *s, void *buf, size_t *bytes)
{
    if (!s || !bytes) return STMOE_ERR_BAD_ARG;
    const stmoe_config_t &c = s->cfg;
    const size_t need = state_bytes(c);
    if (!buf) {
        *bytes = need;
        return STMOE_OK;
    }
    if (*bytes < need) return STMOE_ERR_BAD_ARG;
    *bytes = need;
    CU_TRY(cudaDeviceSynchronize());
    const size_t pairs = c.n_layers > 1 ? c.n_layers - 1 : 0;
    uint8_t *o = (uint8_t *)buf;
    const int32_t hdr[8] = {(int32_t)kStateMagic, 1, c.n_layers, c.n_experts, c.top_k, c.max_batch,
                            c.profile_tokens, s->built ? 1 : 0};
    memcpy(o, hdr, 32), o += 32;
    CU_TRY(cudaMemcpy(o, s->pst.t, 8, cudaMemcpyDeviceToHost));
    o += 8;
    const size_t n_co = pairs * c.n_experts * c.n_experts * 4, n_cct = pairs * c.n_experts * c.top_k;
    if (n_co) CU_TRY(cudaMemcpy(o, s->pst.Co, n_co, cudaMemcpyDeviceToHost));
    o += n_co;
    if (n_cct) CU_TRY(cudaMemcpy(o, s->pst.cct_id, n_cct, cudaMemcpyDeviceToHost));
    o += n_cct;
    if (n_cct) CU_TRY(cudaMemcpy(o, s->pst.cct_conf, n_cct, cudaMemcpyDeviceToHost));
    o += n_cct;
    CU_TRY(cudaMemcpy(o, s->pst.HT, (size_t)c.max_batch * c.n_layers * c.top_k * 2, cudaMemcpyDeviceToHost));
    return STMOE_OK;
}

int stmoe_import_state(stmoe_t *s, const void *buf, size_t bytes)
{
    if (!s || !buf) return STMOE_ERR_BAD_ARG;
    const stmoe_config_t &c = s->cfg;
    if (bytes != state_bytes(c)) return STMOE_ERR_BAD_ARG;
    if (s->next_layer != 0 && !s->failed) return STMOE_ERR_STATE;
    const uint8_t *o = (const uint8_t *)buf;
    int32_t hdr[8];
    memcpy(hdr, o, 32), o += 32;
    if ((uint32_t)hdr[0] != kStateMagic || hdr[1] != 1 || hdr[2] != c.n_layers || hdr[3] != c.n_experts ||
        hdr[4] != c.top_k || hdr[5] != c.max_batch || hdr[6] != c.profile_tokens)
        return STMOE_ERR_BAD_ARG;
    CU_TRY(cudaDeviceSynchronize());
    long long t = 0;
    memcpy(&t, o, 8);
    CU_TRY(cudaMemcpy(s->pst.t, o, 8, cudaMemcpyHostToDevice));
    o += 8;
    const size_t pairs = c.n_layers > 1 ? c.n_layers - 1 : 0;
    const size_t n_co = pairs * c.n_experts * c.n_experts * 4, n_cct = pairs * c.n_experts * c.top_k;
    if (n_co) CU_TRY(cudaMemcpy(s->pst.Co, o, n_co, cudaMemcpyHostToDevice));
    o += n_co;
    if (n_cct) CU_TRY(cudaMemcpy(s->pst.cct_id, o, n_cct, cudaMemcpyHostToDevice));
    o += n_cct;
    if (n_cct) CU_TRY(cudaMemcpy(s->pst.cct_conf, o, n_cct, cudaMemcpyHostToDevice));
    o += n_cct;
    CU_TRY(cudaMemcpy(s->pst.HT, o, (size_t)c.max_batch * c.n_layers * c.top_k * 2, cudaMemcpyHostToDevice));
    CU_TRY(cudaMemset(s->pst.pred_valid, 0, (size_t)c.max_batch * 4));
    s->host_t = t;
    s->built = hdr[7] != 0;
    if (s->failed && offloaded(s)) {  // the slot table may be mid-step: start from an empty cache, same policy
        const int W = s->cache.W, floor = s->cache.floor;
        const bool by_turn = s->cache.by_turn;
        s->cache.init(c.cache_slots, c.n_layers, c.n_experts);
        s->cache.W = W, s->cache.floor = floor, s->cache.by_turn = by_turn;
        std::fill(s->slot_pending.begin(), s->slot_pending.end(), 0);
    }
    s->failed = false, s->next_layer = 0;  // the image is a state between decode steps
    return STMOE_OK;
}

int stmoe_export_cache_tags(stmoe_t *s, int32_t *tags, int64_t n)
{
    if (!s || !tags || n != s->cfg.cache_slots || n == 0) return STMOE_ERR_BAD_ARG;
    memcpy(tags, s->cache.tag.data(), sizeof(int32_t) * (size_t)n);
    return STMOE_OK;
}

int stmoe_router_topk(const float *h, const void *w_router, int wr_dtype, int batch, int n_experts, int hidden,
                      int top_k, float rms_eps, int renorm, float *logits, int32_t *ids, float *w,
                      uint32_t *flags, void *cuda_stream)
{
    if (!h || !w_router || !logits || !ids || !w || batch < 1 || batch > kMaxBatch || n_experts < 1 ||
        n_experts > kMaxExperts || top_k < 1 || top_k > kMaxTopK || top_k > n_experts || hidden < 16 ||
        hidden % 16 || (wr_dtype != STMOE_F32 && wr_dtype != STMOE_BF16))
        return STMOE_ERR_BAD_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float *inv = logits + (size_t)batch * n_experts;  // tail of the caller's buffer
    launch_router_logits(wr_dtype, h, w_router, batch, n_experts, hidden, rms_eps, inv, logits, st);
    TopkArgs ta{};
    ta.logits = logits;
    ta.B = batch, ta.E = n_experts, ta.K = top_k, ta.mt = 1, ta.renorm = renorm;
    ta.ids = ids, ta.w = w, ta.flags_out = flags;
    topk_group_kernel<<<1, 256, 0, st>>>(ta);
    CU_TRY(cudaGetLastError());
    return STMOE_OK;
}

int stmoe_predictor_step(stmoe_t *s, int layer, int batch, const int32_t *routed_ids, int32_t *predicted_ids,
                         int32_t *n_predicted, void *cuda_stream)
{
    if (!s || !routed_ids || batch < 1 || batch > s->cfg.max_batch || layer < 0 || layer >= s->cfg.n_layers)
        return STMOE_ERR_BAD_ARG;
    if (s->failed || layer != s->next_layer) return STMOE_ERR_STATE;
    const stmoe_config_t &c = s->cfg;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int32_t *ids = s->d_ids + (size_t)layer * c.max_batch * c.top_k;
    const int32_t *prev = layer > 0 ? s->d_ids + (size_t)(layer - 1) * c.max_batch * c.top_k : nullptr;
    CU_TRY(cudaMemcpyAsync(ids, routed_ids, sizeof(int32_t) * batch * c.top_k, cudaMemcpyDeviceToDevice, st));
    ST_TRY(launch_predictor(s, layer, batch, ids, prev, predicted_ids, n_predicted, true, st));
    s->next_layer = (layer + 1) % c.n_layers;
    return STMOE_OK;
}

size_t stmoe_expert_image_bytes(int hidden, int inter, int weight_dtype)
{
    return image_bytes(hidden, inter, weight_dtype);
}

// scratch layout: work list | blob table | act | part
static size_t ffn_scratch_layout(int B, int K, int H, int I, int E, int S, size_t *o_tab, size_t *o_act, size_t *o_part,
                                 size_t *o_tiles)
{
    size_t o = round_up(sizeof(int) * (4 + 5 * (size_t)B * K), 256);
    *o_tab = o, o += round_up(sizeof(void *) * (size_t)E, 256);
    *o_act = o, o += round_up(sizeof(float) * (size_t)B * K * I, 256);
    *o_part = o, o += round_up(sizeof(float) * (size_t)B * K * S * H, 256);
    *o_tiles = o, o += round_up(sizeof(unsigned) * (size_t)((H + kTileRows - 1) / kTileRows), 256);
    return o;
}

size_t stmoe_moe_ffn_scratch_bytes(int batch, int top_k, int hidden, int inter)
{
    size_t a, b, c, d;
    return ffn_scratch_layout(batch, top_k, hidden, inter, kMaxExperts, down_splits(inter, STMOE_F32), &a, &b, &c, &d);
}

}  // extern "C"

namespace {

// fills the work list and the expert-image table of a stand-alone FFN call from given routing
__global__ void __launch_bounds__(256)
group_given_ids_kernel(const int32_t *ids, int B, int E, int K, int mt, WorkList wl, const uint8_t *experts,
                       size_t img_bytes, const uint8_t **table, unsigned *tile_done, int n_tiles)
{
    for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) tile_done[i] = 0u;
    __shared__ int s_g[kMaxExperts + 1], s_p[kMaxExperts + 1];
    const int e = threadIdx.x;
    int cnt = 0;
    if (e < E)
        for (int i = 0; i < B * K; ++i) cnt += (ids[i] == e);
    s_g[e + 1] = (cnt + mt - 1) / mt, s_p[e + 1] = cnt;
    if (e == 0) s_g[0] = s_p[0] = 0;
    if (e < E) table[e] = experts + (size_t)e * img_bytes;
    __syncthreads();
    if (e == 0)
        for (int i = 1; i <= kMaxExperts; ++i) s_g[i] += s_g[i - 1], s_p[i] += s_p[i - 1];
    __syncthreads();
    if (e < E && cnt > 0) {
        for (int t = 0, g = s_g[e]; t < cnt; t += mt, ++g)
            wl.g_expert[g] = e, wl.g_start[g] = s_p[e] + t, wl.g_count[g] = min(mt, cnt - t);
        int n = 0;
        for (int i = 0; i < B * K; ++i)
            if (ids[i] == e) wl.pair_token[s_p[e] + n] = i / K, wl.pair_slot[s_p[e] + n] = i, ++n;
    }
    if (e == 0) *wl.n_groups = s_g[kMaxExperts];
}

}  // namespace

extern "C" int stmoe_moe_ffn(const float *h, const float *inv_rms, const int32_t *ids, const float *w,
                             const void *experts, int weight_dtype, int batch, int n_experts, int top_k,
                             int hidden, int inter, float residual_scale, float *h_out, void *scratch,
                             size_t scratch_bytes, void *cuda_stream)
{
    if (!h || !ids || !w || !experts || !h_out || !scratch || batch < 1 || batch > kMaxBatch || n_experts < 1 ||
        n_experts > kMaxExperts || top_k < 1 || top_k > kMaxTopK || top_k > n_experts || hidden < 16 ||
        hidden % 16 || inter < 16 || inter % 16 || weight_dtype < STMOE_F32 || weight_dtype > STMOE_FP8_E4M3 ||
        ((uintptr_t)scratch & 255))
        return STMOE_ERR_BAD_ARG;
    size_t o_tab, o_act, o_part, o_tiles;
    const int S = down_splits(inter, weight_dtype);
    if (scratch_bytes < ffn_scratch_layout(batch, top_k, hidden, inter, kMaxExperts, down_splits(inter, STMOE_F32), &o_tab, &o_act, &o_part, &o_tiles))
        return STMOE_ERR_BAD_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint8_t *sc = (uint8_t *)scratch;
    WorkListMem wlm;
    wlm.bind((int *)sc, batch * top_k);
    const int mt = batch == 1 ? 1 : 4;
    const uint8_t **table = (const uint8_t **)(sc + o_tab);
    group_given_ids_kernel<<<1, 256, 0, st>>>(ids, batch, n_experts, top_k, mt, wlm.wl, (const uint8_t *)experts,
                                             image_bytes(hidden, inter, weight_dtype), table,
                                             (unsigned *)(sc + o_tiles), (hidden + kTileRows - 1) / kTileRows);
    FfnArgs fa{};
    fa.h = h, fa.inv_rms = inv_rms, fa.wl = wlm.wl, fa.blob = table;
    fa.act = (float *)(sc + o_act), fa.part = (float *)(sc + o_part);
    fa.H = hidden, fa.I = inter, fa.E = n_experts, fa.S = S;
    fa.w = w, fa.h_out = h_out, fa.tile_done = (unsigned *)(sc + o_tiles);
    fa.B = batch, fa.K = top_k, fa.n_shared = 0, fa.residual_scale = residual_scale;
    // launch shapes per device ordinal (the SM count differs between devices); filled on first use,
    // and a repeated fill by a racing host thread writes the same values
    static FfnPlan plans[64][3][2];
    int dev = 0;
    CU_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return STMOE_ERR_BAD_ARG;
    FfnPlan &plan = plans[dev][weight_dtype][mt == 1 ? 0 : 1];
    if (plan.grid_down == 0) plan = make_plan(weight_dtype, mt);
    return run_ffn(nullptr, weight_dtype, mt, plan, fa, st);
}

// ---- allocation-free variant of stmoe_moe_ffn ---------------------------------------------
// Scratch for callers that may not allocate device memory lives in this library image: every
// GPU that loads the library holds these bytes until the process exits.
#define STMOE_STATIC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[STMOE_STATIC_SCRATCH_BYTES];
// Device address of g_static_scratch per device ordinal.  In host code the array's name is
// only a handle for the runtime, never a pointer a kernel may use, so the address is looked
// up once per device with that device current.
static void *g_static_scratch_ptr[64] = {};

extern "C" int stmoe_moe_ffn_static(const float *h, const float *inv_rms, const int32_t *ids, const float *w,
                                    const void *experts, int weight_dtype, int batch, int n_experts, int top_k,
                                    int hidden, int inter, float residual_scale, float *h_out, void *cuda_stream)
{
    // the same argument checks as stmoe_moe_ffn, before the capacity check, so that a malformed
    // call reads as a bad argument and the size below is computed from values in range
    if (!h || !ids || !w || !experts || !h_out || batch < 1 || batch > kMaxBatch || n_experts < 1 ||
        n_experts > kMaxExperts || top_k < 1 || top_k > kMaxTopK || top_k > n_experts || hidden < 16 ||
        hidden % 16 || inter < 16 || inter % 16 || weight_dtype < STMOE_F32 || weight_dtype > STMOE_FP8_E4M3)
        return STMOE_ERR_BAD_ARG;
    if (stmoe_moe_ffn_scratch_bytes(batch, top_k, hidden, inter) > (size_t)STMOE_STATIC_SCRATCH_BYTES)
        return STMOE_ERR_TOO_LARGE;
    int dev = -1;
    CU_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return STMOE_ERR_BAD_ARG;
    if (!g_static_scratch_ptr[dev]) {
        void *p = nullptr;
        CU_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        g_static_scratch_ptr[dev] = p;
    }
    return stmoe_moe_ffn(h, inv_rms, ids, w, experts, weight_dtype, batch, n_experts, top_k, hidden, inter,
                         residual_scale, h_out, g_static_scratch_ptr[dev], (size_t)STMOE_STATIC_SCRATCH_BYTES,
                         cuda_stream);
}

// ---- tensor-core expert FFN for many tokens of one expert ------------------------------------
static size_t dense_scratch_layout(int np, int H, int I, size_t *o_act)
{
    size_t o = round_up(sizeof(__nv_bfloat16) * (size_t)np * H, 256);
    *o_act = o, o += round_up(sizeof(__nv_bfloat16) * (size_t)np * I, 256);
    return o;
}

extern "C" size_t stmoe_expert_ffn_dense_scratch_bytes(int m, int hidden, int inter)
{
    if (m < 1 || m > kDenseMaxTokens || hidden < 1 || inter < 1) return 0;
    size_t o_act;
    return dense_scratch_layout((m + 15) / 16 * 16, hidden, inter, &o_act);
}

extern "C" int stmoe_expert_ffn_dense(const float *h, const float *inv_rms, const void *image, int m, int hidden,
                                      int inter, float *y, uint32_t *flags, void *scratch, size_t scratch_bytes,
                                      void *cuda_stream)
{
    if (!h || !image || !y || !flags || !scratch || m < 1 || m > kDenseMaxTokens || hidden < kDenseKStep ||
        hidden % kDenseKStep || inter < kDenseKStep || inter % kDenseKStep || ((uintptr_t)scratch & 255) ||
        ((uintptr_t)image & 15))
        return STMOE_ERR_BAD_ARG;
    const int np = (m + 15) / 16 * 16;
    size_t o_act;
    if (scratch_bytes < dense_scratch_layout(np, hidden, inter, &o_act)) return STMOE_ERR_BAD_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    __nv_bfloat16 *xb = (__nv_bfloat16 *)scratch, *act = (__nv_bfloat16 *)((uint8_t *)scratch + o_act);
    const __nv_bfloat16 *img = (const __nv_bfloat16 *)image;
    const int smem2 = kDenseStages * (2 * kDenseRows + np) * kDenseKStep * 2;
    const int smem1 = kDenseStages * (kDenseRows + np) * kDenseKStep * 2;
    static bool attr_set[64] = {};
    int dev = -1;
    CU_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return STMOE_ERR_BAD_ARG;
    if (!attr_set[dev]) {
        const int smem_max = kDenseStages * (2 * kDenseRows + kDenseMaxTokens) * kDenseKStep * 2;
        CU_TRY(cudaFuncSetAttribute(dense_ffn_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
        CU_TRY(cudaFuncSetAttribute(dense_ffn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
        attr_set[dev] = true;
    }
    dense_cast_kernel<<<148, 256, 0, st>>>(h, inv_rms, m, np, hidden, xb);
    DenseArgs gu{};
    gu.W0 = img, gu.W1 = img + (size_t)inter * hidden, gu.X = xb;
    gu.rows = inter, gu.kd = hidden, gu.m = m, gu.np = np, gu.act_out = act, gu.err = flags;
    dense_ffn_kernel<2><<<(inter + kDenseRows - 1) / kDenseRows, kDenseThreads, smem2, st>>>(gu);
    DenseArgs dn{};
    dn.W0 = img + 2 * (size_t)inter * hidden, dn.X = act;
    dn.rows = hidden, dn.kd = inter, dn.m = m, dn.np = np, dn.y_out = y, dn.err = flags;
    dense_ffn_kernel<1><<<(hidden + kDenseRows - 1) / kDenseRows, kDenseThreads, smem1, st>>>(dn);
    CU_TRY(cudaGetLastError());
    return STMOE_OK;
}
