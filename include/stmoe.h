/*
 * stmoe.h — C ABI of the B200 (sm_100a) decode-time MoE layer step with the
 * spatio-temporal expert predictor of ST-MoE.
 *
 * One layer step = gating network (RMSNorm, router GEMV, softmax, top-K;
 * Section 2) -> verification + table update (Algorithm 3) and prediction of
 * the next layer's experts (Algorithm 2, Eq. 1) -> miss loading and prefetch
 * of predicted experts from a pinned host store into fixed HBM slots
 * (Sections 4.1, 4.3.4) -> routed SwiGLU expert FFNs, probability-weighted
 * sum (Section 2) and the residual update of the stack harness.
 *
 * Conventions
 *   - Every function returns STMOE_OK (0) or a negative STMOE_ERR_* code; no
 *     exception, abort or output crosses this boundary.
 *   - "device" pointers are CUDA global memory of the device that was current
 *     in stmoe_create; "host" pointers are ordinary or pinned host memory.
 *   - load_* calls copy what they are given; the caller keeps its buffers.
 *     The library owns its weight storage, pinned host store, slot cache,
 *     copy stream, events and scratch.
 *   - cuda_stream arguments are cudaStream_t handles passed as void*.
 *   - There is no CPU fallback: without a CUDA device every call fails.
 */
#ifndef STMOE_H
#define STMOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define STMOE_OK 0
#define STMOE_ERR_BAD_ARG (-1)
#define STMOE_ERR_OOM (-2)
#define STMOE_ERR_CUDA (-3)
#define STMOE_ERR_TIMEOUT (-4)
#define STMOE_ERR_STATE (-5)
#define STMOE_ERR_UNIMPLEMENTED (-6)
#define STMOE_ERR_TOO_LARGE (-7)

/* weight_dtype */
#define STMOE_F32 0
#define STMOE_BF16 1
#define STMOE_FP8_E4M3 2 /* e4m3 codes + one bf16 scale per output channel */

/* predictor_mode: which sources feed Algorithm 2 (tables evolve identically) */
#define STMOE_PRED_OFF 0
#define STMOE_PRED_TEMPORAL 1 /* history table only            */
#define STMOE_PRED_SPATIAL 2  /* cross-layer table only        */
#define STMOE_PRED_ST 3       /* both, combined as in Eq. 1    */

/* flags */
#define STMOE_FLAG_RENORM_TOPK 1 /* divide the K gate weights by their sum (off: Section 2 uses
                                    the plain softmax probabilities) */

#define STMOE_FLAG_NO_PERSISTENT 2 /* resident stacks: decode steps as per-layer kernels (replayed as a
                                      CUDA graph) instead of the single persistent kernel */

#define STMOE_FLAG_NO_DENSE 4 /* never use the tensor-core FFN kernels: by default resident bf16 and fp8
                                stacks run decode steps of at least stmoe_set_dense_min_batch() sequences
                                (default 2) with one work-list entry per expert on tcgen05 tiles,
                                rounding the hidden state and the gated activations to bf16 (bf16
                                stacks) or to the sum of three e5m2 values (fp8 stacks, whose e4m3
                                weights are multiplied as stored): relative 2^-9 either way */

#define STMOE_FLAG_NO_FUSED 8 /* resident stacks, one sequence: by default stmoe_decode_token runs a kernel
                                that streams each expert's gate, up and (from a transposed copy made at
                                load time: one third more weight memory) down rows together, one
                                streaming phase and two grid barriers per layer; its sums are exact in
                                fixed point, so results are reproducible but differ in the last bits
                                from the three-phase kernels.  This flag keeps the three-phase kernel. */

/* per-sequence result flags of a layer step */
#define STMOE_TOKEN_NEAR_TIE 1u /* K-th and (K+1)-th router logit closer than 1e-4 */

typedef struct stmoe stmoe_t;

typedef struct {
    int32_t n_layers;
    int32_t n_experts;      /* routed experts per layer, <= 256 (8-bit ids in the CCT) */
    int32_t top_k;          /* K of the gating network = candidates per CCT row, <= 32 */
    int32_t n_shared;       /* always-on experts per layer (weight 1, not predicted)   */
    int32_t hidden;         /* H, multiple of 16                                       */
    int32_t inter;          /* I, multiple of 16                                       */
    int32_t max_batch;      /* sequences decoded together, <= 64                       */
    int32_t weight_dtype;   /* expert weights; the router is fp32 for STMOE_F32, else bf16 */
    int64_t cache_slots;    /* 0: all experts resident in HBM; else number of HBM expert
                               slots (>= max_batch*top_k), experts live in pinned host memory */
    int32_t profile_tokens; /* P of Algorithm 1: decode steps spent counting co-activations */
    int32_t predictor_mode;
    int32_t flags;
    int32_t prefetch_limit; /* max prefetch copies issued per layer step, 0 = no limit */
    float rms_eps;
    float residual_scale;   /* r in h' = h + r * MoE(RMSNorm(h))                       */
} stmoe_config_t;

typedef struct {
    int64_t decode_steps;     /* completed decode steps (one per pass over all layers)   */
    int64_t runtime_steps;    /* (layer, sequence) steps after profiling                  */
    int64_t routed;           /* experts routed in those steps                            */
    int64_t predicted;        /* experts predicted for those steps                        */
    int64_t hits;             /* routed experts that were in the predicted set            */
    int64_t near_ties;        /* sequences flagged STMOE_TOKEN_NEAR_TIE (all steps)       */
    int64_t cache_hits;       /* routed experts found in an HBM slot                      */
    int64_t cache_misses;     /* routed experts demand-loaded from the host store         */
    int64_t prefetch_issued;
    int64_t prefetch_useful;  /* prefetched experts used before eviction                  */
    int64_t prefetch_wasted;  /* prefetched experts evicted unused                        */
    int64_t prefetch_dropped; /* predictions not prefetched (no slot / over the limit)    */
    int64_t prefetch_resident;/* predictions already in a slot                            */
    int64_t h2d_bytes_demand;
    int64_t h2d_bytes_prefetch;
    double transfer_ms;       /* device time of all host->HBM expert copies               */
    double exposed_ms;        /* time the compute stream waited for such copies           */
    int64_t kernel_launches;  /* kernels launched by layer steps since creation           */
    int64_t timed_ffn_launches; /* layer steps whose FFN kernels were timed (see below)   */
    double gate_up_ms;        /* summed device time of the timed gate/up kernels          */
    double down_ms;           /* summed device time of the timed down kernels             */
    double router_ms;         /* summed device time of the timed router kernels           */
    int64_t recovered_faults; /* slot-table inconsistencies found at verification and repaired by a demand load */
} stmoe_stats_t;

/* Create a stack for the current CUDA device.  Allocates weight storage (HBM
 * for resident stacks, pinned host memory plus cache_slots HBM slots
 * otherwise), predictor tables (Co, CCT per adjacent layer pair, HT per layer
 * and sequence) and scratch.  *out is NULL on failure. */
int stmoe_create(const stmoe_config_t *cfg, stmoe_t **out);
int stmoe_destroy(stmoe_t *s);
const char *stmoe_strerror(int code);

/* Router matrix of one layer, [E][H] row-major (w_j of Section 2 in row j), fp32 for
 * STMOE_F32 stacks and bf16 otherwise.  w: host or device.  Synchronous. */
int stmoe_load_router(stmoe_t *s, int layer, const void *w);

/* Weights of experts first_expert .. first_expert+count-1 of one layer (is_shared: the
 * always-on experts).  gate, up: [count][I][H]; down: [count][H][I]; row-major in
 * weight_dtype.  scales (fp8 only, else NULL): [count][2I+H] bf16 = gate rows, up rows,
 * down rows.  Pointers may be host or device.  Synchronous: the sources are read during the call
 * (a device source must be complete: synchronise the stream that produced it first). */
int stmoe_load_experts(stmoe_t *s, int layer, int first_expert, int count, const void *gate,
                       const void *up, const void *down, const void *scales, int is_shared);

/* One layer step for `batch` sequences.  Layers must be called in order 0..L-1 for each
 * decode step (else STMOE_ERR_STATE).
 *   h_in, h_out    device fp32 [batch][H]; may alias
 *   routed_ids     device int32 [batch][K], ascending ids            (NULL: not returned)
 *   routed_w       device fp32  [batch][K], gate weights              (NULL: not returned)
 *   predicted_ids  device int32 [batch][max_pred], ascending ids of the prefetch set for
 *                  layer+1 (after the last layer: layer 0 of the next decode step), padded
 *                  with -1; max_pred = stmoe_max_predicted()          (NULL: not returned)
 *   n_predicted    device int32 [batch]                              (NULL: not returned)
 *   flags          device uint32 [batch], STMOE_TOKEN_*               (NULL: not returned)
 * Resident stacks: the call only enqueues work on cuda_stream.  Stacks with cache_slots > 0:
 * the call waits on the host (bounded, STMOE_ERR_TIMEOUT) for this layer's routing, issues
 * demand and prefetch copies on the library's copy stream and fences them with events.
 * Prediction never changes routing or output (Section 4.3.4).
 * A step that returns an error other than STMOE_ERR_BAD_ARG / STMOE_ERR_STATE may already have
 * applied Algorithm 3 and the history overwrite for this layer; the stack is then marked failed
 * and every further step returns STMOE_ERR_STATE until stmoe_import_state restores a consistent
 * image (retrying the layer would apply the update twice). */
int stmoe_decode_step(stmoe_t *s, int layer, int batch, const float *h_in, float *h_out,
                      int32_t *routed_ids, float *routed_w, int32_t *predicted_ids,
                      int32_t *n_predicted, uint32_t *flags, void *cuda_stream);

/* All layers of one decode step: h_out = stack(h_in).  The per-layer outputs are as in
 * stmoe_decode_step with a leading [n_layers] dimension; any of them may be NULL.  Resident
 * stacks run the whole step as one persistent cooperative kernel (one CTA per SM, bounded grid
 * barriers between the phases of a layer; a barrier that times out makes stmoe_stats return
 * STMOE_ERR_TIMEOUT). */
int stmoe_decode_token(stmoe_t *s, int batch, const float *h_in, float *h_out,
                       int32_t *routed_ids, float *routed_w, int32_t *predicted_ids,
                       int32_t *n_predicted, uint32_t *flags, void *cuda_stream);

/* stmoe_decode_token for callers whose buffers are in HOST memory (pinned for the copies to run
 * at link speed; pageable works): copies h_in_host [batch][H] to the device, runs the decode step,
 * copies h_out_host [batch][H] and, if not NULL, routed_ids_host [n_layers][batch][K] back, and
 * waits for cuda_stream.  The device staging buffers belong to the stack (allocated at the first
 * call).  Errors as stmoe_decode_token; a failed copy or wait returns STMOE_ERR_CUDA. */
int stmoe_decode_token_host(stmoe_t *s, int batch, const float *h_in_host, float *h_out_host,
                            int32_t *routed_ids_host, void *cuda_stream);

int stmoe_max_predicted(const stmoe_t *s); /* min(E, K*K+K) */

/* on != 0: bracket the expert-FFN kernels of every following layer step with CUDA events
 * on the caller's stream (the router kernel too); their summed durations appear in stmoe_stats.
 * Off by default. */
int stmoe_set_kernel_timing(stmoe_t *s, int on);

/* Offloaded stacks: prefetch only queue entries whose score (Eq. 1, summed over the batch's
 * sequences) is at least min_score; entries below it are ignored as if they had not been
 * predicted (they are neither copied nor protected from eviction).  0 (default) prefetches the
 * whole predicted set, the paper's policy; higher values trade recall for fewer wasted copies.
 * Between decode steps; routing, outputs and predictor tables are unaffected. */
int stmoe_set_prefetch_min_score(stmoe_t *s, int min_score);

/* Set threshold of Algorithm 2: an expert is predicted when its score (sum of the confidences of
 * its stored candidates in the routed experts' rows, plus binary 10 if it is in the history table,
 * Eq. 1) reaches `threshold`.  Section 4.2 fixes it at binary 10 = 2 (default); 1 predicts every
 * stored candidate of non-zero confidence, larger values trade recall for precision (threshold
 * sweep of the ablation).  Tables evolve identically for every value.  Between decode steps. */
int stmoe_set_predict_threshold(stmoe_t *s, int threshold);

/* Replacement rule of Algorithm 3.  When a stored candidate misses at confidence 0 the listing
 * replaces it by a routed expert the row does not hold and leaves open which.  live_counts = 0 (default): the
 * lowest such id; the co-activation counts stay as profiling (Algorithm 1) left them.
 * live_counts = 1: counting goes on at run time (for every sequence, in index order, the K x K
 * pairs of (previous layer's routing, this layer's routing) are counted right before that
 * sequence's table update) and the new candidate is the routed expert with the largest count in
 * the row, equal counts -> the lower id.  The exported state then carries the live counts.
 * Between decode steps. */
int stmoe_set_replacement_rule(stmoe_t *s, int live_counts);

/* Replacement policy of the HBM slot cache (the paper stages predicted experts and fetches
 * misses at once, Section 4.3.4, and names no replacement policy).  Victims are taken in this
 * order among the slots not needed by the step in progress: empty slots; the expert with the
 * fewest uses in its history window (history_window bits per expert: routed at its layer's turn i
 * decode steps ago; 0: not counted); with by_turn, the expert whose layer's next turn in the
 * cyclic layer walk is furthest away; the least recently used; the lowest slot.  0, 0 is plain
 * LRU.  prefetch_floor >= 0: a prefetch only takes a slot whose expert has at most that many uses
 * in its window (0: only slots without recent use), otherwise the prediction is dropped; -1: no
 * such test (every predicted expert is prefetched, the paper's behaviour).  A floor needs a
 * history window (history_window > 0), else STMOE_ERR_BAD_ARG.
 * Default: LRU when a decode step cannot touch more experts than there are slots
 * (n_layers * min(n_experts, max_batch * top_k) <= cache_slots), else a 16-step window with
 * by_turn (LRU has hit rate zero on a cyclic walk that is larger than the cache); floor -1.
 * Only before the first decode step of an offloaded stack. */
int stmoe_set_cache_policy(stmoe_t *s, int history_window, int by_turn, int prefetch_floor);

/* Bandwidth sensitivity (the paper's off-chip bandwidth axis): expert copies host -> HBM are issued
 * in chunks of chunk_bytes with gap_us of idle time on the copy stream after each, which lowers
 * the effective link speed to chunk_bytes / (chunk_bytes / link + gap_us).  0, 0: whole images at
 * full speed (default).  Offloaded stacks, between decode steps. */
int stmoe_set_copy_throttle(stmoe_t *s, int64_t chunk_bytes, int gap_us);

/* Host-side fault injection for tests (nothing here faults or hangs the GPU).  Offloaded stacks,
 * between decode steps:
 *   DROP_PREFETCH n   the next n prefetch requests are lost (counted as dropped); the experts
 *                     are demand-loaded if routed
 *   FAIL_COPY n       the n-th next expert copy reports failure: the layer step returns
 *                     STMOE_ERR_CUDA and the stack is failed until stmoe_import_state
 *   DELAY_COPY_US us  the next expert copy is preceded by us microseconds (<= 10000) of idle
 *                     time on the copy stream; the consuming kernels wait on the slot's event
 *   CORRUPT_TAG slot  the slot's tag is overwritten: verification finds the mismatch, reloads
 *                     the expert and counts it in recovered_faults
 *   HOST_WAIT_MS ms   limit of the host's wait for a layer's routing (default 20000); when it
 *                     runs out the step returns STMOE_ERR_TIMEOUT
 * Any stack: POLL_LIMIT n = polls after which a grid-barrier wait of the single-sequence
 * persistent kernel gives up (default 2^22). */
#define STMOE_HOOK_DROP_PREFETCH 1
#define STMOE_HOOK_FAIL_COPY 2
#define STMOE_HOOK_DELAY_COPY_US 3
#define STMOE_HOOK_CORRUPT_TAG 4
#define STMOE_HOOK_HOST_WAIT_MS 5
#define STMOE_HOOK_POLL_LIMIT 6
int stmoe_test_hook(stmoe_t *s, int what, int64_t value);

/* Runs the bounded waits of the persistent kernels on barriers that nobody completes, with a poll
 * limit of a few thousand: which = 0 the grid barrier of the three-phase kernel, 1 the grid barrier
 * of the single-sequence kernel, 2 an mbarrier wait of the tensor-core kernels, 3 the mbarrier wait
 * of the single-sequence kernel's copy ring, 4 the wait of the tensor-core kernel's down-projection
 * loads for an entry's gate/up tiles.  Each wait gives up, the stack's error word is set
 * and stmoe_stats returns STMOE_ERR_TIMEOUT from then on (destroy the stack afterwards); the
 * kernel itself ends normally.  Asynchronous on cuda_stream. */
int stmoe_selftest_bounded_wait(stmoe_t *s, int which, int poll_limit, void *cuda_stream);

/* On-chip staging in the single-sequence persistent decode step of resident stacks: the paper's
 * idea of fetching experts before they are needed (Sections 4.1, 4.3.4), one memory level down.
 * Weight rows are hinted into L2 while HBM would otherwise idle at a grid barrier; results never
 * depend on it (bit-identical on or off).
 *   known_bytes      weights whose addresses are already known: the down projection of the routed
 *                    experts (known since the top-K) ahead of the barrier in front of it, at most
 *                    known_bytes per expert and SM, and the next layer's shared experts ahead of
 *                    its router.  0 = off (default: measured neutral to slower, the phases
 *                    it overlaps with are not idle enough).
 *   predicted_bytes  per layer, summed over the GPU: leading gate/up rows of the experts in
 *                    Algorithm 2's prefetch set for the next layer, hinted ahead of that layer's
 *                    router and top-K.  0 = off (default).
 * Between decode steps. */
int stmoe_set_onchip_staging(stmoe_t *s, int64_t known_bytes, int64_t predicted_bytes);

/* Smallest batch that takes the tensor-core FFN path (see STMOE_FLAG_NO_DENSE); between decode
 * steps.  min_batch < 2 or a stack without that path: STMOE_ERR_BAD_ARG. */
int stmoe_set_dense_min_batch(stmoe_t *s, int min_batch);

/* Counters and timings; synchronises the device. */
int stmoe_stats(stmoe_t *s, stmoe_stats_t *out);

/* Predictor tables as a canonical image: 8 int32 {magic 0x53544D50, version 1, L, E, K, B, P,
 * built}, int64 decode steps, Co u32 [L-1][E][E], CCT ids u8 [L-1][E][K], CCT confidences u8
 * [L-1][E][K], HT i16 [B][L][K] (-1 = empty).  buf == NULL: only *bytes is set.  Host buffer.
 * Synchronises the device.  import restores such an image between decode steps. */
int stmoe_export_state(stmoe_t *s, void *buf, size_t *bytes);
int stmoe_import_state(stmoe_t *s, const void *buf, size_t bytes);

/* tags[slot] = layer*E+expert held by each HBM slot, -1 if empty (host int32 [cache_slots]). */
int stmoe_export_cache_tags(stmoe_t *s, int32_t *tags, int64_t n);

/* ---- single kernels behind the step, exposed for testing and reuse -------------------- */

/* Gating network of Section 2 for `batch` tokens: x = RMSNorm(h), z = W_r x, s = softmax(z),
 * top-K by logit (ties: lower id), ids ascending, w = s[ids].  All pointers device.
 * wr_dtype: STMOE_F32 or STMOE_BF16.  logits: fp32 [batch*E + batch]; receives the logits
 * [batch][E] followed by the per-sequence factors 1/sqrt(mean(h^2)+eps). */
int stmoe_router_topk(const float *h, const void *w_router, int wr_dtype, int batch, int n_experts,
                      int hidden, int top_k, float rms_eps, int renorm, float *logits,
                      int32_t *ids, float *w, uint32_t *flags, void *cuda_stream);

/* Predictor only (Algorithms 1-3 on the stack's tables) driven by given routing:
 * routed_ids device int32 [batch][K] ascending.  Same ordering rules and outputs as
 * stmoe_decode_step; used to replay routing traces. */
int stmoe_predictor_step(stmoe_t *s, int layer, int batch, const int32_t *routed_ids,
                         int32_t *predicted_ids, int32_t *n_predicted, void *cuda_stream);

/* Routed SwiGLU expert FFN, weighted sum and residual for given routing:
 *   h_out[b] = h[b] + r * sum_k w[b][k] * W_d^e ( silu(W_g^e x_b) * (W_u^e x_b) ),
 *   x_b = h[b] * inv_rms[b],  e = ids[b][k].
 * experts: device array of n_experts expert images, each `stmoe_expert_image_bytes` long:
 * gate [I][H], up [I][H], down [H][I], then (fp8) bf16 scales [2I+H].
 * scratch: device, stmoe_moe_ffn_scratch_bytes(batch, top_k, hidden, inter) bytes,
 * 256-byte aligned; contents need not be initialised. */
size_t stmoe_expert_image_bytes(int hidden, int inter, int weight_dtype);
size_t stmoe_moe_ffn_scratch_bytes(int batch, int top_k, int hidden, int inter);
int stmoe_moe_ffn(const float *h, const float *inv_rms, const int32_t *ids, const float *w,
                  const void *experts, int weight_dtype, int batch, int n_experts, int top_k,
                  int hidden, int inter, float residual_scale, float *h_out, void *scratch,
                  size_t scratch_bytes, void *cuda_stream);

/* stmoe_moe_ffn without a scratch argument and without any allocation (the paper has no
 * counterpart; this serves hosts, not the method).  For callers that must not allocate device
 * memory once they are running: serving loops where cudaMalloc could stall the device or fail
 * because a framework already owns all of HBM, and plug-in hosts that forbid allocator calls.
 * The work list, activations and partial sums live in an 8 MiB area built into the library
 * image; each GPU that loads the library holds those 8 MiB until the process exits.
 *   - Same arguments, layout and results as stmoe_moe_ffn; inputs and outputs stay with the
 *     caller.  Calls no cudaMalloc/cudaFree or other allocating routine.
 *   - Returns STMOE_ERR_TOO_LARGE when stmoe_moe_ffn_scratch_bytes(batch, top_k, hidden, inter)
 *     exceeds 8 MiB (for example batch 64, top_k 8, hidden 4096, inter 14336).
 *   - The first call on each device looks up the area's device address (with that device
 *     current); make that first call before starting any stream capture, and from one host
 *     thread (later calls may come from any thread).
 *   - Arguments out of range are STMOE_ERR_BAD_ARG, as in stmoe_moe_ffn; only a well-formed
 *     problem that does not fit is STMOE_ERR_TOO_LARGE.
 *   - All calls on a device share the one area, which keeps whatever the last call left; the
 *     call clears the counters that must start at zero itself.  Two calls whose kernels can
 *     overlap on the GPU (different streams, no ordering between them) race on it: order
 *     them, or use stmoe_moe_ffn with separate scratch buffers. */
int stmoe_moe_ffn_static(const float *h, const float *inv_rms, const int32_t *ids, const float *w,
                         const void *experts, int weight_dtype, int batch, int n_experts, int top_k,
                         int hidden, int inter, float residual_scale, float *h_out, void *cuda_stream);

/* One expert's SwiGLU FFN (Section 2: the expert network of a routed token) for m tokens that
 * share the expert, as bf16 tensor-core GEMMs (tcgen05.mma, accumulators in tensor memory):
 *   y[t] = W_d ( bf16( silu(W_g x_t) * (W_u x_t) ) ),  x_t = bf16( h[t] * inv_rms[t] ),
 * products exact, sums in fp32.  This is the regime where the per-expert token count makes the
 * FFN a real dense contraction; the decode step itself streams weights through the CUDA cores.
 *   h        device fp32 [m][hidden]; inv_rms device fp32 [m] or NULL (= 1).
 *   image    device, one STMOE_BF16 expert image (gate [I][H], up [I][H], down [H][I]).
 *   y        device fp32 [m][hidden], overwritten.
 *   flags    device uint32, caller-zeroed; set to 1 when a bounded wait inside a kernel ran out
 *            (y is then undefined).
 *   scratch  device, stmoe_expert_ffn_dense_scratch_bytes(m, hidden, inter) bytes, 256-byte
 *            aligned, contents need not be initialised.
 * m in 1..64; hidden and inter multiples of 64; else STMOE_ERR_BAD_ARG.  Asynchronous on
 * cuda_stream. */
size_t stmoe_expert_ffn_dense_scratch_bytes(int m, int hidden, int inter);
int stmoe_expert_ffn_dense(const float *h, const float *inv_rms, const void *image, int m, int hidden,
                           int inter, float *y, uint32_t *flags, void *scratch, size_t scratch_bytes,
                           void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* STMOE_H */
