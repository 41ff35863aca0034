/*
 * CPU oracle for the decode-time MoE layer step of ST-MoE.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow and meant to be checked against the
 * paper by eye.  Nothing in the CUDA product path includes, links or calls
 * this file, and this file shares no code with it.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg load the library built from it.
 *
 * Values are stored as fp32; every sum is accumulated in fp64 and rounded
 * once, so results do not depend on summation order.  The predictor and the
 * cache model are integer only.
 *
 * What each part follows:
 *   router, softmax, top-K, weighted expert sum ... Section 2 (gating network)
 *   co-activation counting and CCT construction .. Algorithm 1
 *   expert prediction ............................ Algorithm 2 and Eq. 1
 *   table update ................................. Algorithm 3
 *   verification / miss loading / prefetch ....... Sections 4.1 and 4.3.4
 * Readings of silent or ambiguous points are listed next to each function.
 *
 * Pins (tests/test_oracle_*.py): a hand-worked CCT example, counting
 * invariants, the stationary recall of a planted transition (Markov chain
 * closed form), full sort vs selection, torch.nn.functional on tiny SwiGLU
 * cases, an unbounded-cache replay.  Parity unpinned: the paper's 85 %
 * accuracy figure (needs its models and datasets).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1, ORC_FP8 = 2 };
enum { ORC_MODE_OFF = 0, ORC_MODE_TEMPORAL = 1, ORC_MODE_SPATIAL = 2, ORC_MODE_ST = 3 };

#define ORC_CONF_INIT 2 /* binary 10: "preferred" (Algorithm 1, last loop) */
#define ORC_CONF_MAX 3  /* binary 11: "strongly preferred" */
#define ORC_THRESHOLD 2 /* prefetch when the combined score is >= binary 10 */

void orc_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int orc_get_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ */
/* storage formats                                                     */

float orc_bf16_to_f32(uint16_t v)
{
    uint32_t u = (uint32_t)v << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* e4m3 "fn" variant: 1 sign, 4 exponent (bias 7), 3 mantissa bits, no
 * infinities, S.1111.111 is NaN, exponent 0 holds subnormals m/8 * 2^-6. */
float orc_e4m3_to_f32(uint8_t v)
{
    int sign = v >> 7, ex = (v >> 3) & 15, man = v & 7;
    double mag;
    if (ex == 15 && man == 7) return NAN;
    if (ex == 0)
        mag = ldexp((double)man / 8.0, -6);
    else
        mag = ldexp(1.0 + (double)man / 8.0, ex - 7);
    return (float)(sign ? -mag : mag);
}

/* element (row, col) of a stored matrix with `cols` columns, as fp32.  For
 * fp8 the value is float(e4m3) * float(scale of the output channel = row). */
static float weight_at(const void *w, const void *scale, int dtype, int64_t row, int64_t cols,
                       int64_t col)
{
    int64_t i = row * cols + col;
    switch (dtype) {
    case ORC_F32: return ((const float *)w)[i];
    case ORC_BF16: return orc_bf16_to_f32(((const uint16_t *)w)[i]);
    default:
        return orc_e4m3_to_f32(((const uint8_t *)w)[i]) *
               orc_bf16_to_f32(((const uint16_t *)scale)[row]);
    }
}

/* ------------------------------------------------------------------ */
/* Section 2: gating network, softmax, top-K                           */

/* Pre-norm of the stack harness: x = h / sqrt(mean(h^2) + eps), no gain. */
void orc_rmsnorm(const float *h, int H, float eps, float *x)
{
    double ss = 0.0;
    for (int i = 0; i < H; ++i) ss += (double)h[i] * (double)h[i];
    double inv = 1.0 / sqrt(ss / (double)H + (double)eps);
    for (int i = 0; i < H; ++i) x[i] = (float)((double)h[i] * inv);
}

/* z_j = w_j^T x for the N experts. */
void orc_router_logits(const float *x, const void *Wr, int dtype, int E, int H, float *z)
{
    for (int j = 0; j < E; ++j) {
        double acc = 0.0;
        for (int i = 0; i < H; ++i) acc += (double)weight_at(Wr, NULL, dtype, j, H, i) * (double)x[i];
        z[j] = (float)acc;
    }
}

/* s = softmax(z) over all E experts. */
void orc_softmax(const float *z, int E, float *s)
{
    double m = z[0], sum = 0.0;
    for (int j = 1; j < E; ++j)
        if (z[j] > m) m = z[j];
    for (int j = 0; j < E; ++j) sum += exp((double)z[j] - m);
    for (int j = 0; j < E; ++j) s[j] = (float)(exp((double)z[j] - m) / sum);
}

/* The K experts with the largest gating score (softmax is monotone, so the
 * order is taken on the logits); equal logits: the lower id wins.  ids come
 * back in ascending id order.  *gap = z_(K) - z_(K+1), +inf when K == E. */
void orc_topk(const float *z, int E, int K, int32_t *ids, float *gap)
{
    uint8_t *taken = (uint8_t *)calloc((size_t)E, 1);
    float kth = 0.f;
    for (int r = 0; r < K; ++r) {
        int best = -1;
        for (int j = 0; j < E; ++j)
            if (!taken[j] && (best < 0 || z[j] > z[best])) best = j;
        taken[best] = 1;
        kth = z[best];
    }
    int n = 0;
    float next = -INFINITY;
    for (int j = 0; j < E; ++j) {
        if (taken[j])
            ids[n++] = j;
        else if (z[j] > next)
            next = z[j];
    }
    if (gap) *gap = (K < E) ? kth - next : INFINITY;
    free(taken);
}

/* RMSNorm -> logits -> softmax -> top-K for one token.  w[k] is the plain
 * softmax probability of ids[k] (no renormalisation over the selected K
 * unless renorm != 0).  near_tie = gap < 1e-4. */
void orc_route(const float *h, const void *Wr, int dtype, int E, int H, int K, float eps,
               int renorm, float *x, float *z, int32_t *ids, float *w, int32_t *near_tie)
{
    float *s = (float *)malloc(sizeof(float) * (size_t)E);
    float gap;
    orc_rmsnorm(h, H, eps, x);
    orc_router_logits(x, Wr, dtype, E, H, z);
    orc_softmax(z, E, s);
    orc_topk(z, E, K, ids, &gap);
    double tot = 0.0;
    for (int k = 0; k < K; ++k) tot += s[ids[k]];
    for (int k = 0; k < K; ++k) w[k] = renorm ? (float)((double)s[ids[k]] / tot) : s[ids[k]];
    if (near_tie) *near_tie = gap < 1e-4f;
    free(s);
}

/* ------------------------------------------------------------------ */
/* expert FFN (SwiGLU) and the weighted sum of Section 2                */

/* y = W_d ( silu(W_g x) * (W_u x) ),  silu(g) = g / (1 + exp(-g)). */
void orc_expert_ffn(const float *x, int H, int I, const void *Wg, const void *Wu, const void *Wd,
                    const void *sg, const void *su, const void *sd, int dtype, float *y)
{
    float *a = (float *)malloc(sizeof(float) * (size_t)I);
#pragma omp parallel for schedule(static)
    for (int i = 0; i < I; ++i) {
        double g = 0.0, u = 0.0;
        for (int j = 0; j < H; ++j) {
            g += (double)weight_at(Wg, sg, dtype, i, H, j) * (double)x[j];
            u += (double)weight_at(Wu, su, dtype, i, H, j) * (double)x[j];
        }
        float gf = (float)g, uf = (float)u;
        a[i] = (float)((double)gf / (1.0 + exp(-(double)gf)) * (double)uf);
    }
#pragma omp parallel for schedule(static)
    for (int h = 0; h < H; ++h) {
        double acc = 0.0;
        for (int i = 0; i < I; ++i) acc += (double)weight_at(Wd, sd, dtype, h, I, i) * (double)a[i];
        y[h] = (float)acc;
    }
    free(a);
}

/* h' = h + residual_scale * ( sum_shared y_s + sum_k w_k y_k ).
 * ys: [n_shared][H] outputs of the always-on experts, yk: [K][H]. */
void orc_combine(const float *h, int H, const float *ys, int n_shared, const float *yk,
                 const float *w, int K, float residual_scale, float *h_out)
{
    for (int i = 0; i < H; ++i) {
        double y = 0.0;
        for (int s = 0; s < n_shared; ++s) y += (double)ys[(size_t)s * H + i];
        for (int k = 0; k < K; ++k) y += (double)w[k] * (double)yk[(size_t)k * H + i];
        h_out[i] = (float)((double)h[i] + (double)residual_scale * y);
    }
}

/* ------------------------------------------------------------------ */
/* Algorithm 1: co-activation counts and CCT construction              */

/* One profiling token of one adjacent layer pair: Co[e][f] += 1 for every
 * e routed at layer i and f routed at layer i+1. */
void orc_co_accumulate(uint32_t *Co, int E, const int32_t *Ei, int ni, const int32_t *Fi, int nf)
{
    for (int a = 0; a < ni; ++a)
        for (int b = 0; b < nf; ++b) Co[(size_t)Ei[a] * E + Fi[b]] += 1u;
}

/* Per row e: the K next-layer experts with the largest counts, stored in rank
 * order, every confidence set to binary 10.  Ties (and never-seen rows): the
 * lower id ranks first, so an all-zero row yields ids 0..K-1. */
void orc_cct_build(const uint32_t *Co, int E, int K, uint8_t *cct_id, uint8_t *cct_conf)
{
    uint8_t *taken = (uint8_t *)malloc((size_t)E);
    for (int e = 0; e < E; ++e) {
        memset(taken, 0, (size_t)E);
        for (int r = 0; r < K; ++r) {
            int best = -1;
            for (int f = 0; f < E; ++f)
                if (!taken[f] && (best < 0 || Co[(size_t)e * E + f] > Co[(size_t)e * E + best]))
                    best = f;
            taken[best] = 1;
            cct_id[(size_t)e * K + r] = (uint8_t)best;
            cct_conf[(size_t)e * K + r] = ORC_CONF_INIT;
        }
    }
    free(taken);
}

/* ------------------------------------------------------------------ */
/* Algorithm 2 + Eq. 1: expert prediction                              */

/* score[f] = sum of the confidences of every CCT candidate f found in the
 * rows of the experts routed at layer i (spatial part), plus binary 10 for
 * each valid entry of the next layer's history table (temporal part, Eq. 1).
 * Prefetch set = { f : score[f] >= 2 }.  cct_* == NULL drops the spatial
 * part, ht == NULL the temporal part.  HT entries < 0 are "not yet written".
 *
 * The printed listing overwrites the score of an HT member with 1 and then
 * adds 1; `literal` (optional) receives those scores.  Both give the same
 * set; the function returns -1 if they ever differ, else the set size. */
int orc_predict_thr(int E, int K, const int32_t *Ei, int ni, const uint8_t *cct_id,
                    const uint8_t *cct_conf, const int16_t *ht, int threshold, int32_t *score,
                    int32_t *literal, uint8_t *in_set);

int orc_predict(int E, int K, const int32_t *Ei, int ni, const uint8_t *cct_id,
                const uint8_t *cct_conf, const int16_t *ht, int32_t *score, int32_t *literal,
                uint8_t *in_set)
{
    return orc_predict_thr(E, K, Ei, ni, cct_id, cct_conf, ht, ORC_THRESHOLD, score, literal, in_set);
}

/* The same with the set threshold as a parameter (Section 4.2 fixes it at binary 10; other
 * values are the threshold sweep of the ablation).  The history bonus stays binary 10 (Eq. 1).
 * The printed listing is only comparable at the paper's threshold: for other values the check
 * against it is skipped. */
int orc_predict_thr(int E, int K, const int32_t *Ei, int ni, const uint8_t *cct_id,
                    const uint8_t *cct_conf, const int16_t *ht, int threshold, int32_t *score,
                    int32_t *literal, uint8_t *in_set)
{
    int32_t *lit = literal ? literal : (int32_t *)malloc(sizeof(int32_t) * (size_t)E);
    for (int f = 0; f < E; ++f) score[f] = lit[f] = 0;
    if (cct_id)
        for (int a = 0; a < ni; ++a)
            for (int c = 0; c < K; ++c) {
                int f = cct_id[(size_t)Ei[a] * K + c];
                score[f] += cct_conf[(size_t)Ei[a] * K + c];
                lit[f] += cct_conf[(size_t)Ei[a] * K + c];
            }
    if (ht) {
        for (int c = 0; c < K; ++c)
            if (ht[c] >= 0) score[ht[c]] += ORC_THRESHOLD; /* Eq. 1: CCT(e) + HT(e) */
        for (int c = 0; c < K; ++c)
            if (ht[c] >= 0) lit[ht[c]] = 1;
        for (int c = 0; c < K; ++c)
            if (ht[c] >= 0) lit[ht[c]] += 1;
    }
    int n = 0, same = 1;
    for (int f = 0; f < E; ++f) {
        in_set[f] = score[f] >= threshold;
        if (threshold == ORC_THRESHOLD && in_set[f] != (lit[f] >= ORC_THRESHOLD)) same = 0;
        n += in_set[f];
    }
    if (!literal) free(lit);
    return same ? n : -1;
}

/* ------------------------------------------------------------------ */
/* Algorithm 3: table update                                           */

/* For each expert e routed at layer i (ascending id) and each stored
 * candidate of row e in slot order: confirmed by the layer-(i+1) routing ->
 * confidence +1 capped at 3; not confirmed and confidence > 0 -> -1; not
 * confirmed at confidence 0 -> replaced by an expert of F that the row does
 * not hold, confidence binary 10.  The row is re-read after each replacement
 * so a row never holds an id twice; when every routed expert is already in
 * the row the slot is left.  The listing leaves the choice among several such
 * experts open:
 *   Co == NULL  the lowest id (the default reading);
 *   Co != NULL  the one with the largest count in row e of Co, the pair's
 *               co-activation counts kept up to date at run time (the caller
 *               has already counted this step's pairs); equal counts -> the
 *               lower id. */
void orc_update_rule(int E, int K, const int32_t *Ei, int ni, const int32_t *Fj, int nf,
                     uint8_t *cct_id, uint8_t *cct_conf, const uint32_t *Co)
{
    for (int a = 0; a < ni; ++a) {
        uint8_t *id = cct_id + (size_t)Ei[a] * K, *cf = cct_conf + (size_t)Ei[a] * K;
        const uint32_t *row = Co ? Co + (size_t)Ei[a] * E : NULL;
        for (int c = 0; c < K; ++c) {
            int hit = 0;
            for (int b = 0; b < nf; ++b) hit |= (Fj[b] == id[c]);
            if (hit) {
                cf[c] = (uint8_t)(cf[c] + 1 > ORC_CONF_MAX ? ORC_CONF_MAX : cf[c] + 1);
            } else if (cf[c] > 0) {
                cf[c] -= 1;
            } else {
                int g = -1;
                for (int b = 0; b < nf; ++b) { /* Fj is ascending */
                    int held = 0;
                    for (int d = 0; d < K; ++d) held |= (id[d] == Fj[b]);
                    if (held) continue;
                    if (g < 0) g = Fj[b];
                    if (!row) break;
                    if (row[Fj[b]] > row[g]) g = Fj[b];
                }
                if (g >= 0) {
                    id[c] = (uint8_t)g;
                    cf[c] = ORC_CONF_INIT;
                }
            }
        }
    }
}

void orc_update(int E, int K, const int32_t *Ei, int ni, const int32_t *Fj, int nf,
                uint8_t *cct_id, uint8_t *cct_conf)
{
    orc_update_rule(E, K, Ei, ni, Fj, nf, cct_id, cct_conf, NULL);
}

/* ------------------------------------------------------------------ */
/* predictor state machine over a whole stack                          */

typedef struct {
    int32_t L, E, K, B, P, mode, built, max_pred, threshold, live_counts;
    int64_t t;          /* decode steps completed */
    uint32_t *Co;       /* [L-1][E][E] */
    uint8_t *cct_id;    /* [L-1][E][K] */
    uint8_t *cct_conf;  /* [L-1][E][K] */
    int16_t *HT;        /* [B][L][K], -1 = not yet written */
    int32_t *prev;      /* [B][K] routing of the previous layer, this token */
    uint8_t *pred;      /* [B][E] set predicted for the layer that runs next */
    uint8_t *pred_valid; /* [B] */
    int64_t st_steps, st_routed, st_pred, st_hit;
} orc_pred_t;

static void pred_build(orc_pred_t *p)
{
    for (int i = 0; i < p->L - 1; ++i)
        orc_cct_build(p->Co + (size_t)i * p->E * p->E, p->E, p->K,
                      p->cct_id + (size_t)i * p->E * p->K, p->cct_conf + (size_t)i * p->E * p->K);
    p->built = 1;
}

orc_pred_t *orc_pred_create(int L, int E, int K, int B, int P, int mode)
{
    if (L < 1 || E < 1 || E > 256 || K < 1 || K > E || K > 32 || B < 1 || P < 0) return NULL;
    orc_pred_t *p = (orc_pred_t *)calloc(1, sizeof(*p));
    int pairs = L > 1 ? L - 1 : 0;
    p->L = L, p->E = E, p->K = K, p->B = B, p->P = P, p->mode = mode, p->threshold = ORC_THRESHOLD;
    p->max_pred = (K * K + K < E) ? K * K + K : E;
    p->Co = (uint32_t *)calloc((size_t)pairs * E * E + 1, 4);
    p->cct_id = (uint8_t *)calloc((size_t)pairs * E * K + 1, 1);
    p->cct_conf = (uint8_t *)calloc((size_t)pairs * E * K + 1, 1);
    p->HT = (int16_t *)malloc(sizeof(int16_t) * (size_t)B * L * K);
    for (size_t i = 0; i < (size_t)B * L * K; ++i) p->HT[i] = -1;
    p->prev = (int32_t *)calloc((size_t)B * K, 4);
    p->pred = (uint8_t *)calloc((size_t)B * E, 1);
    p->pred_valid = (uint8_t *)calloc((size_t)B, 1);
    if (P == 0) pred_build(p);
    return p;
}

void orc_pred_destroy(orc_pred_t *p)
{
    if (!p) return;
    free(p->Co), free(p->cct_id), free(p->cct_conf), free(p->HT), free(p->prev), free(p->pred),
        free(p->pred_valid), free(p);
}

int orc_pred_max_pred(const orc_pred_t *p) { return p->max_pred; }

/* Set threshold of Algorithm 2 for this predictor (>= 1; default binary 10).  The set still holds
 * at most K*K + K experts: a member has a stored candidate of non-zero confidence or is in the
 * history table. */
void orc_pred_set_threshold(orc_pred_t *p, int threshold)
{
    p->threshold = threshold < 1 ? 1 : threshold;
}

/* Replacement rule of Algorithm 3 for this predictor.  0 (default): the lowest routed id the
 * row does not hold; the counts stay as profiling left them.  1: counting goes on at run time
 * (for every sequence, Co[e][f] += 1 for e routed at the previous layer and f at this one,
 * right before that sequence's table update) and the new candidate is the routed expert with
 * the largest count in the row. */
void orc_pred_set_replacement(orc_pred_t *p, int live_counts) { p->live_counts = live_counts != 0; }

/* One layer step for sequences 0..batch-1 (Section 4.3.4: R, then V and P).
 *
 *   profiling (t < P): count co-activations of pair (layer-1, layer); the
 *     tables are built right after the last layer of the last profiling step.
 *   runtime (t >= P): V  score the set predicted for this layer against the
 *     routing, then Algorithm 3 on pair (layer-1, layer), sequence by
 *     sequence in index order (the CCT is shared by the batch, the history
 *     table is per sequence);
 *     P  Algorithm 2 for layer+1 from this layer's routing, CCT[layer] and
 *     HT[layer+1] (which still holds the previous token's routing).  After
 *     the last layer the prediction is for layer 0 of the next token and can
 *     only use the history table.
 *   always: HT[layer] <- routing.
 * The mode only selects which sources feed Algorithm 2; the tables evolve
 * identically in every mode.
 *
 * routed   [batch][K] ascending ids
 * pred_ids [batch][max_pred] ascending ids of the prefetch set, -1 padded
 * queue_*  union of the batch's sets, score = sum over sequences, ordered by
 *          (score descending, id ascending): the prefetch priority order.
 * Returns 0, or -1 on a bad argument, -2 if Eq. 1 and the literal listing of
 * Algorithm 2 disagree on a set. */
int orc_pred_step(orc_pred_t *p, int layer, int batch, const int32_t *routed, int32_t *pred_ids,
                  int32_t *n_pred, int32_t *queue_ids, int32_t *queue_score, int32_t *n_queue)
{
    const int E = p->E, K = p->K, L = p->L;
    if (layer < 0 || layer >= L || batch < 1 || batch > p->B) return -1;
    const int runtime = p->t >= p->P;
    int rc = 0;

    if (runtime) {
        for (int b = 0; b < batch; ++b) {
            const int32_t *R = routed + (size_t)b * K;
            int np = 0, nh = 0;
            if (p->pred_valid[b])
                for (int f = 0; f < E; ++f) np += p->pred[(size_t)b * E + f];
            if (p->pred_valid[b])
                for (int k = 0; k < K; ++k) nh += p->pred[(size_t)b * E + R[k]];
            p->st_steps += 1, p->st_routed += K, p->st_pred += np, p->st_hit += nh;
            if (layer > 0) {
                uint32_t *Co = p->Co + (size_t)(layer - 1) * E * E;
                if (p->live_counts) orc_co_accumulate(Co, E, p->prev + (size_t)b * K, K, R, K);
                orc_update_rule(E, K, p->prev + (size_t)b * K, K, R, K,
                                p->cct_id + (size_t)(layer - 1) * E * K,
                                p->cct_conf + (size_t)(layer - 1) * E * K, p->live_counts ? Co : NULL);
            }
        }
    } else if (layer > 0) {
        for (int b = 0; b < batch; ++b)
            orc_co_accumulate(p->Co + (size_t)(layer - 1) * E * E, E, p->prev + (size_t)b * K, K,
                              routed + (size_t)b * K, K);
    }

    if (!runtime && p->t == p->P - 1 && layer == L - 1) pred_build(p);

    const int predict_now = p->built && (runtime || (p->t == p->P - 1 && layer == L - 1));
    int32_t *score = (int32_t *)malloc(sizeof(int32_t) * (size_t)E);
    int32_t *total = (int32_t *)calloc((size_t)E, sizeof(int32_t));
    for (int b = 0; b < batch; ++b) {
        uint8_t *set = p->pred + (size_t)b * E;
        int n = 0;
        memset(set, 0, (size_t)E);
        p->pred_valid[b] = (uint8_t)predict_now;
        if (predict_now && p->mode != ORC_MODE_OFF) {
            const int next = (layer + 1) % L;
            const int spatial = (p->mode & ORC_MODE_SPATIAL) && layer < L - 1;
            const int temporal = (p->mode & ORC_MODE_TEMPORAL) != 0;
            n = orc_predict_thr(E, K, routed + (size_t)b * K, spatial ? K : 0,
                                spatial ? p->cct_id + (size_t)layer * E * K : NULL,
                                spatial ? p->cct_conf + (size_t)layer * E * K : NULL,
                                temporal ? p->HT + ((size_t)b * L + next) * K : NULL, p->threshold, score, NULL, set);
            if (n < 0) rc = -2, n = 0;
            for (int f = 0; f < E; ++f)
                if (set[f]) total[f] += score[f];
        }
        if (n_pred) n_pred[b] = n;
        if (pred_ids) {
            int m = 0;
            for (int f = 0; f < E; ++f)
                if (set[f]) pred_ids[(size_t)b * p->max_pred + m++] = f;
            for (; m < p->max_pred; ++m) pred_ids[(size_t)b * p->max_pred + m] = -1;
        }
    }
    if (n_queue) {
        int n = 0;
        for (int f = 0; f < E; ++f)
            if (total[f] > 0) queue_ids[n] = f, queue_score[n] = total[f], ++n;
        for (int i = 1; i < n; ++i) { /* insertion sort: score desc, id asc */
            int32_t id = queue_ids[i], sc = queue_score[i];
            int j = i - 1;
            while (j >= 0 && queue_score[j] < sc) {
                queue_ids[j + 1] = queue_ids[j], queue_score[j + 1] = queue_score[j];
                --j;
            }
            queue_ids[j + 1] = id, queue_score[j + 1] = sc;
        }
        *n_queue = n;
    }
    free(score), free(total);

    for (int b = 0; b < batch; ++b)
        for (int k = 0; k < K; ++k) {
            p->HT[((size_t)b * L + layer) * K + k] = (int16_t)routed[(size_t)b * K + k];
            p->prev[(size_t)b * K + k] = routed[(size_t)b * K + k];
        }
    if (layer == L - 1) p->t += 1;
    return rc;
}

void orc_pred_stats(const orc_pred_t *p, int64_t *out4)
{
    out4[0] = p->st_steps, out4[1] = p->st_routed, out4[2] = p->st_pred, out4[3] = p->st_hit;
}

/* Canonical state image: 8 int32 {magic, version, L, E, K, B, P, built},
 * int64 t, then Co (u32), cct_id (u8), cct_conf (u8), HT (i16). */
#define ORC_STATE_MAGIC 0x53544D50
size_t orc_pred_state_bytes(const orc_pred_t *p)
{
    size_t pairs = p->L > 1 ? (size_t)p->L - 1 : 0;
    return 32 + 8 + pairs * p->E * p->E * 4 + 2 * pairs * p->E * p->K +
           (size_t)p->B * p->L * p->K * 2;
}

size_t orc_pred_export(const orc_pred_t *p, void *buf)
{
    size_t pairs = p->L > 1 ? (size_t)p->L - 1 : 0;
    uint8_t *o = (uint8_t *)buf;
    int32_t hdr[8] = {ORC_STATE_MAGIC, 1, p->L, p->E, p->K, p->B, p->P, p->built};
    memcpy(o, hdr, 32), o += 32;
    memcpy(o, &p->t, 8), o += 8;
    memcpy(o, p->Co, pairs * p->E * p->E * 4), o += pairs * p->E * p->E * 4;
    memcpy(o, p->cct_id, pairs * p->E * p->K), o += pairs * p->E * p->K;
    memcpy(o, p->cct_conf, pairs * p->E * p->K), o += pairs * p->E * p->K;
    memcpy(o, p->HT, (size_t)p->B * p->L * p->K * 2), o += (size_t)p->B * p->L * p->K * 2;
    return (size_t)(o - (uint8_t *)buf);
}

/* ------------------------------------------------------------------ */
/* verification, miss loading and prefetch as an integer cache model   */

/* The paper stages predicted experts in an on-chip buffer and fetches a
 * mispredicted expert at once (Section 4.3.4); it names no replacement
 * policy.  Model used here: S slots.
 *   use history  every (layer, expert) key carries W bits: bit i = the key was
 *            routed at its layer's turn i decode steps ago (bit 0 = this
 *            step).  At the start of a layer's step the histories of that
 *            layer's keys shift by one; routed keys then set bit 0.
 *   victim   among the slots not protected in this step: an empty slot first,
 *            else the key with the fewest uses in its window; then (by_turn)
 *            the key whose layer's next turn is furthest away: a decode step
 *            walks the layers in a fixed cycle, so a key of layer m waits
 *            (m - layer) mod L layer steps, L for the layer in progress; then
 *            the least recently used (a clock that ticks once per layer step);
 *            then the lowest slot index.  W = 0 without by_turn is plain LRU.
 *            (Once a decode step touches more keys than there are slots, LRU
 *            evicts every key just before its next turn and the hit rate is
 *            zero; use counts keep the popular keys and the turn order keeps a
 *            stable subset among equally popular ones.)
 *   verify   each routed expert (ascending id): resident -> hit, else a
 *            demand load into a victim that no routed expert of this step
 *            occupies;
 *   prefetch each queued expert of the next layer, in queue order: skipped
 *            if resident, else loaded into a victim that holds neither a
 *            routed expert of this step nor any queued expert; dropped when
 *            no such slot exists, when `limit` copies were issued this step,
 *            or when the victim's key has more than `floor` uses in its
 *            window (floor < 0: no such test): a speculative copy may then
 *            only take slots whose content has not been of use lately.
 * A prefetched expert that is evicted before its first use counts as wasted. */
typedef struct {
    int64_t S, clock;
    int32_t L, E, W, floor, by_turn, cur_layer;
    int32_t *slot_of;   /* [L*E] slot or -1 */
    int32_t *tag;       /* [S]   layer*E+expert or -1 */
    int64_t *stamp;     /* [S] */
    uint32_t *hist;     /* [L*E] use history, W <= 32 bits */
    uint8_t *pf_unused; /* [S] brought by prefetch, not used yet */
    uint8_t *guard;     /* [S] scratch: protected during the current pass */
    int64_t hits, misses, pf_issued, pf_useful, pf_wasted, pf_dropped, pf_resident;
} orc_cache_t;

orc_cache_t *orc_cache_create2(int64_t S, int L, int E, int W, int floor, int by_turn)
{
    if (W < 0 || W > 32) return NULL;
    orc_cache_t *c = (orc_cache_t *)calloc(1, sizeof(*c));
    c->S = S, c->L = L, c->E = E, c->W = W, c->floor = floor, c->by_turn = by_turn;
    c->slot_of = (int32_t *)malloc(sizeof(int32_t) * (size_t)L * E);
    c->tag = (int32_t *)malloc(sizeof(int32_t) * (size_t)S);
    c->stamp = (int64_t *)malloc(sizeof(int64_t) * (size_t)S);
    c->hist = (uint32_t *)calloc((size_t)L * E, sizeof(uint32_t));
    c->pf_unused = (uint8_t *)calloc((size_t)S, 1);
    c->guard = (uint8_t *)calloc((size_t)S, 1);
    for (int i = 0; i < L * E; ++i) c->slot_of[i] = -1;
    for (int64_t s = 0; s < S; ++s) c->tag[s] = -1, c->stamp[s] = -1;
    return c;
}

orc_cache_t *orc_cache_create(int64_t S, int L, int E) { return orc_cache_create2(S, L, E, 0, -1, 0); }

void orc_cache_destroy(orc_cache_t *c)
{
    if (!c) return;
    free(c->slot_of), free(c->tag), free(c->stamp), free(c->hist), free(c->pf_unused), free(c->guard), free(c);
}

static int cache_uses(const orc_cache_t *c, int64_t s)
{
    if (c->tag[s] < 0) return -1; /* empty: before everything */
    int n = 0;
    for (uint32_t h = c->hist[c->tag[s]]; h; h >>= 1) n += (int)(h & 1u);
    return n;
}

/* layer steps until the turn of the layer that the slot's key belongs to */
static int cache_wait(const orc_cache_t *c, int64_t s)
{
    if (!c->by_turn || c->tag[s] < 0) return 0;
    int d = (c->tag[s] / c->E - c->cur_layer) % c->L;
    if (d < 0) d += c->L;
    return d == 0 ? c->L : d;
}

static int64_t cache_victim(const orc_cache_t *c)
{
    int64_t best = -1;
    int best_uses = 0, best_wait = 0;
    for (int64_t s = 0; s < c->S; ++s) {
        if (c->guard[s]) continue;
        int u = cache_uses(c, s), w = cache_wait(c, s);
        if (best < 0 || u < best_uses || (u == best_uses && (w > best_wait || (w == best_wait && c->stamp[s] < c->stamp[best]))))
            best = s, best_uses = u, best_wait = w;
    }
    return best;
}

static void cache_place(orc_cache_t *c, int64_t s, int32_t key, int by_prefetch)
{
    if (c->tag[s] >= 0) {
        c->slot_of[c->tag[s]] = -1;
        if (c->pf_unused[s]) c->pf_wasted += 1;
    }
    c->tag[s] = key, c->slot_of[key] = (int32_t)s;
    c->stamp[s] = c->clock, c->pf_unused[s] = (uint8_t)by_prefetch;
}

/* U: nU distinct routed experts of `layer`, ascending.  Q: nQ queued experts
 * of `next_layer` in priority order.  u_slot[i]: slot serving U[i];
 * u_loaded[i]: 1 if it had to be demand loaded.  q_slot[i]: slot a prefetch
 * copy of Q[i] was issued into, else -1.  Returns 0, or -1 when the routed
 * experts do not fit in the cache. */
int orc_cache_step(orc_cache_t *c, int layer, const int32_t *U, int nU, int next_layer,
                   const int32_t *Q, int nQ, int limit, int32_t *u_slot, uint8_t *u_loaded,
                   int32_t *q_slot)
{
    const uint32_t mask = c->W >= 32 ? 0xffffffffu : ((1u << c->W) - 1u);
    c->cur_layer = layer;
    for (int e = 0; e < c->E; ++e) c->hist[layer * c->E + e] = (c->hist[layer * c->E + e] << 1) & mask;
    memset(c->guard, 0, (size_t)c->S);
    for (int i = 0; i < nU; ++i) {
        int32_t s = c->slot_of[layer * c->E + U[i]];
        if (s >= 0) c->guard[s] = 1;
    }
    for (int i = 0; i < nU; ++i) {
        int32_t key = layer * c->E + U[i];
        int64_t s = c->slot_of[key];
        if (c->W > 0) c->hist[key] |= 1u;
        if (s >= 0) {
            c->hits += 1;
            if (c->pf_unused[s]) c->pf_useful += 1, c->pf_unused[s] = 0;
            c->stamp[s] = c->clock;
            u_loaded[i] = 0;
        } else {
            s = cache_victim(c);
            if (s < 0) return -1;
            c->misses += 1;
            cache_place(c, s, key, 0);
            c->guard[s] = 1;
            u_loaded[i] = 1;
        }
        u_slot[i] = (int32_t)s;
    }
    for (int i = 0; i < nQ; ++i) {
        int32_t s = c->slot_of[next_layer * c->E + Q[i]];
        if (s >= 0) c->guard[s] = 1;
    }
    int issued = 0;
    for (int i = 0; i < nQ; ++i) {
        int32_t key = next_layer * c->E + Q[i];
        q_slot[i] = -1;
        if (c->slot_of[key] >= 0) {
            c->pf_resident += 1;
            continue;
        }
        int64_t s = (limit > 0 && issued >= limit) ? -1 : cache_victim(c);
        if (s >= 0 && c->floor >= 0 && cache_uses(c, s) > c->floor) s = -1;
        if (s < 0) {
            c->pf_dropped += 1;
            continue;
        }
        cache_place(c, s, key, 1);
        c->guard[s] = 1;
        c->pf_issued += 1, ++issued;
        q_slot[i] = (int32_t)s;
    }
    c->clock += 1;
    return 0;
}

void orc_cache_stats(const orc_cache_t *c, int64_t *out7)
{
    out7[0] = c->hits, out7[1] = c->misses, out7[2] = c->pf_issued, out7[3] = c->pf_useful;
    out7[4] = c->pf_wasted, out7[5] = c->pf_dropped, out7[6] = c->pf_resident;
}

void orc_cache_tags(const orc_cache_t *c, int32_t *tags) { memcpy(tags, c->tag, 4 * (size_t)c->S); }
