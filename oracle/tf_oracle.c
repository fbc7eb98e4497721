/*
 * Token Filtering oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of the per-layer online pruning step of
 * Token Filtering ("Leveraging KV Similarity for Online Structured Pruning in
 * LLMs"), restated for a whole prefill sequence: every token t is treated as
 * "the current token" of Algorithm 1 with tokens 0..t-1 as its past.
 *
 * Only the tests, the smoke check and the benchmark's cpu_baseline / reference
 * arm may call this file.  It shares no code with the CUDA library and the CUDA
 * library never calls it.
 *
 * Layout of every tensor: token-major, contiguous, [B, S, H, d] (d fastest).
 * Inputs are float32 arrays holding the exact fp32 / bf16 input values; every
 * arithmetic step widens to double first.  Loops are written in the order of
 * the paper's steps, with no blocking, fusion or reordering.
 *
 * Parity pins (tests/test_oracle_*.py) cover every function below against
 * closed forms, invariants, brute force and library routines; the one thing no
 * pin can decide is which of the documented readings (anchor excludes/includes
 * the current token; Eq. 2 literal or inverse-variance; pruned tokens' K/V
 * still visible or not) the authors ran: "parity unpinned" for that choice
 * only -- every reading is implemented behind a mode flag.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* mode flags (values mirror nothing but this file's Python wrapper) */
enum { TFO_ANCHOR_PAST_MEAN = 0, TFO_ANCHOR_INCL_MEAN = 1, TFO_ANCHOR_EMA = 2 };
enum { TFO_FUSE_INVVAR = 0, TFO_FUSE_EQ2_LITERAL = 1, TFO_FUSE_KEY_ONLY = 2,
       TFO_FUSE_VALUE_ONLY = 3, TFO_FUSE_MEAN = 4 };
enum { TFO_SELECT_RATIO = 0, TFO_SELECT_THRESHOLD = 1 };
enum { TFO_KV_ALL = 0, TFO_KV_RETAINED = 1 };

#define TFO_NORM_EPS 1e-8

/* cosine similarity with each norm clamped from below (the convention of the
 * framework the paper ran on); Algorithm 1, cosine_sim(Anchor, k_last). */
static double cosine_clamped(const double *a, const double *x, int d)
{
    double dot = 0.0, na = 0.0, nx = 0.0;
    for (int i = 0; i < d; ++i) {
        dot += a[i] * x[i];
        na += a[i] * a[i];
        nx += x[i] * x[i];
    }
    na = sqrt(na);
    nx = sqrt(nx);
    if (na < TFO_NORM_EPS) na = TFO_NORM_EPS;
    if (nx < TFO_NORM_EPS) nx = TFO_NORM_EPS;
    return dot / (na * nx);
}

/*
 * Steps a1 + a2: anchors and per-head cosine similarity.
 * Algorithm 1 (AnchorK <- mean(K); cosine_sim(AnchorK, k_last)), Section 3.2
 * ("anchor key is defined as the mean of all previous keys"), Eq. 1 (EMA).
 *
 *   X         [B,S,H,d]   keys (or values)
 *   sum_in    [B,H,d]     optional: sum of the tokens that came before this
 *                         call (chunked prefill); NULL = none
 *   count_in  [B]         optional: how many tokens sum_in holds
 *   sim       [B,S,H]     out: cosine of token t to its anchor
 *   sum_out   [B,H,d]     optional out: sum over carry + all S tokens
 *                         (EMA mode: the final EMA anchor itself)
 *
 * PAST_MEAN: anchor_t = mean of tokens before t (none -> similarity 0).
 * INCL_MEAN: anchor_t = mean of tokens up to and including t (Alg. 1 read
 *            literally: K already holds k_last when mean(K) is taken).
 * EMA:       anchor compared first, then anchor <- g*anchor + (1-g)*x (Eq. 1),
 *            anchor starts at sum_in (or 0 = "no past").
 */
void tfo_anchor_similarity(const float *X, int B, int S, int H, int d,
                           int anchor_mode, double gamma,
                           const float *sum_in, const int64_t *count_in,
                           double *sim, double *sum_out)
{
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double *run = (double *)malloc(sizeof(double) * d);    /* running sum / EMA */
            double *anchor = (double *)malloc(sizeof(double) * d);
            double *x = (double *)malloc(sizeof(double) * d);
            int64_t n_past = 0;
            for (int i = 0; i < d; ++i) run[i] = 0.0;
            if (sum_in) {
                for (int i = 0; i < d; ++i) run[i] = (double)sum_in[((size_t)b * H + h) * d + i];
                n_past = count_in ? count_in[b] : 0;
            }
            for (int t = 0; t < S; ++t) {
                const float *xp = X + (((size_t)b * S + t) * H + h) * d;
                for (int i = 0; i < d; ++i) x[i] = (double)xp[i];
                double c;
                if (anchor_mode == TFO_ANCHOR_INCL_MEAN) {
                    for (int i = 0; i < d; ++i) run[i] += x[i];
                    n_past += 1;
                    for (int i = 0; i < d; ++i) anchor[i] = run[i] / (double)n_past;
                    c = cosine_clamped(anchor, x, d);
                } else if (anchor_mode == TFO_ANCHOR_EMA) {
                    c = (n_past == 0) ? 0.0 : cosine_clamped(run, x, d);
                    for (int i = 0; i < d; ++i) run[i] = gamma * run[i] + (1.0 - gamma) * x[i];
                    n_past += 1;
                } else { /* PAST_MEAN */
                    if (n_past == 0) {
                        c = 0.0;
                    } else {
                        for (int i = 0; i < d; ++i) anchor[i] = run[i] / (double)n_past;
                        c = cosine_clamped(anchor, x, d);
                    }
                    for (int i = 0; i < d; ++i) run[i] += x[i];
                    n_past += 1;
                }
                sim[((size_t)b * S + t) * H + h] = c;
            }
            if (sum_out)
                for (int i = 0; i < d; ++i) sum_out[((size_t)b * H + h) * d + i] = run[i];
            free(run);
            free(anchor);
            free(x);
        }
    }
}

/*
 * Step a3: mean and variance over heads, variance-aware weight, fused score.
 * Algorithm 1 lines "(s_k, sigma_k^2) <- (mean, var)(cosine_sim(...))",
 * "alpha <- ...", "s_KV <- alpha s_k + (1-alpha) s_v"; Eq. 2 and Eq. 3.
 *
 * Population variance over the H heads of one token.
 * INVVAR:      alpha = (var_v + e) / (var_k + var_v + 2e)   lower-variance side
 *              gets the larger weight (the paper's prose).
 * EQ2_LITERAL: alpha = (var_k + e) / (var_k + var_v + 2e)   Eq. 2 as printed,
 *              (1/var_v)/(1/var_k + 1/var_v), multiplied through by var_k var_v.
 * KEY_ONLY / VALUE_ONLY / MEAN: alpha = 1 / 0 / 0.5 (criterion ablation, and
 *              the figure caption's unweighted combination).
 * Outputs score [B,S]; optional s_k, s_v, var_k, var_v, alpha [B,S] each.
 */
void tfo_score_fuse(const double *sim_k, const double *sim_v, int B, int S, int H,
                    int fuse_mode, double var_eps, double *score,
                    double *o_sk, double *o_sv, double *o_vark, double *o_varv, double *o_alpha)
{
    for (int b = 0; b < B; ++b) {
        for (int t = 0; t < S; ++t) {
            const double *ck = sim_k + ((size_t)b * S + t) * H;
            const double *cv = sim_v + ((size_t)b * S + t) * H;
            double sk = 0.0, sv = 0.0;
            for (int h = 0; h < H; ++h) { sk += ck[h]; sv += cv[h]; }
            sk /= (double)H;
            sv /= (double)H;
            double vk = 0.0, vv = 0.0;
            for (int h = 0; h < H; ++h) {
                vk += (ck[h] - sk) * (ck[h] - sk);
                vv += (cv[h] - sv) * (cv[h] - sv);
            }
            vk /= (double)H;
            vv /= (double)H;
            double alpha;
            switch (fuse_mode) {
            case TFO_FUSE_EQ2_LITERAL: alpha = (vk + var_eps) / (vk + vv + 2.0 * var_eps); break;
            case TFO_FUSE_KEY_ONLY:    alpha = 1.0; break;
            case TFO_FUSE_VALUE_ONLY:  alpha = 0.0; break;
            case TFO_FUSE_MEAN:        alpha = 0.5; break;
            default:                   alpha = (vv + var_eps) / (vk + vv + 2.0 * var_eps); break;
            }
            double s = alpha * sk + (1.0 - alpha) * sv;
            if (s == 0.0) s = 0.0; /* -0 -> +0 */
            size_t o = (size_t)b * S + t;
            score[o] = s;
            if (o_sk) o_sk[o] = sk;
            if (o_sv) o_sv[o] = sv;
            if (o_vark) o_vark[o] = vk;
            if (o_varv) o_varv[o] = vv;
            if (o_alpha) o_alpha[o] = alpha;
        }
    }
}

/* ordering used by ratio selection: higher score first, then higher index */
typedef struct { double s; int32_t idx; } tfo_cand;
static int cand_cmp(const void *pa, const void *pb)
{
    const tfo_cand *a = (const tfo_cand *)pa, *b = (const tfo_cand *)pb;
    if (a->s > b->s) return -1;
    if (a->s < b->s) return 1;
    if (a->idx > b->idx) return -1;
    if (a->idx < b->idx) return 1;
    return 0;
}

/*
 * Step a4: which tokens skip attention.
 * Algorithm 1 "Skip layer if s_KV > tau" (strict); Section 3.2 warm-up phase
 * (no pruning at the start); Section 3.3 (each layer holds its skip ratio at
 * the target).  RATIO mode is the fixed point of the threshold controller:
 * exactly P = min(E, floor(ratio * S)) eligible tokens with the highest score
 * are pruned, ties broken toward the later token.  THRESHOLD mode prunes the
 * eligible tokens whose score is strictly above threshold[b].
 *
 * eligible [B,S] optional (1 = may be pruned), ANDed with t >= warmup_tokens.
 * A NaN score is never pruned.
 * Outputs: keep_mask [B,S] (1 = retained), kept_idx [B,S] ascending retained
 * positions padded with -1, n_kept [B], theta [B] = lowest pruned score
 * (+inf when nothing is pruned), n_nan [B] optional.
 */
void tfo_select(const double *score, int B, int S, double prune_ratio, int warmup_tokens,
                const uint8_t *eligible, int select_mode, const double *threshold,
                uint8_t *keep_mask, int32_t *kept_idx, int32_t *n_kept, double *theta,
                int32_t *n_nan)
{
    for (int b = 0; b < B; ++b) {
        const double *sc = score + (size_t)b * S;
        uint8_t *km = keep_mask + (size_t)b * S;
        tfo_cand *cand = (tfo_cand *)malloc(sizeof(tfo_cand) * (size_t)(S > 0 ? S : 1));
        int n_cand = 0, nan_count = 0;
        for (int t = 0; t < S; ++t) {
            km[t] = 1;
            if (isnan(sc[t])) { nan_count++; continue; }
            int ok = (t >= warmup_tokens) && (!eligible || eligible[(size_t)b * S + t]);
            if (ok) { cand[n_cand].s = sc[t]; cand[n_cand].idx = t; n_cand++; }
        }
        double th = INFINITY;
        if (select_mode == TFO_SELECT_THRESHOLD) {
            double tau = threshold[b];
            for (int i = 0; i < n_cand; ++i)
                if (cand[i].s > tau) {
                    km[cand[i].idx] = 0;
                    if (cand[i].s < th) th = cand[i].s;
                }
        } else {
            long P = (long)floor(prune_ratio * (double)S);
            if (P > n_cand) P = n_cand;
            qsort(cand, (size_t)n_cand, sizeof(tfo_cand), cand_cmp);
            for (long i = 0; i < P; ++i) km[cand[i].idx] = 0;
            if (P > 0) th = cand[P - 1].s;
        }
        int k = 0;
        for (int t = 0; t < S; ++t)
            if (km[t]) kept_idx[(size_t)b * S + k++] = t;
        n_kept[b] = k;
        for (; k < S; ++k) kept_idx[(size_t)b * S + k] = -1;
        if (theta) theta[b] = th;
        if (n_nan) n_nan[b] = nan_count;
        free(cand);
    }
}

/* one output row: softmax(scale * q.K[j]) V[j] over the visible keys j */
static void attention_row(const float *Q, const float *K, const float *V,
                          int S, int Hq, int Hkv, int d, int window, double scale,
                          int b, int t, int qh, const uint8_t *visible_mask /* [S] or NULL */,
                          double *out /* [d] */, double *logits /* scratch [S] */)
{
    int g = Hq / Hkv, kh = qh / g;
    int lo = (window > 0) ? (t - window + 1) : 0;
    if (lo < 0) lo = 0;
    const float *q = Q + (((size_t)b * S + t) * Hq + qh) * d;
    double m = -INFINITY;
    int any = 0;
    for (int j = lo; j <= t; ++j) {
        if (visible_mask && !visible_mask[j]) continue;
        const float *k = K + (((size_t)b * S + j) * Hkv + kh) * d;
        double a = 0.0;
        for (int i = 0; i < d; ++i) a += (double)q[i] * (double)k[i];
        a *= scale;
        logits[j] = a;
        if (a > m) m = a;
        any = 1;
    }
    for (int i = 0; i < d; ++i) out[i] = 0.0;
    if (!any) return;
    double denom = 0.0;
    for (int j = lo; j <= t; ++j) {
        if (visible_mask && !visible_mask[j]) continue;
        double p = exp(logits[j] - m);
        denom += p;
        const float *v = V + (((size_t)b * S + j) * Hkv + kh) * d;
        for (int i = 0; i < d; ++i) out[i] += p * (double)v[i];
    }
    for (int i = 0; i < d; ++i) out[i] /= denom;
}

/*
 * Step a5: causal (optionally sliding-window) softmax attention for retained
 * tokens only; a pruned token's attention output is zero (Section 3.2: "the
 * attention output for that token is replaced with zero").
 *
 * Q [B,S,Hq,d], K,V [B,S,Hkv,d]; query head q reads kv head q / (Hq/Hkv).
 * Key j is visible to query t iff max(0, t-window+1) <= j <= t (window 0 = all
 * j <= t) and, in KV_RETAINED mode, keep_mask[b,j] == 1.
 * keep_mask [B,S]; O [B,S,Hq,d] double, every row written.
 */
void tfo_pruned_attention(const float *Q, const float *K, const float *V,
                          int B, int S, int Hq, int Hkv, int d, int window, double scale,
                          const uint8_t *keep_mask, int kv_visibility, double *O)
{
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int qh = 0; qh < Hq; ++qh) {
            double *logits = (double *)malloc(sizeof(double) * (size_t)(S > 0 ? S : 1));
            const uint8_t *vis = (kv_visibility == TFO_KV_RETAINED) ? keep_mask + (size_t)b * S : NULL;
            for (int t = 0; t < S; ++t) {
                double *o = O + (((size_t)b * S + t) * Hq + qh) * d;
                if (!keep_mask[(size_t)b * S + t]) {
                    for (int i = 0; i < d; ++i) o[i] = 0.0;
                    continue;
                }
                attention_row(Q, K, V, S, Hq, Hkv, d, window, scale, b, t, qh, vis, o, logits);
            }
            free(logits);
        }
    }
}

/*
 * The same rows, one at a time, for spot checks at sizes where the full output
 * is too much work: rows[i] = (b, t, q head); out [n_rows, d].  A row whose
 * token is pruned comes back zero.
 */
void tfo_attention_rows(const float *Q, const float *K, const float *V,
                        int B, int S, int Hq, int Hkv, int d, int window, double scale,
                        const uint8_t *keep_mask, int kv_visibility,
                        const int32_t *rows, int n_rows, double *out)
{
    (void)B;
#pragma omp parallel for schedule(dynamic, 8)
    for (int r = 0; r < n_rows; ++r) {
        int b = rows[3 * r + 0], t = rows[3 * r + 1], qh = rows[3 * r + 2];
        double *o = out + (size_t)r * d;
        if (!keep_mask[(size_t)b * S + t]) {
            for (int i = 0; i < d; ++i) o[i] = 0.0;
            continue;
        }
        double *logits = (double *)malloc(sizeof(double) * (size_t)S);
        const uint8_t *vis = (kv_visibility == TFO_KV_RETAINED) ? keep_mask + (size_t)b * S : NULL;
        attention_row(Q, K, V, S, Hq, Hkv, d, window, scale, b, t, qh, vis, o, logits);
        free(logits);
    }
}

/* how many threads the parallel loops above will use */
#ifdef _OPENMP
#include <omp.h>
int tfo_num_threads(void) { return omp_get_max_threads(); }
void tfo_set_num_threads(int n) { omp_set_num_threads(n); }
#else
int tfo_num_threads(void) { return 1; }
void tfo_set_num_threads(int n) { (void)n; }
#endif
