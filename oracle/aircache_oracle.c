/*
 * AirCache CPU oracle  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, obviously-correct restatement of the compress-then-decode
 * path of AirCache (arXiv 2503.23956), one definition per function, fp64
 * arithmetic on the bf16-rounded inputs, no blocking, no fusion, no
 * vectorisation.  It shares no code with the CUDA library and is only ever
 * called by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Parity status of each function (what pins it to something other than
 * itself is listed in tests/test_oracle_pins.py):
 *   oracle_elite / oracle_score   Eq. 4-8   pinned (closed forms, library softmax, invariants)
 *   oracle_moments                Eq. 9-10  pinned (closed forms, scipy.stats.skew)
 *   oracle_allocate               Eq. 11, Alg. 1 second loop  pinned (brute-force apportionment, invariants)
 *   oracle_select                 Alg. 1 "I[N_v x r]"         pinned (subset enumeration)
 *   oracle_compact                Alg. 1 Concat(K_v[..], K_t) pinned (r = 1 identity, text rows)
 *   oracle_decode                 Section 3.1 token decoding  pinned (masked dense attention, library SDPA)
 *   oracle_score_groups, oracle_allocate_groups, oracle_compact_groups
 *                                 Eq. 8-11 and Alg. 1's second loop per KV group (a refinement the paper does not
 *                                 evaluate)  pinned (mean over groups = the per-layer score, budget sum, library sort)
 *   End-to-end against the authors' implementation: PARITY UNPINNED -- the
 *   paper prints no worked numerical example.
 *
 * Conventions.  bf16 tensors arrive as uint16_t bit patterns.  The full cache
 * is addressed with element strides (layer, batch, kv-head, token), head_dim
 * contiguous; tokens 0..Nv-1 are visual, Nv..Nv+Nt-1 are text (Eq. 3: X =
 * Concat(X_v, X_t)).  The observation-window candidates are the last W text
 * tokens; candidate w is token Nv+Nt-W+w and the reference row of Eq. 4 is the
 * last one (w = W-1).  All loops that are marked with an OpenMP pragma run
 * independent work items; the arithmetic of an item is unaffected.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

typedef struct {
    int32_t n_layers, batch, n_q_heads, n_kv_heads, head_dim;
    int32_t n_visual, n_text, window;
} oracle_dims_t;

/* fp64 dot product of two bf16 rows, c = 0..d-1 in order. */
static double dot_bf16(const uint16_t *a, const uint16_t *b, int d) {
    double acc = 0.0;
    for (int c = 0; c < d; ++c) acc += bf16_to_f64(a[c]) * bf16_to_f64(b[c]);
    return acc;
}

/*
 * Eq. 4-5: elite key-text-token set of one query head.
 * The last text token is the reference query.  Softmax is monotone and the
 * threshold is relative to the row maximum, so A[j] >= alpha * max A  <=>
 * t_j - t_max >= ln(alpha): the normaliser of A_tt cancels.  This decision is
 * an integer outcome of floating point, so it is taken in the precision the
 * CUDA path states for it: the fp64 dot product is rounded to fp32, scaled in
 * fp32, and the difference to the maximum is compared in fp32 with
 * (float)log((double)alpha).  alpha = 0 keeps every candidate.
 * Returns a W-bit mask (bit w set <=> candidate w is elite; W <= 128); logits_out
 * (may be NULL) receives the W fp32 logits.
 */
typedef unsigned __int128 mask128_t;   /* one bit per candidate, W <= 128 */

static mask128_t elite_of_head(const uint16_t *q_last, const uint16_t *k_cand0, int64_t k_stride_token,
                               int W, int d, float scale, float alpha, float *logits_out) {
    float t[128];
    float tmax = -INFINITY;
    for (int w = 0; w < W; ++w) {
        float dotf = (float)dot_bf16(q_last, k_cand0 + (int64_t)w * k_stride_token, d);
        t[w] = dotf * scale;
        if (t[w] > tmax) tmax = t[w];
        if (logits_out) logits_out[w] = t[w];
    }
    mask128_t mask = 0;
    if (alpha <= 0.0f) {
        for (int w = 0; w < W; ++w) mask |= (mask128_t)1 << w;
        return mask;
    }
    float ln_alpha = (float)log((double)alpha);
    for (int w = 0; w < W; ++w) {
        float diff = t[w] - tmax;
        if (diff >= ln_alpha) mask |= (mask128_t)1 << w;
    }
    return mask;
}

/*
 * Eq. 4-8 for every (layer, sequence): importance score of each visual token.
 *   k            bf16 full key cache, strides in elements
 *   q_window     bf16 [L, B, W, Hq, d] contiguous: queries of the W candidate text tokens
 *   scores       fp32 [L, B, Nv]      (output)  I_v, rounded to fp32 once at the end
 *   elite_mask   u64  [L, B, Hq, ceil(W/64)]  (output, may be NULL) candidate w is bit w % 64 of word w / 64
 *   text_mass    f64  [L, B, Hq]      (output, may be NULL) mean over elite rows of the
 *                                     softmax mass that fell on text keys (for the sum-to-one pin)
 *   elite_logits fp32 [L, B, Hq, W]   (output, may be NULL) the Eq. 4 logits the decision used
 * Per query head h (KV head g = h / (Hq/Hkv)):
 *   E_h from Eq. 5; for each elite row w the softmax of Eq. 7 runs over all Nv
 *   visual keys plus the elite text keys w' <= w (causal among text; non-elite
 *   text keys are not part of K_vtk, Eq. 6); Eq. 8 averages the visual columns
 *   over the elite rows.  The per-layer score is the plain mean over the Hq heads.
 */
static int score_worker(const oracle_dims_t *dm, const uint16_t *k, int64_t s_layer, int64_t s_batch,
                        int64_t s_head, int64_t s_token, const uint16_t *q_window, float scale, float alpha,
                        float *scores, uint64_t *elite_mask, double *text_mass, float *elite_logits,
                        float *group_scores);

int oracle_score(const oracle_dims_t *dm, const uint16_t *k, int64_t s_layer, int64_t s_batch,
                 int64_t s_head, int64_t s_token, const uint16_t *q_window, float scale, float alpha,
                 float *scores, uint64_t *elite_mask, double *text_mass, float *elite_logits) {
    return score_worker(dm, k, s_layer, s_batch, s_head, s_token, q_window, scale, alpha, scores, elite_mask,
                        text_mass, elite_logits, NULL);
}

/*
 * Eq. 4-8 with the importance kept apart per KV group (the per-KV-head refinement): group g's score of a visual
 * token is the plain mean of Eq. 8 over the query heads that read KV head g.
 *   group_scores  fp32 [L, B, Hkv, Nv]  (output), rounded to fp32 once at the end
 * The mean of the groups' scores over g is the per-layer score of oracle_score (groups have equal size).
 */
int oracle_score_groups(const oracle_dims_t *dm, const uint16_t *k, int64_t s_layer, int64_t s_batch,
                        int64_t s_head, int64_t s_token, const uint16_t *q_window, float scale, float alpha,
                        float *group_scores, uint64_t *elite_mask) {
    return score_worker(dm, k, s_layer, s_batch, s_head, s_token, q_window, scale, alpha, NULL, elite_mask, NULL,
                        NULL, group_scores);
}

static int score_worker(const oracle_dims_t *dm, const uint16_t *k, int64_t s_layer, int64_t s_batch,
                        int64_t s_head, int64_t s_token, const uint16_t *q_window, float scale, float alpha,
                        float *scores, uint64_t *elite_mask, double *text_mass, float *elite_logits,
                        float *group_scores) {
    const int L = dm->n_layers, B = dm->batch, Hq = dm->n_q_heads, Hkv = dm->n_kv_heads;
    const int d = dm->head_dim, Nv = dm->n_visual, Nt = dm->n_text, W = dm->window;
    if (W < 1 || W > 128 || W > Nt || Hq % Hkv != 0 || Nv < 1) return -1;
    const int words = (W + 63) / 64;
    const int G = Hq / Hkv;
    const int N = Nv + Nt;
    int status = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int l = 0; l < L; ++l) {
        for (int b = 0; b < B; ++b) {
            double *acc = (double *)calloc((size_t)Nv, sizeof(double));   /* sum over heads of I_h */
            double *acc_g = (double *)calloc((size_t)Nv, sizeof(double)); /* the same over the heads of one KV group */
            double *logit = (double *)malloc((size_t)Nv * sizeof(double));
            double *per_head = (double *)malloc((size_t)Nv * sizeof(double));
            if (!acc || !acc_g || !logit || !per_head) {
                status = -2; free(acc); free(acc_g); free(logit); free(per_head); continue;
            }
            const uint16_t *k_lb = k + (int64_t)l * s_layer + (int64_t)b * s_batch;
            const uint16_t *q_lb = q_window + ((int64_t)l * B + b) * (int64_t)W * Hq * d;
            for (int h = 0; h < Hq; ++h) {
                const int g = h / G;
                const uint16_t *k_g = k_lb + (int64_t)g * s_head;
                const uint16_t *q_last = q_lb + ((int64_t)(W - 1) * Hq + h) * d;
                float *lg = elite_logits ? elite_logits + (((int64_t)l * B + b) * Hq + h) * W : NULL;
                mask128_t E = elite_of_head(q_last, k_g + (int64_t)(N - W) * s_token, s_token, W, d, scale,
                                            alpha, lg);
                if (elite_mask)
                    for (int j = 0; j < words; ++j)
                        elite_mask[(((int64_t)l * B + b) * Hq + h) * words + j] = (uint64_t)(E >> (64 * j));
                int n_elite = 0;
                for (int w = 0; w < W; ++w) n_elite += (int)((E >> w) & 1);
                for (int i = 0; i < Nv; ++i) per_head[i] = 0.0;
                double tmass = 0.0;
                for (int w = 0; w < W; ++w) {
                    if (!((E >> w) & 1)) continue;
                    const uint16_t *q_w = q_lb + ((int64_t)w * Hq + h) * d;
                    /* Eq. 7 row: logits against K_vtk = Concat(K_v, K_t[k]), causal among text */
                    double m = -INFINITY;
                    for (int i = 0; i < Nv; ++i) {
                        logit[i] = (double)scale * dot_bf16(q_w, k_g + (int64_t)i * s_token, d);
                        if (logit[i] > m) m = logit[i];
                    }
                    double tl[128];
                    for (int w2 = 0; w2 <= w; ++w2) {
                        if (!((E >> w2) & 1)) continue;
                        tl[w2] = (double)scale * dot_bf16(q_w, k_g + (int64_t)(N - W + w2) * s_token, d);
                        if (tl[w2] > m) m = tl[w2];
                    }
                    double Z = 0.0;
                    for (int i = 0; i < Nv; ++i) Z += exp(logit[i] - m);
                    double Zt = 0.0;
                    for (int w2 = 0; w2 <= w; ++w2)
                        if ((E >> w2) & 1) Zt += exp(tl[w2] - m);
                    Z += Zt;
                    for (int i = 0; i < Nv; ++i) per_head[i] += exp(logit[i] - m) / Z;
                    tmass += Zt / Z;
                }
                /* Eq. 8: average pooling over the elite rows */
                for (int i = 0; i < Nv; ++i) acc[i] += per_head[i] / (double)n_elite;
                for (int i = 0; i < Nv; ++i) acc_g[i] += per_head[i] / (double)n_elite;
                if (text_mass) text_mass[((int64_t)l * B + b) * Hq + h] = tmass / (double)n_elite;
                if (h % G == G - 1) {   /* last head of KV group g: its mean, then start the next group */
                    if (group_scores) {
                        float *og = group_scores + (((int64_t)l * B + b) * Hkv + g) * Nv;
                        for (int i = 0; i < Nv; ++i) og[i] = (float)(acc_g[i] / (double)G);
                    }
                    for (int i = 0; i < Nv; ++i) acc_g[i] = 0.0;
                }
            }
            if (scores) {
                float *out = scores + ((int64_t)l * B + b) * Nv;
                for (int i = 0; i < Nv; ++i) out[i] = (float)(acc[i] / (double)Hq);
            }
            free(acc); free(acc_g); free(logit); free(per_head);
        }
    }
    return status;
}

/*
 * Eq. 9-10 on the fp32 scores: strength s_t = sum I_v; skewness s_k = adjusted
 * Fisher-Pearson coefficient  Nv/((Nv-1)(Nv-2)) * sum(((I - mu)/sigma)^3)  with the
 * sample standard deviation (ddof = 1).  sigma = 0 gives s_k = 0.  Needs Nv >= 3.
 */
int oracle_moments(const float *scores, int64_t n_regions, int32_t n_visual, double *strength,
                   double *skewness) {
    if (n_visual < 3) return -1;
    const double n = (double)n_visual;
    for (int64_t r = 0; r < n_regions; ++r) {
        const float *x = scores + r * n_visual;
        double s = 0.0;
        for (int i = 0; i < n_visual; ++i) s += (double)x[i];
        const double mu = s / n;
        double ss = 0.0;
        for (int i = 0; i < n_visual; ++i) { double c = (double)x[i] - mu; ss += c * c; }
        const double sigma = sqrt(ss / (n - 1.0));
        double cube = 0.0;
        if (sigma > 0.0)
            for (int i = 0; i < n_visual; ++i) { double z = ((double)x[i] - mu) / sigma; cube += z * z * z; }
        strength[r] = s;
        skewness[r] = (sigma > 0.0) ? n / ((n - 1.0) * (n - 2.0)) * cube : 0.0;
    }
    return 0;
}

/* Total visual rows one sequence keeps: round-half-up of ratio * (Nv * L). */
int64_t oracle_total_kept(int32_t n_visual, int32_t n_layers, double ratio) {
    int64_t cells = (int64_t)n_visual * (int64_t)n_layers;
    return (int64_t)floor(ratio * (double)cells + 0.5);
}

/*
 * Eq. 11 and the second loop of Algorithm 1, per sequence.
 *   mode 0: w_l = (s't + s'k)/2   1: w_l = s't   2: w_l = s'k   3: w_l = 1 (uniform)
 * "Normalised across layers" is read as division by the across-layer mean, the
 * reading that keeps the mean of r_hat equal to r; negative skewness counts as
 * 0; a zero mean makes that factor 1 for every layer.
 * The integer budgets n_l: T = round-half-up(ratio*Nv*L); proportional shares of
 * T by weight, with every layer capped at Nv and the excess re-shared among the
 * rest; floors, then the remaining units go one each to the largest fractional
 * parts, ties to the lower layer.
 *   strength, skewness  f64 [L, B];   budgets  i32 [L, B] (output)
 */
int oracle_allocate(const double *strength, const double *skewness, int32_t n_layers, int32_t batch,
                    int32_t n_visual, double ratio, int32_t mode, int32_t *budgets) {
    const int L = n_layers, B = batch;
    if (L < 1 || ratio < 0.0 || ratio > 1.0) return -1;
    double *w = (double *)malloc((size_t)L * sizeof(double));
    double *share = (double *)malloc((size_t)L * sizeof(double));
    char *active = (char *)malloc((size_t)L);
    if (!w || !share || !active) { free(w); free(share); free(active); return -2; }
    for (int b = 0; b < B; ++b) {
        double mean_t = 0.0, mean_k = 0.0;
        for (int l = 0; l < L; ++l) {
            mean_t += strength[(int64_t)l * B + b];
            double sk = skewness[(int64_t)l * B + b];
            mean_k += (sk > 0.0) ? sk : 0.0;
        }
        mean_t /= (double)L;
        mean_k /= (double)L;
        for (int l = 0; l < L; ++l) {
            double st = strength[(int64_t)l * B + b];
            double sk = skewness[(int64_t)l * B + b];
            if (sk < 0.0) sk = 0.0;
            double nt = (mean_t > 0.0) ? st / mean_t : 1.0;
            double nk = (mean_k > 0.0) ? sk / mean_k : 1.0;
            if (mode == 0) w[l] = 0.5 * (nt + nk);
            else if (mode == 1) w[l] = nt;
            else if (mode == 2) w[l] = nk;
            else w[l] = 1.0;
            active[l] = 1;
        }
        int64_t R = oracle_total_kept(n_visual, L, ratio);
        int32_t *n = budgets + b;   /* n[l*B] */
        /* capped proportional split */
        for (;;) {
            double wsum = 0.0;
            int n_active = 0;
            for (int l = 0; l < L; ++l) if (active[l]) { wsum += w[l]; ++n_active; }
            if (n_active == 0) break;
            int moved = 0;
            for (int l = 0; l < L; ++l) {
                if (!active[l]) continue;
                share[l] = (wsum > 0.0) ? (double)R * w[l] / wsum : (double)R / (double)n_active;
            }
            for (int l = 0; l < L; ++l) {
                if (active[l] && share[l] >= (double)n_visual) {
                    n[(int64_t)l * B] = n_visual;
                    active[l] = 0;
                    R -= n_visual;
                    moved = 1;
                }
            }
            if (!moved) break;
        }
        /* floors, then largest remainders (ties -> lower layer) */
        int64_t given = 0;
        for (int l = 0; l < L; ++l) {
            if (!active[l]) continue;
            int32_t f = (int32_t)floor(share[l]);
            n[(int64_t)l * B] = f;
            given += f;
            share[l] -= (double)f;           /* fractional part */
        }
        for (int64_t left = R - given; left > 0; --left) {
            int best = -1;
            for (int l = 0; l < L; ++l)
                if (active[l] && (best < 0 || share[l] > share[best])) best = l;
            if (best < 0) break;
            n[(int64_t)best * B] += 1;
            active[best] = 0;                /* at most one extra unit per layer */
        }
    }
    free(w); free(share); free(active);
    return 0;
}

/*
 * Alg. 1 "K_v(I[N_v x r_hat])": the n visual tokens of largest score, equal
 * scores -> the lower token index wins; emitted in ascending token order.
 * Selection by repeated scan for the best remaining token (no sort library).
 */
int oracle_select(const float *scores, int32_t n_visual, int32_t n_keep, int32_t *kept) {
    if (n_keep < 0 || n_keep > n_visual) return -1;
    char *taken = (char *)calloc((size_t)n_visual + 1, 1);
    if (!taken) return -2;
    for (int j = 0; j < n_keep; ++j) {
        int best = -1;
        for (int i = 0; i < n_visual; ++i) {
            if (taken[i]) continue;
            if (best < 0 || scores[i] > scores[best]) best = i;   /* strict > keeps the lower index on ties */
        }
        taken[best] = 1;
    }
    int o = 0;
    for (int i = 0; i < n_visual; ++i) if (taken[i]) kept[o++] = i;
    free(taken);
    return 0;
}

/*
 * Alg. 1 second loop for every (layer, sequence): select, then
 *   K' = Concat(K_v[kept], K_t),  V' = Concat(V_v[kept], V_t)
 * written as rows of [Hkv, d] into one packed ragged buffer; region (l,b) has index
 * r = l*B + b and starts at row offsets[r] = sum over r' < r of (budget[r'] + Nt + slack).
 *   kept_idx  i32, region r's list at position offsets[r] - r*(Nt+slack)   (output)
 *   offsets   i64 [L*B + 1], lens i32 [L*B]                               (outputs)
 */
int oracle_compact(const oracle_dims_t *dm, int32_t slack, const uint16_t *k, const uint16_t *v,
                   int64_t s_layer, int64_t s_batch, int64_t s_head, int64_t s_token, const float *scores,
                   const int32_t *budgets, uint16_t *k_out, uint16_t *v_out, int64_t *offsets, int32_t *lens,
                   int32_t *kept_idx) {
    const int L = dm->n_layers, B = dm->batch, Hkv = dm->n_kv_heads, d = dm->head_dim;
    const int Nv = dm->n_visual, Nt = dm->n_text;
    int64_t row = 0, kept_pos = 0;
    for (int l = 0; l < L; ++l) {
        for (int b = 0; b < B; ++b) {
            const int64_t r = (int64_t)l * B + b;
            const int32_t n = budgets[r];
            offsets[r] = row;
            lens[r] = n + Nt;
            int32_t *kept = kept_idx + kept_pos;
            int rc = oracle_select(scores + r * Nv, Nv, n, kept);
            if (rc) return rc;
            for (int j = 0; j < n + Nt; ++j) {
                const int64_t tok = (j < n) ? kept[j] : (int64_t)Nv + (j - n);
                for (int g = 0; g < Hkv; ++g) {
                    const int64_t src = (int64_t)l * s_layer + (int64_t)b * s_batch + (int64_t)g * s_head +
                                        tok * s_token;
                    const int64_t dst = ((row + j) * Hkv + g) * d;
                    memcpy(k_out + dst, k + src, (size_t)d * sizeof(uint16_t));
                    memcpy(v_out + dst, v + src, (size_t)d * sizeof(uint16_t));
                }
            }
            row += n + Nt + slack;
            kept_pos += n;
        }
    }
    offsets[(int64_t)L * B] = row;
    return 0;
}

/*
 * Eq. 11 per KV group: the cells (layer, KV head) of one sequence take the place of the layers.  Strength and
 * skewness are normalised by their mean over the L * Hkv cells of the sequence, and T = round-half-up(ratio * Nv *
 * L * Hkv) rows are split over the cells exactly as oracle_allocate splits a sequence's rows over its layers
 * (cell order: layer-major, KV head within the layer; ties to the lower cell).
 *   strength, skewness  f64 [L, B, Hkv];   budgets  i32 [L, B, Hkv] (output)
 */
int oracle_allocate_groups(const double *strength, const double *skewness, int32_t n_layers, int32_t batch,
                           int32_t n_kv_heads, int32_t n_visual, double ratio, int32_t mode, int32_t *budgets) {
    const int cells = n_layers * n_kv_heads;
    double *st = (double *)malloc((size_t)cells * sizeof(double));
    double *sk = (double *)malloc((size_t)cells * sizeof(double));
    int32_t *bud = (int32_t *)malloc((size_t)cells * sizeof(int32_t));
    if (!st || !sk || !bud) { free(st); free(sk); free(bud); return -2; }
    int rc = 0;
    for (int b = 0; b < batch && !rc; ++b) {
        for (int l = 0; l < n_layers; ++l)
            for (int g = 0; g < n_kv_heads; ++g) {
                const int64_t at = ((int64_t)l * batch + b) * n_kv_heads + g;
                st[l * n_kv_heads + g] = strength[at];
                sk[l * n_kv_heads + g] = skewness[at];
            }
        rc = oracle_allocate(st, sk, cells, 1, n_visual, ratio, mode, bud);   /* the cells as the layers of one sequence */
        for (int l = 0; l < n_layers; ++l)
            for (int g = 0; g < n_kv_heads; ++g)
                budgets[((int64_t)l * batch + b) * n_kv_heads + g] = bud[l * n_kv_heads + g];
    }
    free(st); free(sk); free(bud);
    return rc;
}

/*
 * Alg. 1's second loop per KV group: cell (l, b, g) keeps its own budgets[l, b, g] visual tokens of largest
 * group score and all text tokens; rows are single-head rows of d elements.  Cell index c = (l*B + b)*Hkv + g,
 * first row offsets[c] = sum over c' < c of (budget[c'] + Nt + slack).
 *   k_out, v_out  bf16 [rows, d];  offsets i64 [L*B*Hkv + 1];  lens i32 [L*B*Hkv];  kept_idx packed per cell
 */
int oracle_compact_groups(const oracle_dims_t *dm, int32_t slack, const uint16_t *k, const uint16_t *v,
                          int64_t s_layer, int64_t s_batch, int64_t s_head, int64_t s_token,
                          const float *group_scores, const int32_t *budgets, uint16_t *k_out, uint16_t *v_out,
                          int64_t *offsets, int32_t *lens, int32_t *kept_idx) {
    const int L = dm->n_layers, B = dm->batch, Hkv = dm->n_kv_heads, d = dm->head_dim;
    const int Nv = dm->n_visual, Nt = dm->n_text;
    int64_t row = 0, kept_pos = 0;
    for (int64_t c = 0; c < (int64_t)L * B * Hkv; ++c) {
        const int g = (int)(c % Hkv), b = (int)(c / Hkv % B), l = (int)(c / Hkv / B);
        const int32_t n = budgets[c];
        offsets[c] = row;
        lens[c] = n + Nt;
        int32_t *kept = kept_idx + kept_pos;
        int rc = oracle_select(group_scores + c * Nv, Nv, n, kept);
        if (rc) return rc;
        for (int j = 0; j < n + Nt; ++j) {
            const int64_t tok = (j < n) ? kept[j] : (int64_t)Nv + (j - n);
            const int64_t src = (int64_t)l * s_layer + (int64_t)b * s_batch + (int64_t)g * s_head + tok * s_token;
            memcpy(k_out + (row + j) * d, k + src, (size_t)d * sizeof(uint16_t));
            memcpy(v_out + (row + j) * d, v + src, (size_t)d * sizeof(uint16_t));
        }
        row += n + Nt + slack;
        kept_pos += n;
    }
    offsets[(int64_t)L * B * Hkv] = row;
    return 0;
}

/*
 * Section 3.1 token decoding: one query token per (layer, sequence, query head)
 * attends to that region of the compressed cache:
 *   o_h = sum_j softmax_j(scale * <q_h, K'_g[j]>) * V'_g[j],   g = h / (Hq/Hkv)
 *   k_c, v_c  bf16 [rows, Hkv, d];  q bf16 [L, B, Hq, d];  out fp32 [L, B, Hq, d]
 */
int oracle_decode(const oracle_dims_t *dm, const uint16_t *k_c, const uint16_t *v_c, const int64_t *offsets,
                  const int32_t *lens, const uint16_t *q, float scale, float *out) {
    const int L = dm->n_layers, B = dm->batch, Hq = dm->n_q_heads, Hkv = dm->n_kv_heads, d = dm->head_dim;
    const int G = Hq / Hkv;
    const int64_t n_items = (int64_t)L * B * Hq;
#pragma omp parallel for schedule(dynamic)
    for (int64_t it = 0; it < n_items; ++it) {
        const int64_t r = it / Hq;
        const int h = (int)(it % Hq), g = h / G;
        const int len = lens[r];
        const uint16_t *qh = q + it * d;
        float *o = out + it * d;
        double *p = (double *)malloc((size_t)(len > 0 ? len : 1) * sizeof(double));
        double m = -INFINITY;
        for (int j = 0; j < len; ++j) {
            p[j] = (double)scale * dot_bf16(qh, k_c + ((offsets[r] + j) * Hkv + g) * d, d);
            if (p[j] > m) m = p[j];
        }
        double Z = 0.0;
        for (int j = 0; j < len; ++j) { p[j] = exp(p[j] - m); Z += p[j]; }
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int j = 0; j < len; ++j) acc += p[j] * bf16_to_f64(v_c[((offsets[r] + j) * Hkv + g) * d + c]);
            o[c] = (len > 0) ? (float)(acc / Z) : 0.0f;
        }
        free(p);
    }
    return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
