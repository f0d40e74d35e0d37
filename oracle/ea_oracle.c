/*
 * fp64 CPU oracle for Expected Attention KV-cache scoring and pruning.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what
 * the method computes, used to check the CUDA library and to provide a timed
 * CPU baseline.  It shares no code, header, table or constant with the CUDA
 * path and must never be called from it.
 *
 * Everything is double precision.  bf16 inputs are widened exactly.  Loops are
 * written in the order of the paper's equations with no blocking or fusion;
 * OpenMP only spreads independent (unit, head) problems over cores.
 *
 * Notation (paper Sec. 2): d head dimension, W window queries u_w (pre-RoPE),
 * n cached keys k_i (post-RoPE), T future positions, Hq query heads, Hkv KV
 * heads, G = Hq/Hkv, query head h reads KV head h / G.
 *
 * Parity status: every function below is pinned by tests against closed
 * forms, library routines, sampling or brute force.  Numeric agreement with
 * the authors' own implementation is UNPINNED: the paper prints no worked
 * example, so parity is to the paper's definitions only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { EAO_ROPE_HALF_SPLIT = 0, EAO_ROPE_INTERLEAVED = 1 };
enum { EAO_GROUP_MEAN_PROB = 0, EAO_GROUP_SUM_PROB = 1, EAO_GROUP_MEAN_LOGIT = 2 };
enum { EAO_COV_POPULATION = 0, EAO_COV_SAMPLE = 1 };

static double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int eao_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void eao_set_num_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* Channel indices (a, b) of rotation pair m.  Half-split pairs channel m with
 * m + d/2; interleaved pairs 2m with 2m + 1. */
static void pair_channels(int layout, int d, int m, int *a, int *b) {
    if (layout == EAO_ROPE_INTERLEAVED) { *a = 2 * m; *b = 2 * m + 1; }
    else                                { *a = m;     *b = m + d / 2; }
}

/*
 * Query statistics (Eq. 5 with the queries given directly; the listing's
 * compute_statistics step).  For each of n_heads windows q[W][d]:
 *   mu = (1/W) sum_w u_w,   Sigma = (1/N) sum_w (u_w - mu)(u_w - mu)^T,
 * N = W (population) or W - 1 (sample).
 */
void eao_mean_cov(const uint16_t *q_win, int64_t n_heads, int W, int d, int cov_norm,
                  double *mu, double *sigma) {
    double denom = (cov_norm == EAO_COV_SAMPLE) ? (double)(W - 1) : (double)W;
#pragma omp parallel for schedule(dynamic)
    for (int64_t h = 0; h < n_heads; ++h) {
        const uint16_t *q = q_win + h * (int64_t)W * d;
        double *m = mu + h * d;
        double *S = sigma + h * (int64_t)d * d;
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int w = 0; w < W; ++w) acc += bf16_to_f64(q[(int64_t)w * d + c]);
            m[c] = acc / (double)W;
        }
        for (int a = 0; a < d; ++a)
            for (int b = 0; b < d; ++b) {
                double acc = 0.0;
                for (int w = 0; w < W; ++w)
                    acc += (bf16_to_f64(q[(int64_t)w * d + a]) - m[a]) *
                           (bf16_to_f64(q[(int64_t)w * d + b]) - m[b]);
                S[(int64_t)a * d + b] = acc / denom;
            }
    }
}

/*
 * Query statistics from hidden states (Eq. 5 as the paper writes it): the hidden
 * states of a unit, h_w (W rows of d_model), have mean mu_h and covariance
 * Sigma_h; the queries of head j are q = W_Q^j h (pre-RoPE), so
 *   mu_j = W_Q^j mu_h,     Sigma_j = W_Q^j Sigma_h W_Q^j^T.
 * hidden: bf16 [n_units, W, dm]; w_q: bf16 [n_sets, Hq * d, dm], units are set-major: unit u uses
 * set u / (n_units / n_sets) (row j * d + c of a set is row c of W_Q^j).  Sigma_h is built in
 * full (dm x dm) and the two products are plain triple loops.
 */
void eao_hidden_mean_cov(const uint16_t *hidden, const uint16_t *w_q, int n_units, int n_sets, int Hq,
                         int W, int d, int dm, int cov_norm, double *mu, double *sigma) {
    double denom = (cov_norm == EAO_COV_SAMPLE) ? (double)(W - 1) : (double)W;
    for (int u = 0; u < n_units; ++u) {
        const uint16_t *H = hidden + (int64_t)u * W * dm;
        const uint16_t *WQ = w_q + (int64_t)(u / (n_units / n_sets)) * Hq * d * dm;
        double *mh = (double *)calloc((size_t)dm, sizeof(double));
        double *Sh = (double *)calloc((size_t)dm * dm, sizeof(double));
        for (int a = 0; a < dm; ++a) {
            double acc = 0.0;
            for (int w = 0; w < W; ++w) acc += bf16_to_f64(H[(int64_t)w * dm + a]);
            mh[a] = acc / (double)W;
        }
#pragma omp parallel for schedule(static)
        for (int a = 0; a < dm; ++a)
            for (int b = 0; b < dm; ++b) {
                double acc = 0.0;
                for (int w = 0; w < W; ++w)
                    acc += (bf16_to_f64(H[(int64_t)w * dm + a]) - mh[a]) *
                           (bf16_to_f64(H[(int64_t)w * dm + b]) - mh[b]);
                Sh[(int64_t)a * dm + b] = acc / denom;
            }
#pragma omp parallel for schedule(dynamic)
        for (int j = 0; j < Hq; ++j) {
            const uint16_t *Wj = WQ + (int64_t)j * d * dm;
            double *m = mu + ((int64_t)u * Hq + j) * d;
            double *S = sigma + ((int64_t)u * Hq + j) * d * d;
            double *tmp = (double *)calloc((size_t)d * dm, sizeof(double));      /* W_Q Sigma_h */
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int a = 0; a < dm; ++a) acc += bf16_to_f64(Wj[(int64_t)c * dm + a]) * mh[a];
                m[c] = acc;
            }
            for (int c = 0; c < d; ++c)
                for (int b = 0; b < dm; ++b) {
                    double acc = 0.0;
                    for (int a = 0; a < dm; ++a)
                        acc += bf16_to_f64(Wj[(int64_t)c * dm + a]) * Sh[(int64_t)a * dm + b];
                    tmp[(int64_t)c * dm + b] = acc;
                }
            for (int c = 0; c < d; ++c)
                for (int e = 0; e < d; ++e) {
                    double acc = 0.0;
                    for (int b = 0; b < dm; ++b)
                        acc += tmp[(int64_t)c * dm + b] * bf16_to_f64(Wj[(int64_t)e * dm + b]);
                    S[(int64_t)c * d + e] = acc;
                }
            free(tmp);
        }
        free(Sh);
        free(mh);
    }
}

/*
 * Averaged RoPE rotation (Eq. 6): R_bar = (1/T) sum_j R_p over the T future
 * positions p = pos_next .. pos_next + T - 1 (0-based positions; the paper's
 * t+1 .. t+T with 1-based keys 1..t).  R_p is block diagonal with one 2x2
 * rotation by angle p * theta_m per pair, theta_m = base^(-2m/d).  The average
 * of each block is [[cbar, -sbar], [sbar, cbar]] with cbar, sbar the means of
 * cos and sin.  Explicit sum, no closed form.
 */
void eao_rope_average(const int64_t *pos_next, int n_units, int T, double rope_base, int d,
                      double *cbar, double *sbar) {
    int half = d / 2;
    for (int u = 0; u < n_units; ++u)
        for (int m = 0; m < half; ++m) {
            double theta = pow(rope_base, -2.0 * (double)m / (double)d);
            double c = 0.0, s = 0.0;
            for (int j = 0; j < T; ++j) {
                double ang = (double)(pos_next[u] + j) * theta;
                c += cos(ang);
                s += sin(ang);
            }
            cbar[(int64_t)u * half + m] = c / (double)T;
            sbar[(int64_t)u * half + m] = s / (double)T;
        }
}

/*
 * Position-averaged Gaussian (Eq. 6): mu_bar = R_bar mu, Sigma_bar = R_bar
 * Sigma R_bar^T.  R_bar is built as a dense d x d matrix and the products are
 * written out as plain triple loops.
 */
void eao_apply_rope_average(const double *mu, const double *sigma, const double *cbar,
                            const double *sbar, int n_units, int Hq, int d, int layout,
                            double *mu_bar, double *sigma_bar) {
    int half = d / 2;
#pragma omp parallel for schedule(dynamic)
    for (int64_t uh = 0; uh < (int64_t)n_units * Hq; ++uh) {
        int u = (int)(uh / Hq);
        double *R = (double *)calloc((size_t)d * d, sizeof(double));
        double *tmp = (double *)calloc((size_t)d * d, sizeof(double));
        for (int m = 0; m < half; ++m) {
            int a, b;
            pair_channels(layout, d, m, &a, &b);
            double c = cbar[(int64_t)u * half + m], s = sbar[(int64_t)u * half + m];
            R[(int64_t)a * d + a] = c;  R[(int64_t)a * d + b] = -s;
            R[(int64_t)b * d + a] = s;  R[(int64_t)b * d + b] = c;
        }
        const double *m_in = mu + uh * d;
        const double *S = sigma + uh * (int64_t)d * d;
        double *m_out = mu_bar + uh * d;
        double *S_out = sigma_bar + uh * (int64_t)d * d;
        for (int i = 0; i < d; ++i) {
            double acc = 0.0;
            for (int j = 0; j < d; ++j) acc += R[(int64_t)i * d + j] * m_in[j];
            m_out[i] = acc;
        }
        for (int i = 0; i < d; ++i)            /* tmp = R Sigma */
            for (int j = 0; j < d; ++j) {
                double acc = 0.0;
                for (int l = 0; l < d; ++l) acc += R[(int64_t)i * d + l] * S[(int64_t)l * d + j];
                tmp[(int64_t)i * d + j] = acc;
            }
        for (int i = 0; i < d; ++i)            /* Sigma_bar = tmp R^T */
            for (int j = 0; j < d; ++j) {
                double acc = 0.0;
                for (int l = 0; l < d; ++l) acc += tmp[(int64_t)i * d + l] * R[(int64_t)j * d + l];
                S_out[(int64_t)i * d + j] = acc;
            }
        free(R);
        free(tmp);
    }
}

/*
 * Log of the expected unnormalised attention (Eq. 7):
 *   s_{h,i} = mu_bar_h . k_i / sqrt(d) + k_i^T Sigma_bar_h k_i / (2 d)
 * for every query head h and every key i of KV head h / G.  Kept in the log
 * domain: exp(s) overflows for outlier-heavy activations.
 * k: bf16 [n_units, Hkv, n, d];  s: [n_units, Hq, n].
 */
void eao_logits(const uint16_t *k, const double *mu_bar, const double *sigma_bar, int n_units,
                int Hq, int Hkv, int64_t n, int d, double *s) {
    int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic)
    for (int64_t uh = 0; uh < (int64_t)n_units * Hq; ++uh) {
        int u = (int)(uh / Hq), h = (int)(uh % Hq), g = h / G;
        const double *m = mu_bar + uh * d;
        const double *S = sigma_bar + uh * (int64_t)d * d;
        const uint16_t *kk = k + ((int64_t)u * Hkv + g) * n * d;
        double *key = (double *)malloc((size_t)d * sizeof(double));
        for (int64_t i = 0; i < n; ++i) {
            for (int c = 0; c < d; ++c) key[c] = bf16_to_f64(kk[i * d + c]);
            double lin = 0.0, quad = 0.0;
            for (int a = 0; a < d; ++a) lin += m[a] * key[a];
            for (int a = 0; a < d; ++a)
                for (int b = 0; b < d; ++b) quad += key[a] * S[(int64_t)a * d + b] * key[b];
            s[uh * n + i] = lin / sqrt((double)d) + quad / (2.0 * (double)d);
        }
        free(key);
    }
}

/* log sum_i exp(x_i), max-subtracted. */
static double log_sum_exp(const double *x, int64_t n) {
    double mx = x[0];
    for (int64_t i = 1; i < n; ++i) if (x[i] > mx) mx = x[i];
    double acc = 0.0;
    for (int64_t i = 0; i < n; ++i) acc += exp(x[i] - mx);
    return mx + log(acc);
}

/*
 * Expected attention (Eq. 8), GQA reduction, and contribution score (Eq. 9
 * with ||v|| in place of ||W_o v||, as the paper's implementation note says):
 *   a_hat_{h,i} = exp(s_{h,i} - LSE_h)                      softmax over keys
 *   MEAN_PROB : a_{g,i} = (1/G) sum_{h in g} a_hat_{h,i}
 *   SUM_PROB  : a_{g,i} =       sum_{h in g} a_hat_{h,i}
 *   MEAN_LOGIT: a_{g,i} = softmax_i( (1/G) sum_{h in g} s_{h,i} )
 *   score_{g,i} = (a_{g,i} + eps) * ||v_{g,i}||_2
 * s: [n_units, Hq, n]; v: bf16 [n_units, Hkv, n, d]; score: [n_units, Hkv, n];
 * a_out (optional, may be NULL): [n_units, Hkv, n].
 */
void eao_scores(const double *s, const uint16_t *v, int n_units, int Hq, int Hkv, int64_t n,
                int d, double eps, int group_mode, double *score, double *a_out) {
    int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic)
    for (int64_t ug = 0; ug < (int64_t)n_units * Hkv; ++ug) {
        int u = (int)(ug / Hkv), g = (int)(ug % Hkv);
        double *a = (double *)calloc((size_t)n, sizeof(double));
        if (group_mode == EAO_GROUP_MEAN_LOGIT) {
            double *avg = (double *)calloc((size_t)n, sizeof(double));
            for (int j = 0; j < G; ++j) {
                const double *sh = s + ((int64_t)u * Hq + (int64_t)g * G + j) * n;
                for (int64_t i = 0; i < n; ++i) avg[i] += sh[i] / (double)G;
            }
            double lse = n > 0 ? log_sum_exp(avg, n) : 0.0;
            for (int64_t i = 0; i < n; ++i) a[i] = exp(avg[i] - lse);
            free(avg);
        } else {
            for (int j = 0; j < G; ++j) {
                const double *sh = s + ((int64_t)u * Hq + (int64_t)g * G + j) * n;
                double lse = n > 0 ? log_sum_exp(sh, n) : 0.0;
                for (int64_t i = 0; i < n; ++i) a[i] += exp(sh[i] - lse);
            }
            if (group_mode == EAO_GROUP_MEAN_PROB)
                for (int64_t i = 0; i < n; ++i) a[i] /= (double)G;
        }
        const uint16_t *vv = v + ug * n * d;
        for (int64_t i = 0; i < n; ++i) {
            double ss = 0.0;
            for (int c = 0; c < d; ++c) {
                double x = bf16_to_f64(vv[i * d + c]);
                ss += x * x;
            }
            score[ug * n + i] = (a[i] + eps) * sqrt(ss);
            if (a_out) a_out[ug * n + i] = a[i];
        }
        free(a);
    }
}

/*
 * Contribution score with the output projection (Eq. 9 as written, ||W_o v||).
 * The output projection W_o is [dm, Hq * d]; query head h multiplies the value it
 * reads by its own slice W_o^h = W_o[:, h*d : (h+1)*d], so the pair (g, i) leaves
 * the head-h branch with magnitude ||W_o^h v_{g,i}||.  Per query head
 *   c_{h,i} = (a_hat_{h,i} + eps) * ||W_o^h v_{g,i}||_2,    a_hat from Eq. 8,
 * and the heads of a group are reduced as the attention is:
 *   MEAN_PROB: score_{g,i} = (1/G) sum_{h in g} c_{h,i};   SUM_PROB: the plain sum.
 * w_o: bf16 [n_sets, dm, Hq * d], unit u uses set u / (n_units / n_sets).  The product W_o^h v
 * is formed explicitly (dm entries) and its norm taken.
 */
void eao_scores_wo(const double *s, const uint16_t *v, const uint16_t *w_o, int n_units, int n_sets,
                   int Hq, int Hkv, int64_t n, int d, int dm, double eps, int group_mode,
                   double *score) {
    int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic)
    for (int64_t ug = 0; ug < (int64_t)n_units * Hkv; ++ug) {
        int u = (int)(ug / Hkv), g = (int)(ug % Hkv);
        const uint16_t *Wo = w_o + (int64_t)(u / (n_units / n_sets)) * dm * Hq * d;
        const uint16_t *vv = v + ug * n * d;
        for (int64_t i = 0; i < n; ++i) score[ug * n + i] = 0.0;
        for (int j = 0; j < G; ++j) {
            int h = g * G + j;
            const double *sh = s + ((int64_t)u * Hq + h) * n;
            double lse = n > 0 ? log_sum_exp(sh, n) : 0.0;
            for (int64_t i = 0; i < n; ++i) {
                double ss = 0.0;
                for (int a = 0; a < dm; ++a) {
                    double y = 0.0;
                    for (int c = 0; c < d; ++c)
                        y += bf16_to_f64(Wo[(int64_t)a * Hq * d + (int64_t)h * d + c]) *
                             bf16_to_f64(vv[i * d + c]);
                    ss += y * y;
                }
                score[ug * n + i] += (exp(sh[i] - lse) + eps) * sqrt(ss);
            }
        }
        if (group_mode == EAO_GROUP_MEAN_PROB)
            for (int64_t i = 0; i < n; ++i) score[ug * n + i] /= (double)G;
    }
}

typedef struct { double score; int32_t idx; } eao_item;

/* Total order: higher score first; equal scores: lower index first. */
static int item_cmp(const void *pa, const void *pb) {
    const eao_item *a = (const eao_item *)pa, *b = (const eao_item *)pb;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

static int int_cmp(const void *pa, const void *pb) {
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/*
 * Eviction (the compression paragraph of Sec. 2.2): per head, sort all keys
 * by (score descending, index ascending), keep the first n_kept, and report
 * them in ascending index order.  score: [n_heads, n]; idx: [n_heads, n_kept].
 */
void eao_select(const double *score, int64_t n_heads, int64_t n, int64_t n_kept, int32_t *idx) {
#pragma omp parallel for schedule(dynamic)
    for (int64_t h = 0; h < n_heads; ++h) {
        eao_item *items = (eao_item *)malloc((size_t)(n > 0 ? n : 1) * sizeof(eao_item));
        for (int64_t i = 0; i < n; ++i) { items[i].score = score[h * n + i]; items[i].idx = (int32_t)i; }
        qsort(items, (size_t)n, sizeof(eao_item), item_cmp);
        int32_t *out = idx + h * n_kept;
        for (int64_t j = 0; j < n_kept; ++j) out[j] = items[j].idx;
        qsort(out, (size_t)n_kept, sizeof(int32_t), int_cmp);
        free(items);
    }
}

/* Compaction: out[h][j][:] = rows[h][idx[h][j]][:] for bf16 rows of length d. */
void eao_gather(const uint16_t *rows, const int32_t *idx, int64_t n_heads, int64_t n,
                int64_t n_kept, int d, uint16_t *out) {
    for (int64_t h = 0; h < n_heads; ++h)
        for (int64_t j = 0; j < n_kept; ++j)
            for (int c = 0; c < d; ++c)
                out[(h * n_kept + j) * d + c] = rows[(h * n + idx[h * n_kept + j]) * d + c];
}

/*
 * Head-adaptive eviction (the head-adaptive paragraph of Sec. 2.2, which adopts the
 * per-layer budget allocation of Ada-KV; the paper prints no formula, so the rule is
 * the published one: a safeguard share per head, the rest of the layer's budget to the
 * best remaining pairs of the layer whichever head they belong to).
 *
 * One unit = one layer of one sequence with Hkv heads of n keys.  Its budget is
 * Hkv * n_kept pairs.
 *   1. Safeguard: every head keeps its n_floor best keys
 *      (order: score descending, index ascending).
 *   2. The other Hkv * (n_kept - n_floor) places go to the best pairs not kept in
 *      step 1, over all heads of the unit
 *      (order: score descending, head ascending, index ascending).
 *   3. The kept indices of a head are reported ascending; heads are concatenated in
 *      head order: idx[u][offsets[u][g] .. offsets[u][g+1]) belongs to head g.
 * score: [n_units, Hkv, n]; idx: [n_units, Hkv * n_kept]; offsets: [n_units, Hkv + 1].
 * Needs 0 <= n_floor <= n_kept <= n.
 */
typedef struct { double score; int32_t head; int32_t idx; } eao_pair;

static int pair_cmp(const void *pa, const void *pb) {
    const eao_pair *a = (const eao_pair *)pa, *b = (const eao_pair *)pb;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    if (a->head != b->head) return (a->head > b->head) - (a->head < b->head);
    return (a->idx > b->idx) - (a->idx < b->idx);
}

void eao_select_adaptive(const double *score, int64_t n_units, int64_t Hkv, int64_t n, int64_t n_kept,
                         int64_t n_floor, int32_t *idx, int32_t *offsets) {
    const int64_t budget = Hkv * n_kept;
#pragma omp parallel for schedule(dynamic)
    for (int64_t u = 0; u < n_units; ++u) {
        const double *sc = score + u * Hkv * n;
        char *kept = (char *)calloc((size_t)(Hkv * n > 0 ? Hkv * n : 1), 1);
        eao_item *items = (eao_item *)malloc((size_t)(n > 0 ? n : 1) * sizeof(eao_item));
        eao_pair *rest = (eao_pair *)malloc((size_t)(Hkv * n > 0 ? Hkv * n : 1) * sizeof(eao_pair));
        /* step 1: the safeguard share of every head */
        for (int64_t g = 0; g < Hkv; ++g) {
            for (int64_t i = 0; i < n; ++i) { items[i].score = sc[g * n + i]; items[i].idx = (int32_t)i; }
            qsort(items, (size_t)n, sizeof(eao_item), item_cmp);
            for (int64_t j = 0; j < n_floor; ++j) kept[g * n + items[j].idx] = 1;
        }
        /* step 2: the rest of the budget over the whole unit */
        int64_t n_rest = 0;
        for (int64_t g = 0; g < Hkv; ++g)
            for (int64_t i = 0; i < n; ++i)
                if (!kept[g * n + i]) {
                    rest[n_rest].score = sc[g * n + i];
                    rest[n_rest].head = (int32_t)g;
                    rest[n_rest].idx = (int32_t)i;
                    ++n_rest;
                }
        qsort(rest, (size_t)n_rest, sizeof(eao_pair), pair_cmp);
        const int64_t places = budget - Hkv * n_floor;
        for (int64_t j = 0; j < places; ++j) kept[(int64_t)rest[j].head * n + rest[j].idx] = 1;
        /* step 3: ascending indices per head, heads in order */
        int32_t *out = idx + u * budget, *off = offsets + u * (Hkv + 1);
        int64_t pos = 0;
        for (int64_t g = 0; g < Hkv; ++g) {
            off[g] = (int32_t)pos;
            for (int64_t i = 0; i < n; ++i)
                if (kept[g * n + i]) out[pos++] = (int32_t)i;
        }
        off[Hkv] = (int32_t)pos;
        free(rest);
        free(items);
        free(kept);
    }
}

/* Ragged compaction: out[u][j][:] = rows[u][g][idx[u][j]][:] with g the head whose range holds j. */
void eao_gather_adaptive(const uint16_t *rows, const int32_t *idx, const int32_t *offsets, int64_t n_units,
                         int64_t Hkv, int64_t n, int64_t budget, int d, uint16_t *out) {
    for (int64_t u = 0; u < n_units; ++u)
        for (int64_t g = 0; g < Hkv; ++g)
            for (int64_t j = offsets[u * (Hkv + 1) + g]; j < offsets[u * (Hkv + 1) + g + 1]; ++j)
                for (int c = 0; c < d; ++c)
                    out[(u * budget + j) * d + c] = rows[((u * Hkv + g) * n + idx[u * budget + j]) * d + c];
}

/* Safeguard share floor(alpha * n_kept), evaluated in double. */
int64_t eao_n_floor(int64_t n_kept, double alpha) {
    double x = (double)n_kept * alpha;
    int64_t k = (int64_t)x;
    if (k < 0) k = 0;
    if (k > n_kept) k = n_kept;
    return k;
}

/* int(n * (1 - r)) evaluated in double, as the listing computes n_kept. */
int64_t eao_n_kept(int64_t n, double compression_ratio) {
    double x = (double)n * (1.0 - compression_ratio);
    int64_t k = (int64_t)x;            /* truncation toward zero */
    if (k < 0) k = 0;
    if (k > n) k = n;
    return k;
}
