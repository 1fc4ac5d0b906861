/*
 * CPU oracle for the STILL intra-layer hybrid attention layer forward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision
 * statement of what the layer computes.  It shares no code with the CUDA
 * library and must never be called from the product path; only the tests, the
 * smoke check and the CPU-baseline leg of the benchmark execute it.
 *
 * Two independent formulations are given, as in the paper:
 *   - still_oracle_recurrent : the Recurrent Form of Sec. 3.3 (delayed
 *     selection Eq. "delayed_selection", cache routing Eq. "cache_routing_sum",
 *     merge y = (N_SA+N_LA)/(D_SA+D_LA)), stepping one token at a time with
 *     explicit containers h, s, z; the score is taken token-wise from the
 *     window-set definition of Sec. 3.1.
 *   - still_oracle_chunkwise : Algorithm 1 (Chunk-Wise Parallel Form), chunk
 *     tiles s_in / s_prev with the masks M_down, M_up, M_diag, Top(S, lambda),
 *     the cumulative LA state lagged by two chunks, the SA branch over
 *     [selected of chunks <= t-2, chunk t-1, causal chunk t].
 * The paper claims both have the same routing and memory-update behaviour; a
 * test checks that they agree.
 *
 * Readings of the paper taken here (each one is listed in the design notes):
 *   - logits are sm_scale * q.k in the score and in the SA branch; the NP-Map
 *     sees the raw q and k;
 *   - a masked logit is excluded from its softmax (it is not set to zero);
 *     the first chunk has no previous chunk;
 *   - a token that is alone in its window has an all-zero a_nodiag;
 *   - f(x) = xW + b, a single linear map of width d_f, feature dim d' = 2 d_f;
 *   - only tokens of M^LA enter the LA state (the routing equation governs),
 *     z is a vector of d' entries;
 *   - the gate multiplies N_LA only;
 *   - Top-lambda uses the total order (score descending, index ascending),
 *     NaN ranks lowest, and the result is listed in ascending index order;
 *   - salient-cache budget (max_salient > 0; 0 = unbounded, the routing equation
 *     as written): the paper's long-context experiments cap the number of cached
 *     salient tokens but the method section gives no rule.  PARITY UNPINNED for the
 *     choice of rule.  The rule taken here: tokens enter the salient cache in
 *     routing order; whenever it holds more than max_salient tokens the oldest is
 *     removed and folded into (s, z) through phi_k exactly like an unselected
 *     token, so every token outside the local region is counted exactly once.
 *
 * Indices are 0-based here: token i (0-based) is in chunk i / C; the paper's
 * token t is i+1 and its chunk c is i/C + 1.
 *
 * Pins (see tests/test_oracle_*.py): closed forms of the score, brute force on
 * tiny inputs, lambda = C against textbook causal softmax attention, lambda = 0
 * against textbook normalised linear attention over the lagged prefix, NP-Map
 * norm / sum invariants, constant-V invariance, partition invariant, and the
 * agreement of the two formulations.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------ */
/* small helpers                                                            */
/* ------------------------------------------------------------------------ */

static double dotd(const double *a, const double *b, int d) {
    double s = 0.0;
    for (int i = 0; i < d; ++i) s += a[i] * b[i];
    return s;
}

/* softmax of n values in place (n >= 1). */
static void softmax_inplace(double *x, int n) {
    double m = x[0];
    for (int i = 1; i < n; ++i)
        if (x[i] > m) m = x[i];
    double z = 0.0;
    for (int i = 0; i < n; ++i) {
        x[i] = exp(x[i] - m);
        z += x[i];
    }
    for (int i = 0; i < n; ++i) x[i] /= z;
}

/* ------------------------------------------------------------------------ */
/* Self-Saliency Score, token-wise (Sec. 3.1: window set W_t, a_diag,        */
/* a_nodiag, Score_t).                                                       */
/* ------------------------------------------------------------------------ */

void still_oracle_score_tokenwise(const double *q, const double *k, int64_t N, int d, int w,
                                  double sm_scale, double eps, double *score) {
    double *ad = (double *)malloc(sizeof(double) * (size_t)w);
    double *an = (double *)malloc(sizeof(double) * (size_t)w);
    for (int64_t t = 0; t < N; ++t) {
        int64_t lo = t - w + 1;
        if (lo < 0) lo = 0;
        int n = (int)(t - lo + 1); /* |W_t|, the last entry is j = t */
        for (int j = 0; j < n; ++j) ad[j] = sm_scale * dotd(q + t * d, k + (lo + j) * d, d);
        for (int j = 0; j < n - 1; ++j) an[j] = ad[j];
        softmax_inplace(ad, n);
        if (n > 1) softmax_inplace(an, n - 1);
        an[n - 1] = 0.0; /* j = t */
        double s = 0.0;
        for (int j = 0; j < n; ++j) s += ad[j] * log((ad[j] + eps) / (an[j] + eps));
        score[t] = s;
    }
    free(ad);
    free(an);
}

/* ------------------------------------------------------------------------ */
/* Self-Saliency Score, chunk-wise (Algorithm 1, "Compute Self-Saliency      */
/* Score"): s_in, s_prev, masks M_down / M_up / M_diag.                      */
/* ------------------------------------------------------------------------ */

void still_oracle_score_chunkwise(const double *q, const double *k, int64_t N, int d, int C,
                                  double sm_scale, double eps, double *score) {
    int64_t T = (N + C - 1) / C;
    double *s_in = (double *)malloc(sizeof(double) * (size_t)C * C);
    double *s_prev = (double *)malloc(sizeof(double) * (size_t)C * C);
    double *ad = (double *)malloc(sizeof(double) * 2 * (size_t)C);
    double *an = (double *)malloc(sizeof(double) * 2 * (size_t)C);
    int *isdiag = (int *)malloc(sizeof(int) * 2 * (size_t)C);
    for (int64_t c = 0; c < T; ++c) {
        int64_t base = c * C;
        int n_c = (int)((N - base < C) ? (N - base) : C);
        for (int r = 0; r < n_c; ++r)
            for (int s = 0; s < n_c; ++s)
                s_in[r * C + s] = sm_scale * dotd(q + (base + r) * d, k + (base + s) * d, d);
        if (c > 0)
            for (int r = 0; r < n_c; ++r)
                for (int s = 0; s < C; ++s)
                    s_prev[r * C + s] = sm_scale * dotd(q + (base + r) * d, k + (base - C + s) * d, d);
        for (int r = 0; r < n_c; ++r) {
            /* a_diag over [s_in . M_down, s_prev . M_up]; a_nodiag over
               [s_in . M_diag, s_prev . M_up]; a masked entry is excluded. */
            int nd = 0, nn = 0;
            if (c > 0)
                for (int s = 0; s < C; ++s)
                    if (r < s) { /* M_up */
                        ad[nd] = s_prev[r * C + s];
                        isdiag[nd] = 0;
                        ++nd;
                        an[nn++] = s_prev[r * C + s];
                    }
            for (int s = 0; s < n_c; ++s) {
                if (r >= s) { /* M_down */
                    ad[nd] = s_in[r * C + s];
                    isdiag[nd] = (s == r);
                    ++nd;
                }
                if (r > s) an[nn++] = s_in[r * C + s]; /* M_diag */
            }
            softmax_inplace(ad, nd);
            if (nn > 0) softmax_inplace(an, nn);
            double sc = 0.0;
            int jn = 0;
            for (int j = 0; j < nd; ++j) {
                double b = 0.0;
                if (!isdiag[j]) b = an[jn++];
                sc += ad[j] * log((ad[j] + eps) / (b + eps));
            }
            score[base + r] = sc;
        }
    }
    free(s_in);
    free(s_prev);
    free(ad);
    free(an);
    free(isdiag);
}

/* ------------------------------------------------------------------------ */
/* Top-lambda per chunk (delayed selection, Eq. "delayed_selection";         */
/* Algorithm 1 "Local-Global Consistent Selection").                         */
/* idx is [T, lam] absolute 0-based positions, ascending, padded with -1.    */
/* ------------------------------------------------------------------------ */

typedef struct {
    double key;
    int64_t pos;
} rank_item;

static int rank_cmp(const void *pa, const void *pb) {
    const rank_item *a = (const rank_item *)pa, *b = (const rank_item *)pb;
    if (a->key > b->key) return -1; /* larger score first */
    if (a->key < b->key) return 1;
    return (a->pos < b->pos) ? -1 : (a->pos > b->pos); /* then smaller index */
}

static int pos_cmp(const void *pa, const void *pb) {
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a < b) ? -1 : (a > b);
}

void still_oracle_select(const double *score, int64_t N, int C, int lam, int32_t *idx) {
    int64_t T = (N + C - 1) / C;
    rank_item *it = (rank_item *)malloc(sizeof(rank_item) * (size_t)C);
    for (int64_t c = 0; c < T; ++c) {
        int64_t base = c * C;
        int n_c = (int)((N - base < C) ? (N - base) : C);
        for (int r = 0; r < n_c; ++r) {
            double s = score[base + r];
            it[r].key = isnan(s) ? -INFINITY : s;
            it[r].pos = base + r;
        }
        qsort(it, (size_t)n_c, sizeof(rank_item), rank_cmp);
        int n_sel = (lam < n_c) ? lam : n_c;
        int32_t *out = idx + c * lam;
        for (int j = 0; j < lam; ++j) out[j] = (j < n_sel) ? (int32_t)it[j].pos : -1;
        qsort(out, (size_t)n_sel, sizeof(int32_t), pos_cmp);
    }
    free(it);
}

/* ------------------------------------------------------------------------ */
/* Norm-Preserved Feature Map (Eq. "feature_map").                           */
/* x [n,d], W [d,df], b [df] or NULL -> phi [n, 2 df].                        */
/* ------------------------------------------------------------------------ */

void still_oracle_npmap(const double *x, int64_t n, int d, int df, const double *W, const double *b,
                        double *phi) {
    double *u = (double *)malloc(sizeof(double) * (size_t)df);
    for (int64_t r = 0; r < n; ++r) {
        const double *xr = x + r * d;
        double nx = 0.0, nf = 0.0;
        for (int i = 0; i < d; ++i) nx += xr[i] * xr[i];
        nx = sqrt(nx);
        for (int j = 0; j < df; ++j) {
            double f = b ? b[j] : 0.0;
            for (int i = 0; i < d; ++i) f += xr[i] * W[(size_t)i * df + j];
            u[j] = f;
            nf += f * f;
        }
        nf = sqrt(nf);
        if (nf < 1e-12) nf = 1e-12;
        double *pr = phi + r * 2 * df;
        for (int j = 0; j < df; ++j) {
            u[j] = u[j] / nf * nx; /* direction of f(x), norm of x */
            pr[j] = u[j];
            pr[df + j] = -u[j];
        }
        softmax_inplace(pr, df);
        softmax_inplace(pr + df, df);
    }
    free(u);
}

/* ------------------------------------------------------------------------ */
/* Merge with a common shift: y = (N_SA + N_LA) / (D_SA + D_LA) where the SA */
/* logits l_i are given; everything is multiplied by exp(-m), m = max(l, 0). */
/* parts (optional) receives [N_SA(d), D_SA, N_LA(d), D_LA, m] un-shifted by */
/* exp(-m) i.e. as "shifted" values plus the shift m so a test can undo it.  */
/* ------------------------------------------------------------------------ */

typedef struct {
    int d;
    double m;      /* running shift */
    double *num;   /* [d] shifted numerator of SA */
    double den;    /* shifted denominator of SA */
} sa_acc;

static void sa_add(sa_acc *a, double logit, const double *v) {
    if (logit > a->m) {
        double r = exp(a->m - logit);
        for (int i = 0; i < a->d; ++i) a->num[i] *= r;
        a->den *= r;
        a->m = logit;
    }
    double e = exp(logit - a->m);
    for (int i = 0; i < a->d; ++i) a->num[i] += e * v[i];
    a->den += e;
}

static void merge_row(const sa_acc *a, const double *phi_q, const double *S, const double *z,
                      const double *g, int d, int dp, double *y, double *parts) {
    /* N_LA = (phi_q S) . g ; D_LA = phi_q . z  (definitions below the merge equation) */
    double e0 = exp(-a->m); /* a->m >= 0 since it starts at 0 */
    double dla = 0.0;
    for (int f = 0; f < dp; ++f) dla += phi_q[f] * z[f];
    for (int i = 0; i < d; ++i) {
        double nla = 0.0;
        for (int f = 0; f < dp; ++f) nla += phi_q[f] * S[(size_t)f * d + i];
        if (g) nla *= g[i];
        y[i] = (a->num[i] + e0 * nla) / (a->den + e0 * dla);
        if (parts) {
            parts[i] = a->num[i];
            parts[d + 1 + i] = nla;
        }
    }
    if (parts) {
        parts[d] = a->den;
        parts[2 * d + 1] = dla;
        parts[2 * d + 2] = a->m;
    }
}

/* ------------------------------------------------------------------------ */
/* Algorithm 1: Chunk-Wise Parallel Form, one head.                          */
/*                                                                           */
/* forced_idx : NULL, or a [T, lam] selection to use instead of Top(S, lam). */
/* rows       : NULL (all N rows), or n_rows ascending row positions; the    */
/*              score / selection / state steps always cover the sequence.   */
/* y          : [n_out, d]; score_out [N] and idx_out [T, lam] optional;     */
/* parts      : optional [n_out, 2d+3] = N_SA(d), D_SA, N_LA(d), D_LA, m     */
/*              with N_SA, D_SA holding the factor exp(-m).                  */
/* The cumulative sums s, z of the algorithm are kept as running sums with   */
/* the two-chunk lag, which is the same arithmetic as Cumsum + shift.        */
/* ------------------------------------------------------------------------ */

void still_oracle_chunkwise(const double *q, const double *k, const double *v, const double *g,
                            int64_t N, int d, int df, int C, int lam, double sm_scale, double eps,
                            int64_t max_salient, const double *Wq, const double *bq, const double *Wk, const double *bk,
                            const int32_t *forced_idx, const int64_t *rows, int64_t n_rows,
                            double *y, double *score_out, int32_t *idx_out, double *parts) {
    int64_t T = (N + C - 1) / C;
    int dp = 2 * df;
    double *score = (double *)malloc(sizeof(double) * (size_t)N);
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T * (lam > 0 ? lam : 1)));
    still_oracle_score_chunkwise(q, k, N, d, C, sm_scale, eps, score);
    if (forced_idx)
        memcpy(idx, forced_idx, sizeof(int32_t) * (size_t)(T * lam));
    else
        still_oracle_select(score, N, C, lam, idx);
    if (score_out) memcpy(score_out, score, sizeof(double) * (size_t)N);
    if (idx_out) memcpy(idx_out, idx, sizeof(int32_t) * (size_t)(T * lam));

    /* M^SA as a 0/1 vector; M^LA is its complement. */
    char *in_sa = (char *)calloc((size_t)N, 1);
    for (int64_t j = 0; j < T * lam; ++j)
        if (idx[j] >= 0) in_sa[idx[j]] = 1;

    double *S = (double *)calloc((size_t)dp * d, sizeof(double)); /* s_shift[t] = s[t-2] */
    double *z = (double *)calloc((size_t)dp, sizeof(double));
    double *phi = (double *)malloc(sizeof(double) * (size_t)dp);
    double *num = (double *)malloc(sizeof(double) * (size_t)d);
    int64_t out_i = 0, row_cursor = 0;
    /* salient cache of the routed chunks in routing (= position) order; [sal_head, n_sal) is live */
    int64_t *sal = (int64_t *)malloc(sizeof(int64_t) * (size_t)(N + 1));
    int64_t n_sal = 0, sal_head = 0;

    for (int64_t c = 0; c < T; ++c) {
        /* Linear Attention Branch: the state seen by chunk c holds the LA tokens
           of chunks <= c-2; fold chunk c-2 in now. */
        if (c >= 2) {
            int64_t b0 = (c - 2) * C;
            for (int64_t i = b0; i < b0 + C; ++i) {
                if (in_sa[i]) continue;
                still_oracle_npmap(k + i * d, 1, d, df, Wk, bk, phi);
                for (int f = 0; f < dp; ++f) {
                    for (int e = 0; e < d; ++e) S[(size_t)f * d + e] += phi[f] * v[i * d + e];
                    z[f] += phi[f];
                }
            }
            /* the selected tokens of chunk c-2 enter the salient cache; beyond the budget the oldest
               leave it for the LA state */
            for (int j = 0; j < lam; ++j) {
                int32_t p = idx[(c - 2) * lam + j];
                if (p >= 0) sal[n_sal++] = p;
            }
            while (max_salient > 0 && n_sal - sal_head > max_salient) {
                int64_t i = sal[sal_head++];
                still_oracle_npmap(k + i * d, 1, d, df, Wk, bk, phi);
                for (int f = 0; f < dp; ++f) {
                    for (int e = 0; e < d; ++e) S[(size_t)f * d + e] += phi[f] * v[i * d + e];
                    z[f] += phi[f];
                }
            }
        }
        int64_t base = c * C;
        int n_c = (int)((N - base < C) ? (N - base) : C);
        for (int r = 0; r < n_c; ++r) {
            int64_t t = base + r;
            if (rows) {
                if (row_cursor >= n_rows || rows[row_cursor] != t) continue;
                ++row_cursor;
            }
            /* Softmax Attention Branch for row t. */
            sa_acc acc;
            acc.d = d;
            acc.m = 0.0;
            acc.num = num;
            acc.den = 0.0;
            for (int i = 0; i < d; ++i) num[i] = 0.0;
            /* q k_SA^T . M_chunk : selected tokens of chunks 0..c-2 (those still in the cache) */
            for (int64_t j = sal_head; j < n_sal; ++j)
                sa_add(&acc, sm_scale * dotd(q + t * d, k + sal[j] * d, d), v + sal[j] * d);
            /* s_prev : all of chunk c-1 */
            if (c >= 1)
                for (int64_t p = base - C; p < base; ++p)
                    sa_add(&acc, sm_scale * dotd(q + t * d, k + p * d, d), v + p * d);
            /* s_in . M_down : chunk c up to and including t */
            for (int64_t p = base; p <= t; ++p)
                sa_add(&acc, sm_scale * dotd(q + t * d, k + p * d, d), v + p * d);
            /* phi_q(q) s_shift . g and phi_q(q) z_shift, merged under one denominator */
            still_oracle_npmap(q + t * d, 1, d, df, Wq, bq, phi);
            merge_row(&acc, phi, S, z, g ? g + t * d : NULL, d, dp, y + out_i * d,
                      parts ? parts + out_i * (2 * d + 3) : NULL);
            ++out_i;
        }
    }
    free(score);
    free(idx);
    free(in_sa);
    free(S);
    free(z);
    free(phi);
    free(num);
    free(sal);
}

/* ------------------------------------------------------------------------ */
/* Recurrent Form (Sec. 3.3), one head, one token per step.                  */
/*                                                                           */
/* The paper writes t = (a+1) T + b with 1-based t, chunk size T, b in 1..T. */
/* Here C is the chunk size.  The containers are explicit:                   */
/*   sal    : positions of the salient pairs appended so far (h minus the    */
/*            local region),                                                 */
/*   s, z   : KV state and normaliser,                                       */
/*   score  : Score of every token seen so far (kept so that chunk a can be  */
/*            ranked when it leaves the local region).                       */
/* forced_idx, if given, replaces Top_lambda for the routed chunk.           */
/* ------------------------------------------------------------------------ */

void still_oracle_recurrent(const double *q, const double *k, const double *v, const double *g,
                            int64_t N, int d, int df, int C, int lam, double sm_scale, double eps,
                            int64_t max_salient, const double *Wq, const double *bq, const double *Wk, const double *bk,
                            const int32_t *forced_idx, double *y, double *score_out,
                            int32_t *idx_out) {
    int dp = 2 * df;
    int64_t Tn = (N + C - 1) / C;
    double *score = (double *)malloc(sizeof(double) * (size_t)N);
    int64_t *sal = (int64_t *)malloc(sizeof(int64_t) * (size_t)(N + 1));
    int64_t n_sal = 0, sal_head = 0; /* [sal_head, n_sal) is the live salient cache */
    double *s = (double *)calloc((size_t)dp * d, sizeof(double));
    double *z = (double *)calloc((size_t)dp, sizeof(double));
    double *phi = (double *)malloc(sizeof(double) * (size_t)dp);
    double *num = (double *)malloc(sizeof(double) * (size_t)d);
    double *win = (double *)malloc(sizeof(double) * (size_t)C);
    double *win2 = (double *)malloc(sizeof(double) * (size_t)C);
    char *taken = (char *)malloc((size_t)C);
    if (idx_out)
        for (int64_t j = 0; j < Tn * lam; ++j) idx_out[j] = -1;

    for (int64_t t1 = 1; t1 <= N; ++t1) { /* 1-based step index as in the paper */
        const double *qt = q + (t1 - 1) * d;
        /* Score of the current token over W_t = {max(1,t-w+1) .. t}, w = C. */
        {
            int64_t lo = t1 - C + 1;
            if (lo < 1) lo = 1;
            int n = (int)(t1 - lo + 1);
            for (int j = 0; j < n; ++j) win[j] = sm_scale * dotd(qt, k + (lo - 1 + j) * d, d);
            for (int j = 0; j < n - 1; ++j) win2[j] = win[j];
            softmax_inplace(win, n);
            if (n > 1) softmax_inplace(win2, n - 1);
            double sc = 0.0;
            for (int j = 0; j < n; ++j) {
                double b = (j == n - 1) ? 0.0 : win2[j];
                sc += win[j] * log((win[j] + eps) / (b + eps));
            }
            score[t1 - 1] = sc;
        }
        /* t = (a+1) C + b,  b in 1..C  =>  a = ceil(t / C) - 2. */
        int64_t a = (t1 + C - 1) / C - 2;
        int64_t b = t1 - (a + 1) * C;
        if (a >= 1 && b == 1) {
            /* Route chunk a (tokens (a-1)C+1 .. aC): Top_lambda -> salient cache,
               the rest -> (s, z). */
            int64_t first = (a - 1) * C + 1; /* 1-based */
            memset(taken, 0, (size_t)C);
            if (forced_idx) {
                for (int j = 0; j < lam; ++j) {
                    int32_t p = forced_idx[(a - 1) * lam + j];
                    if (p >= 0) taken[p - (first - 1)] = 1;
                }
            } else {
                for (int pick = 0; pick < lam && pick < C; ++pick) {
                    int best = -1;
                    double bs = 0.0;
                    for (int i = 0; i < C; ++i) {
                        if (taken[i]) continue;
                        double si = score[first - 1 + i];
                        if (isnan(si)) si = -INFINITY;
                        if (best < 0 || si > bs) { /* strict: ties keep the smaller index */
                            best = i;
                            bs = si;
                        }
                    }
                    if (best >= 0) taken[best] = 1;
                }
            }
            int w = 0;
            for (int i = 0; i < C; ++i) {
                int64_t p0 = first - 1 + i; /* 0-based position */
                if (taken[i]) {
                    sal[n_sal++] = p0;
                    if (idx_out) idx_out[(a - 1) * lam + w++] = (int32_t)p0;
                } else {
                    still_oracle_npmap(k + p0 * d, 1, d, df, Wk, bk, phi);
                    for (int f = 0; f < dp; ++f) {
                        for (int e = 0; e < d; ++e) s[(size_t)f * d + e] += phi[f] * v[p0 * d + e];
                        z[f] += phi[f];
                    }
                }
            }
            /* budget: the oldest salient pairs leave the cache for the state */
            while (max_salient > 0 && n_sal - sal_head > max_salient) {
                int64_t p0 = sal[sal_head++];
                still_oracle_npmap(k + p0 * d, 1, d, df, Wk, bk, phi);
                for (int f = 0; f < dp; ++f) {
                    for (int e = 0; e < d; ++e) s[(size_t)f * d + e] += phi[f] * v[p0 * d + e];
                    z[f] += phi[f];
                }
            }
        }
        /* h_t = local region { max(0, aC) < i <= t } united with the salient pairs. */
        sa_acc acc;
        acc.d = d;
        acc.m = 0.0;
        acc.num = num;
        acc.den = 0.0;
        for (int i = 0; i < d; ++i) num[i] = 0.0;
        for (int64_t j = sal_head; j < n_sal; ++j)
            sa_add(&acc, sm_scale * dotd(qt, k + sal[j] * d, d), v + sal[j] * d);
        int64_t lo = (a > 0 ? a * C : 0); /* exclusive, 1-based */
        for (int64_t i = lo + 1; i <= t1; ++i)
            sa_add(&acc, sm_scale * dotd(qt, k + (i - 1) * d, d), v + (i - 1) * d);
        still_oracle_npmap(qt, 1, d, df, Wq, bq, phi);
        merge_row(&acc, phi, s, z, g ? g + (t1 - 1) * d : NULL, d, dp, y + (t1 - 1) * d, NULL);
    }
    /* Chunks that never left the local region are not routed by the recurrence;
       report their would-be selection so that the index table is complete. */
    if (idx_out) {
        int32_t *full = (int32_t *)malloc(sizeof(int32_t) * (size_t)(Tn * (lam > 0 ? lam : 1)));
        still_oracle_select(score, N, C, lam, full);
        int64_t routed = (N >= 1) ? ((N + C - 1) / C - 2) : 0; /* chunks 1..a routed */
        if (routed < 0) routed = 0;
        for (int64_t c = routed; c < Tn; ++c)
            for (int j = 0; j < lam; ++j)
                idx_out[c * lam + j] = forced_idx ? forced_idx[c * lam + j] : full[c * lam + j];
        free(full);
    }
    if (score_out) memcpy(score_out, score, sizeof(double) * (size_t)N);
    free(score);
    free(sal);
    free(s);
    free(z);
    free(phi);
    free(num);
    free(win);
    free(win2);
    free(taken);
}

/* ------------------------------------------------------------------------ */
/* Whole layer: B x H independent heads, query head h uses KV head           */
/* h / (H / Hkv).  Runs the chunk-wise form per head, heads in parallel.     */
/* Layouts: Q,G,Y [B,H,N,d]; K,V [B,Hkv,N,d]; Wq [H,d,df]; bq [H,df];        */
/* Wk [Hkv,d,df]; bk [Hkv,df]; score [B,H,N]; idx [B,H,T,lam];               */
/* rows (optional) shared by all heads; y is then [B,H,n_rows,d].            */
/* Returns the number of threads used.                                       */
/* ------------------------------------------------------------------------ */

int still_oracle_layer(const double *Q, const double *K, const double *V, const double *G, int B,
                       int H, int Hkv, int64_t N, int d, int df, int C, int lam, double sm_scale,
                       double eps, int64_t max_salient, const double *Wq, const double *bq, const double *Wk,
                       const double *bk, const int32_t *forced_idx, const int64_t *rows,
                       int64_t n_rows, double *Y, double *score_out, int32_t *idx_out) {
    int64_t T = (N + C - 1) / C;
    int64_t n_out = rows ? n_rows : N;
    int rep = H / Hkv;
    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int bh = 0; bh < B * H; ++bh) {
        int b = bh / H, h = bh % H, kv = h / rep;
        const double *q = Q + (size_t)bh * N * d;
        const double *k = K + ((size_t)b * Hkv + kv) * N * d;
        const double *v = V + ((size_t)b * Hkv + kv) * N * d;
        still_oracle_chunkwise(q, k, v, G ? G + (size_t)bh * N * d : NULL, N, d, df, C, lam,
                               sm_scale, eps, max_salient, Wq + (size_t)h * d * df, bq ? bq + (size_t)h * df : NULL,
                               Wk + (size_t)kv * d * df, bk ? bk + (size_t)kv * df : NULL,
                               forced_idx ? forced_idx + (size_t)bh * T * lam : NULL, rows, n_rows,
                               Y + (size_t)bh * n_out * d,
                               score_out ? score_out + (size_t)bh * N : NULL,
                               idx_out ? idx_out + (size_t)bh * T * lam : NULL, NULL);
    }
    return threads;
}
