/*
 * CPU oracle for the PaFu-KV inference hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64 restatement of what the path computes, written from the
 * paper's definitions.  It shares no code with the CUDA library and must never
 * be called from the product path; only tests, the smoke check and the
 * benchmark's CPU-baseline leg use it.
 *
 *   score    S-MLP salience head: two linear layers with an activation in
 *            between, mean over the output units (Sec. 3.3; Appendix A "S-MLP").
 *   select   retain the top-k salient tokens (Sec. 3.4 inference paragraph;
 *            Algorithm 2 "Top-k") with the frame sink (Sec. 4.1) and an always
 *            kept recent suffix.
 *   compact  KV <- Select(KV; ids), SL <- Select(SL; ids) (Algorithm 2).
 *   attn     P = softmax(Q K^T / sqrt(D)) (Sec. 3.2), O = P V over the retained
 *            cache followed by the chunk's own tokens (Eq. 2 / Eq. 7).
 *   sse      teacher-side salience target of Eq. 4 and Eq. 5 (and the same in Algorithm 3's
 *            order: mean over heads before the maximum over queries).
 *
 * All token tensors are bf16 bit patterns (uint16), token-major
 * [tokens, n_heads, d_head]; they are widened exactly to fp64 and every sum is
 * taken in fp64 in index order.  OpenMP is used only across independent rows.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int pafu_oracle_abi_version(void) { return 1; }

/* ---------------------------------------------------------------- score ---
 * act: 0 = GELU, exact form x * Phi(x) = x/2 * (1 + erf(x / sqrt 2)); 1 = SiLU x * sigma(x).
 * final: 0 = none, 1 = logistic sigmoid of the mean.
 * w1 [d_hidden, d_in], w2 [d_out, d_hidden] row-major; b1, b2 may be NULL.
 */
static double act_f64(double a, int act) {
    if (act == 0) return 0.5 * a * (1.0 + erf(a / sqrt(2.0)));
    return a / (1.0 + exp(-a));
}

void pafu_oracle_score(const uint16_t *X, int64_t n_tokens, int64_t ldx,
                       int32_t d_in, int32_t d_hidden, int32_t d_out,
                       int32_t act, int32_t final,
                       const uint16_t *w1, const uint16_t *b1,
                       const uint16_t *w2, const uint16_t *b2,
                       float *scores) {
    double *W1 = (double *)malloc(sizeof(double) * (size_t)d_hidden * d_in);
    double *W2 = (double *)malloc(sizeof(double) * (size_t)d_out * d_hidden);
    for (int64_t i = 0; i < (int64_t)d_hidden * d_in; ++i) W1[i] = bf16_to_f64(w1[i]);
    for (int64_t i = 0; i < (int64_t)d_out * d_hidden; ++i) W2[i] = bf16_to_f64(w2[i]);
#pragma omp parallel
    {
        double *x = (double *)malloc(sizeof(double) * d_in);
        double *h = (double *)malloc(sizeof(double) * d_hidden);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < n_tokens; ++t) {
            for (int32_t i = 0; i < d_in; ++i) x[i] = bf16_to_f64(X[t * ldx + i]);
            for (int32_t j = 0; j < d_hidden; ++j) {
                double a = b1 ? bf16_to_f64(b1[j]) : 0.0;
                const double *wr = W1 + (size_t)j * d_in;
                for (int32_t i = 0; i < d_in; ++i) a += wr[i] * x[i];
                h[j] = act_f64(a, act);
            }
            double mean = 0.0;
            for (int32_t o = 0; o < d_out; ++o) {
                double y = b2 ? bf16_to_f64(b2[o]) : 0.0;
                const double *wr = W2 + (size_t)o * d_hidden;
                for (int32_t j = 0; j < d_hidden; ++j) y += wr[j] * h[j];
                mean += y;
            }
            mean /= (double)d_out;
            if (final == 1) mean = 1.0 / (1.0 + exp(-mean));
            scores[t] = (float)mean;
        }
        free(x);
        free(h);
    }
    free(W1);
    free(W2);
}

/* --------------------------------------------------------------- select ---
 * Kept set = [0, n_sink') U top-k of scores[n_sink' : T - n_recent') U [T - n_recent', T),
 * written in ascending token order.  T <= budget keeps everything.  Otherwise the recent
 * window is honoured first, then the sink, then k = budget - n_sink' - n_recent'.
 * Ranking: higher score first; equal scores (-0 == +0) -> lower index first; NaN ranks
 * below every number including -inf.  Returns the number of indices written, or -1 on
 * negative arguments.
 */
typedef struct { float s; int32_t i; } cand_t;

static int cand_before(const cand_t *a, const cand_t *b) {
    /* 1 if a ranks strictly before b */
    int an = isnan(a->s), bn = isnan(b->s);
    if (an || bn) {
        if (an && bn) return a->i < b->i;
        return bn; /* a number ranks before NaN */
    }
    if (a->s > b->s) return 1;
    if (a->s < b->s) return 0;
    return a->i < b->i;
}

static int cand_cmp(const void *pa, const void *pb) {
    const cand_t *a = (const cand_t *)pa, *b = (const cand_t *)pb;
    if (cand_before(a, b)) return -1;
    if (cand_before(b, a)) return 1;
    return 0;
}

int64_t pafu_oracle_select(const float *scores, int64_t T, int64_t n_sink, int64_t n_recent,
                           int64_t budget, int32_t *idx) {
    if (T < 0 || n_sink < 0 || n_recent < 0 || budget < 0) return -1;
    if (T <= budget) {
        for (int64_t t = 0; t < T; ++t) idx[t] = (int32_t)t;
        return T;
    }
    int64_t nr = n_recent < budget ? n_recent : budget;
    int64_t ns = n_sink < budget - nr ? n_sink : budget - nr;
    int64_t k = budget - ns - nr;
    int64_t M = T - ns - nr;
    cand_t *c = (cand_t *)malloc(sizeof(cand_t) * (size_t)(M > 0 ? M : 1));
    for (int64_t j = 0; j < M; ++j) { c[j].s = scores[ns + j]; c[j].i = (int32_t)(ns + j); }
    /* the comparison is a strict total order (index breaks every tie), so any full sort
       gives the one stable order */
    qsort(c, (size_t)M, sizeof(cand_t), cand_cmp);
    uint8_t *keep = (uint8_t *)calloc((size_t)T, 1);
    for (int64_t t = 0; t < ns; ++t) keep[t] = 1;
    for (int64_t j = 0; j < k; ++j) keep[c[j].i] = 1;
    for (int64_t t = T - nr; t < T; ++t) keep[t] = 1;
    int64_t n = 0;
    for (int64_t t = 0; t < T; ++t) if (keep[t]) idx[n++] = (int32_t)t;
    free(keep);
    free(c);
    return n;
}

/* -------------------------------------------------------------- compact ---
 * out[i, :] = in[idx[i], :] as raw element copies (row_bytes bytes per row).
 */
void pafu_oracle_gather_rows(const uint8_t *in, const int32_t *idx, int64_t n_idx,
                             int64_t row_bytes, uint8_t *out) {
    for (int64_t i = 0; i < n_idx; ++i)
        memcpy(out + i * row_bytes, in + (int64_t)idx[i] * row_bytes, (size_t)row_bytes);
}

/* ------------------------------------------------------------ attention ---
 * One stream.  For head n and query row r (from `rows`, or all rows when rows == NULL):
 *   z_j = (q . k_j) * scale over the B retained keys then the Lq chunk keys,
 *   m = max_j z_j, p_j = exp(z_j - m), o = sum_j p_j v_j / sum_j p_j, lse = m + log sum_j p_j.
 * O is [n_rows, N, D] fp64, LSE (nullable) is [N, n_rows] fp64.  Either key segment may be
 * empty; with no keys at all the output row is 0 and lse = -inf.
 */
void pafu_oracle_attn(const uint16_t *Q, int64_t Lq,
                      const uint16_t *Kc, const uint16_t *Vc, int64_t B,
                      const uint16_t *Kq, const uint16_t *Vq, int64_t Lkq,
                      int32_t N, int32_t D, double scale,
                      const int64_t *rows, int64_t n_rows,
                      double *O, double *LSE) {
    if (!rows) n_rows = Lq;
    const int64_t Lk = B + Lkq;
    const int64_t dm = (int64_t)N * D;
#pragma omp parallel
    {
        double *z = (double *)malloc(sizeof(double) * (size_t)(Lk > 0 ? Lk : 1));
        double *q = (double *)malloc(sizeof(double) * D);
#pragma omp for collapse(2) schedule(dynamic, 4)
        for (int64_t ri = 0; ri < n_rows; ++ri) {
            for (int32_t n = 0; n < N; ++n) {
                const int64_t r = rows ? rows[ri] : ri;
                double *o = O + (ri * N + n) * D;
                for (int32_t d = 0; d < D; ++d) { q[d] = bf16_to_f64(Q[r * dm + n * D + d]); o[d] = 0.0; }
                double m = -INFINITY;
                for (int64_t j = 0; j < Lk; ++j) {
                    const uint16_t *k = (j < B) ? Kc + j * dm + n * D : Kq + (j - B) * dm + n * D;
                    double acc = 0.0;
                    for (int32_t d = 0; d < D; ++d) acc += q[d] * bf16_to_f64(k[d]);
                    z[j] = acc * scale;
                    if (z[j] > m) m = z[j];
                }
                double l = 0.0;
                for (int64_t j = 0; j < Lk; ++j) {
                    const uint16_t *v = (j < B) ? Vc + j * dm + n * D : Vq + (j - B) * dm + n * D;
                    double p = exp(z[j] - m);
                    l += p;
                    for (int32_t d = 0; d < D; ++d) o[d] += p * bf16_to_f64(v[d]);
                }
                if (Lk > 0) for (int32_t d = 0; d < D; ++d) o[d] /= l;
                if (LSE) LSE[(int64_t)n * n_rows + ri] = (Lk > 0) ? m + log(l) : -INFINITY;
            }
        }
        free(z);
        free(q);
    }
}

/* ------------------------------------------------------------------ sse ---
 * Teacher salience target (Eq. 4, Eq. 5).  Q, K are [L, N, D] bf16 bits, full bidirectional
 * attention P = softmax(Q K^T * scale) per head.  With block length LB, query i lies in block
 * b(i) = floor(i / LB) spanning keys [l(i), h(i)).  For key j:
 *   low_j  = mean_n max_{i : j <  l(i)} P[n,i,j]     (queries in later blocks)
 *   diag_j = mean_n max_{i : l(i) <= j < h(i)} P     (queries in the same block)
 *   up_j   = mean_n max_{i : j >= h(i)} P            (queries in earlier blocks)
 * An empty index set contributes 0.  Eq. 5: the first block averages (diag + low) / 2,
 * the last block (diag + up) / 2, the rest (up + diag + low) / 3.  Requires L >= 2 LB for
 * the three ranges of Eq. 5 to be disjoint; with L < 2 LB the first matching case is used.
 * Outputs: s [L] fp64 and, when comp != NULL, comp [3, L] = low, diag, up.
 */
void pafu_oracle_sse(const uint16_t *Q, const uint16_t *K, int64_t L, int32_t N, int32_t D,
                     int64_t LB, double scale, double *s, double *comp) {
    double *low = (double *)calloc((size_t)L, sizeof(double));
    double *diag = (double *)calloc((size_t)L, sizeof(double));
    double *up = (double *)calloc((size_t)L, sizeof(double));
    const int64_t dm = (int64_t)N * D;
    for (int32_t n = 0; n < N; ++n) {
        double *mlow = (double *)calloc((size_t)L, sizeof(double));
        double *mdiag = (double *)calloc((size_t)L, sizeof(double));
        double *mup = (double *)calloc((size_t)L, sizeof(double));
        double *P = (double *)malloc(sizeof(double) * (size_t)L * (size_t)L);
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < L; ++i) {
            double *p = P + i * L;
            double m = -INFINITY;
            for (int64_t j = 0; j < L; ++j) {
                double acc = 0.0;
                for (int32_t d = 0; d < D; ++d)
                    acc += bf16_to_f64(Q[i * dm + n * D + d]) * bf16_to_f64(K[j * dm + n * D + d]);
                p[j] = acc * scale;
                if (p[j] > m) m = p[j];
            }
            double l = 0.0;
            for (int64_t j = 0; j < L; ++j) { p[j] = exp(p[j] - m); l += p[j]; }
            for (int64_t j = 0; j < L; ++j) p[j] /= l;
        }
        for (int64_t i = 0; i < L; ++i) {
            const int64_t lo = (i / LB) * LB, hi = lo + LB;
            const double *p = P + i * L;
            for (int64_t j = 0; j < L; ++j) {
                double *dst = (j < lo) ? mlow : (j < hi) ? mdiag : mup;
                if (p[j] > dst[j]) dst[j] = p[j];
            }
        }
        for (int64_t j = 0; j < L; ++j) { low[j] += mlow[j]; diag[j] += mdiag[j]; up[j] += mup[j]; }
        free(P); free(mlow); free(mdiag); free(mup);
    }
    for (int64_t j = 0; j < L; ++j) {
        low[j] /= N; diag[j] /= N; up[j] /= N;
        if (j < LB) s[j] = (diag[j] + low[j]) / 2.0;
        else if (j < L - LB) s[j] = (up[j] + diag[j] + low[j]) / 3.0;
        else s[j] = (diag[j] + up[j]) / 2.0;
        if (comp) { comp[j] = low[j]; comp[L + j] = diag[j]; comp[2 * L + j] = up[j]; }
    }
    free(low); free(diag); free(up);
}

/* --------------------------------------------- sse in Algorithm 3's order of operations ---
 * Algorithm 3 takes the mean over heads BEFORE the maximum over queries (Eq. 4 as printed takes
 * the maximum per head first and then the mean):
 *   a[i,j]  = (1/N) sum_n P[n,i,j]
 *   low_j   = max_{i : j <  l(i)} a[i,j],  diag_j = max_{i : l(i) <= j < h(i)} a[i,j],
 *   up_j    = max_{i : j >= h(i)} a[i,j]   (an empty index set gives 0), then Eq. 5 as above.
 * One query row at a time: the row's softmax per head is added into a buffer of L means.
 */
void pafu_oracle_sse_meanfirst(const uint16_t *Q, const uint16_t *K, int64_t L, int32_t N, int32_t D,
                               int64_t LB, double scale, double *s, double *comp) {
    double *low = (double *)calloc((size_t)L, sizeof(double));
    double *diag = (double *)calloc((size_t)L, sizeof(double));
    double *up = (double *)calloc((size_t)L, sizeof(double));
    double *a = (double *)malloc(sizeof(double) * (size_t)L);
    double *p = (double *)malloc(sizeof(double) * (size_t)L);
    const int64_t dm = (int64_t)N * D;
    for (int64_t i = 0; i < L; ++i) {
        for (int64_t j = 0; j < L; ++j) a[j] = 0.0;
        for (int32_t n = 0; n < N; ++n) {
            double m = -INFINITY;
            for (int64_t j = 0; j < L; ++j) {
                double acc = 0.0;
                for (int32_t d = 0; d < D; ++d)
                    acc += bf16_to_f64(Q[i * dm + n * D + d]) * bf16_to_f64(K[j * dm + n * D + d]);
                p[j] = acc * scale;
                if (p[j] > m) m = p[j];
            }
            double l = 0.0;
            for (int64_t j = 0; j < L; ++j) { p[j] = exp(p[j] - m); l += p[j]; }
            for (int64_t j = 0; j < L; ++j) a[j] += p[j] / l;
        }
        const int64_t lo = (i / LB) * LB, hi = lo + LB;
        for (int64_t j = 0; j < L; ++j) {
            const double v = a[j] / N;
            double *dst = (j < lo) ? low : (j < hi) ? diag : up;
            if (v > dst[j]) dst[j] = v;
        }
    }
    for (int64_t j = 0; j < L; ++j) {
        if (j < LB) s[j] = (diag[j] + low[j]) / 2.0;
        else if (j < L - LB) s[j] = (up[j] + diag[j] + low[j]) / 3.0;
        else s[j] = (diag[j] + up[j]) / 2.0;
        if (comp) { comp[j] = low[j]; comp[L + j] = diag[j]; comp[2 * L + j] = up[j]; }
    }
    free(low); free(diag); free(up); free(a); free(p);
}

/* ------------------------------------------------------------- sse, sampled columns ---
 * The same definition (Eq. 4, Eq. 5) evaluated for a list of key positions only, for sequences
 * too long to hold P: per head, every row's log-sum-exp is computed first (one streaming pass
 * over all L x L logits), then for each listed key j the column P[i, j] = exp(z_ij - lse_i) is
 * walked over all queries i and split by the query's block into the three maxima.
 * Outputs: s [n_cols], comp [3, n_cols] = low, diag, up (comp may be NULL).
 */
void pafu_oracle_sse_cols(const uint16_t *Q, const uint16_t *K, int64_t L, int32_t N, int32_t D,
                          int64_t LB, double scale, const int64_t *cols, int64_t n_cols,
                          double *s, double *comp) {
    const int64_t dm = (int64_t)N * D;
    double *low = (double *)calloc((size_t)n_cols, sizeof(double));
    double *diag = (double *)calloc((size_t)n_cols, sizeof(double));
    double *up = (double *)calloc((size_t)n_cols, sizeof(double));
    double *q = (double *)malloc(sizeof(double) * (size_t)L * D);
    double *k = (double *)malloc(sizeof(double) * (size_t)L * D);
    double *lse = (double *)malloc(sizeof(double) * (size_t)L);
    for (int32_t n = 0; n < N; ++n) {
        for (int64_t i = 0; i < L; ++i)
            for (int32_t d = 0; d < D; ++d) {
                q[i * D + d] = bf16_to_f64(Q[i * dm + n * D + d]);
                k[i * D + d] = bf16_to_f64(K[i * dm + n * D + d]);
            }
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < L; ++i) {
            double *z = (double *)malloc(sizeof(double) * (size_t)L);
            double m = -INFINITY;
            for (int64_t j = 0; j < L; ++j) {
                double acc = 0.0;
                for (int32_t d = 0; d < D; ++d) acc += q[i * D + d] * k[j * D + d];
                z[j] = acc * scale;
                if (z[j] > m) m = z[j];
            }
            double l = 0.0;
            for (int64_t j = 0; j < L; ++j) l += exp(z[j] - m);
            lse[i] = m + log(l);
            free(z);
        }
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < n_cols; ++c) {
            const int64_t j = cols[c];
            double mlow = 0.0, mdiag = 0.0, mup = 0.0;
            for (int64_t i = 0; i < L; ++i) {
                double acc = 0.0;
                for (int32_t d = 0; d < D; ++d) acc += q[i * D + d] * k[j * D + d];
                const double p = exp(acc * scale - lse[i]);
                const int64_t lo = (i / LB) * LB, hi = lo + LB;
                if (j < lo) { if (p > mlow) mlow = p; }
                else if (j < hi) { if (p > mdiag) mdiag = p; }
                else { if (p > mup) mup = p; }
            }
            low[c] += mlow; diag[c] += mdiag; up[c] += mup;
        }
    }
    for (int64_t c = 0; c < n_cols; ++c) {
        const int64_t j = cols[c];
        low[c] /= N; diag[c] /= N; up[c] /= N;
        if (j < LB) s[c] = (diag[c] + low[c]) / 2.0;
        else if (j < L - LB) s[c] = (up[c] + diag[c] + low[c]) / 3.0;
        else s[c] = (diag[c] + up[c]) / 2.0;
        if (comp) { comp[c] = low[c]; comp[n_cols + c] = diag[c]; comp[2 * n_cols + c] = up[c]; }
    }
    free(low); free(diag); free(up); free(q); free(k); free(lse);
}

/* ------------------------------------------------------- global max pooling ---
 * The "Max" alternative of the paper's ablation on the salience score (Sec. 4.3, Table 3):
 * g_j = mean over heads of max over ALL queries i of P[n, i, j], P = softmax(Q K^T * scale);
 * and, when avg != NULL, the "Avg" alternative avg_j = mean over heads and queries of P[n, i, j].
 */
void pafu_oracle_sse_gmax(const uint16_t *Q, const uint16_t *K, int64_t L, int32_t N, int32_t D,
                          double scale, double *g, double *avg) {
    const int64_t dm = (int64_t)N * D;
    for (int64_t j = 0; j < L; ++j) { g[j] = 0.0; if (avg) avg[j] = 0.0; }
    double *P = (double *)malloc(sizeof(double) * (size_t)L * (size_t)L);
    for (int32_t n = 0; n < N; ++n) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < L; ++i) {
            double *p = P + i * L;
            double m = -INFINITY, l = 0.0;
            for (int64_t j = 0; j < L; ++j) {
                double acc = 0.0;
                for (int32_t d = 0; d < D; ++d)
                    acc += bf16_to_f64(Q[i * dm + n * D + d]) * bf16_to_f64(K[j * dm + n * D + d]);
                p[j] = acc * scale;
                if (p[j] > m) m = p[j];
            }
            for (int64_t j = 0; j < L; ++j) { p[j] = exp(p[j] - m); l += p[j]; }
            for (int64_t j = 0; j < L; ++j) p[j] /= l;
        }
        for (int64_t j = 0; j < L; ++j) {
            double mx = 0.0;
            for (int64_t i = 0; i < L; ++i) if (P[i * L + j] > mx) mx = P[i * L + j];
            g[j] += mx / N;
            if (avg) {      /* the "Avg" alternative: mean over all queries */
                double sm = 0.0;
                for (int64_t i = 0; i < L; ++i) sm += P[i * L + j];
                avg[j] += sm / L / N;
            }
        }
    }
    free(P);
}
