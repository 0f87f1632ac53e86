/*
 * fp64 CPU oracle for packed variable-length multi-head attention, forward and backward.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call this file; it exists so
 * that the tests, the smoke check and the CPU-baseline leg of the benchmark have a slow,
 * plain answer to compare the CUDA kernels with.  It shares no source with the kernels.
 *
 * What it computes.  The paper names the operation only as the attention library that its
 * training runs enable (Section 4.1, "Experiment Setup") and states that this operation
 * dominates run time (Section 4.2); it gives no formula, so the definition below is the
 * textbook one: for every packed sequence b (tokens cu[b] .. cu[b+1]-1, length L) and head h,
 *
 *     S_ij  = scale * sum_c Q_ic K_jc                      (i, j relative to the sequence)
 *     key j is visible to query i  iff  (not causal) or j <= i
 *     m_i   = max_j S_ij,  l_i = sum_j exp(S_ij - m_i)     (visible j only)
 *     P_ij  = exp(S_ij - m_i) / l_i,   lse_i = m_i + ln l_i
 *     O_i   = sum_j P_ij V_j
 *
 * and for the loss  sum_i <O_i, dO_i>:
 *
 *     D_i   = sum_c dO_ic O_ic            (O is this file's own fp64 O)
 *     dP_ij = sum_c dO_ic V_jc
 *     dS_ij = P_ij (dP_ij - D_i)
 *     dQ_i  = scale * sum_j dS_ij K_j
 *     dK_j  = scale * sum_i dS_ij Q_i
 *     dV_j  = sum_i P_ij dO_i
 *
 * Inputs are bf16 bit patterns (uint16) laid out [T, H, d]; each is widened exactly to
 * double.  Outputs are double: O, dQ, dK, dV as [T, H, d]; lse as [H, T].
 * Softmax is the exact two-pass form per row.  There is no tiling and no online rescaling.
 * Matrix-vector products are written as "for each term, add a scaled vector" so that a
 * compiler may vectorise them without changing the order of any sum.
 *
 * Entry points:
 *   oracle_attn_fwd   all rows of all sequences and heads
 *   oracle_attn_bwd   all gradients (runs the forward internally)
 *   oracle_attn_rows  O, lse, dQ for chosen query rows of one (sequence, head)
 *   oracle_attn_cols  dK, dV for chosen key columns of one (sequence, head)
 * The last two exist because the definition separates by row and by column: a row needs
 * only K and V; a column needs m_i, l_i, D_i of every row that sees it.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define HOT __attribute__((target_clones("default", "avx2", "avx512f")))

static double bf16_to_double(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Widen one (sequence, head) slice x[start .. start+L-1][h][0..d-1] into a dense L x d
 * array (row-major) and, if xt != NULL, its transpose d x L. */
static void widen_slice(const uint16_t* x, int64_t start, int64_t L, int H, int h, int d,
                        double* dense, double* xt)
{
    for (int64_t i = 0; i < L; ++i) {
        const uint16_t* row = x + ((start + i) * H + h) * (int64_t)d;
        for (int c = 0; c < d; ++c) {
            double val = bf16_to_double(row[c]);
            if (dense) dense[i * d + c] = val;
            if (xt) xt[(int64_t)c * L + i] = val;
        }
    }
}

/* s[j] = scale * sum_c a[c] * Bt[c][j]  for j in [0, n).  Bt is d x ldb, row c holds element c
 * of every vector. */
HOT static void scaled_dots(const double* a, const double* Bt, int64_t ldb, int d, int64_t n,
                            double scale, double* s)
{
    for (int64_t j = 0; j < n; ++j) s[j] = 0.0;
    for (int c = 0; c < d; ++c) {
        const double ac = a[c];
        const double* brow = Bt + (int64_t)c * ldb;
        for (int64_t j = 0; j < n; ++j) s[j] += ac * brow[j];
    }
    for (int64_t j = 0; j < n; ++j) s[j] *= scale;
}

/* out[c] = sum_j w[j] * X[j][c]   (X is n x d, row-major) */
HOT static void weighted_sum(const double* w, const double* X, int d, int64_t n, double* out)
{
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        const double wj = w[j];
        const double* xr = X + j * d;
        for (int c = 0; c < d; ++c) out[c] += wj * xr[c];
    }
}

/* Exact two-pass softmax statistics of s[0..n): returns m, writes l, replaces s by exp(s-m)/l. */
HOT static double softmax_row(double* s, int64_t n, double* l_out)
{
    double m = s[0];
    for (int64_t j = 1; j < n; ++j) m = s[j] > m ? s[j] : m;
    double l = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        s[j] = exp(s[j] - m);
        l += s[j];
    }
    for (int64_t j = 0; j < n; ++j) s[j] /= l;
    *l_out = l;
    return m;
}

/* Number of keys visible to query row i of a length-L sequence. */
static int64_t visible(int64_t i, int64_t L, int causal) { return causal ? i + 1 : L; }

/* ---------------------------------------------------------------------------------------- */

int oracle_attn_fwd(const uint16_t* q, const uint16_t* k, const uint16_t* v, const int32_t* cu,
                    int B, int H, int d, int causal, double scale, double* O, double* lse)
{
    if (!q || !k || !v || !cu || B < 0 || H <= 0 || d <= 0) return 1;
    const int64_t T = cu[B];
    for (int b = 0; b < B; ++b) {
        const int64_t start = cu[b], L = cu[b + 1] - cu[b];
        if (L < 0) return 1;
        if (L == 0) continue;
        for (int h = 0; h < H; ++h) {
            double* Qd = malloc(sizeof(double) * L * d);
            double* Kt = malloc(sizeof(double) * L * d);
            double* Vd = malloc(sizeof(double) * L * d);
            if (!Qd || !Kt || !Vd) return 2;
            widen_slice(q, start, L, H, h, d, Qd, NULL);
            widen_slice(k, start, L, H, h, d, NULL, Kt);
            widen_slice(v, start, L, H, h, d, Vd, NULL);
#pragma omp parallel
            {
                double* s = malloc(sizeof(double) * L);
#pragma omp for schedule(dynamic, 8)
                for (int64_t i = 0; i < L; ++i) {
                    const int64_t n = visible(i, L, causal);
                    double l;
                    scaled_dots(Qd + i * d, Kt, L, d, n, scale, s);
                    double m = softmax_row(s, n, &l);
                    weighted_sum(s, Vd, d, n, O + ((start + i) * H + h) * (int64_t)d);
                    lse[(int64_t)h * T + start + i] = m + log(l);
                }
                free(s);
            }
            free(Qd); free(Kt); free(Vd);
        }
    }
    return 0;
}

/* Gradients of one (sequence, head).  Row phase: dQ and the per-row statistics m, l, D.
 * Column phase: dK, dV, each column summing over the rows that see it. */
static int bwd_slice(const uint16_t* q, const uint16_t* k, const uint16_t* v, const uint16_t* dO,
                     int64_t start, int64_t L, int H, int h, int d, int causal, double scale,
                     double* dQ, double* dK, double* dV)
{
    double* Qd = malloc(sizeof(double) * L * d);
    double* Qt = malloc(sizeof(double) * L * d);
    double* Kd = malloc(sizeof(double) * L * d);
    double* Kt = malloc(sizeof(double) * L * d);
    double* Vd = malloc(sizeof(double) * L * d);
    double* Vt = malloc(sizeof(double) * L * d);
    double* Gd = malloc(sizeof(double) * L * d);   /* dO */
    double* Gt = malloc(sizeof(double) * L * d);
    double* m = malloc(sizeof(double) * L);
    double* l = malloc(sizeof(double) * L);
    double* D = malloc(sizeof(double) * L);
    if (!Qd || !Qt || !Kd || !Kt || !Vd || !Vt || !Gd || !Gt || !m || !l || !D) return 2;
    widen_slice(q, start, L, H, h, d, Qd, Qt);
    widen_slice(k, start, L, H, h, d, Kd, Kt);
    widen_slice(v, start, L, H, h, d, Vd, Vt);
    widen_slice(dO, start, L, H, h, d, Gd, Gt);

#pragma omp parallel
    {
        double* p = malloc(sizeof(double) * L);
        double* dp = malloc(sizeof(double) * L);
        double* o = malloc(sizeof(double) * d);
        double* acc = malloc(sizeof(double) * d);
#pragma omp for schedule(dynamic, 8)
        for (int64_t i = 0; i < L; ++i) {
            const int64_t n = visible(i, L, causal);
            scaled_dots(Qd + i * d, Kt, L, d, n, scale, p);
            m[i] = softmax_row(p, n, &l[i]);
            weighted_sum(p, Vd, d, n, o);
            double Di = 0.0;
            for (int c = 0; c < d; ++c) Di += Gd[i * d + c] * o[c];
            D[i] = Di;
            scaled_dots(Gd + i * d, Vt, L, d, n, 1.0, dp);
            for (int64_t j = 0; j < n; ++j) dp[j] = p[j] * (dp[j] - Di);   /* dS_ij */
            weighted_sum(dp, Kd, d, n, acc);
            double* out = dQ + ((start + i) * H + h) * (int64_t)d;
            for (int c = 0; c < d; ++c) out[c] = scale * acc[c];
        }
#pragma omp for schedule(dynamic, 8)
        for (int64_t j = 0; j < L; ++j) {
            /* rows that see key j: all rows, or rows i >= j when causal */
            const int64_t i0 = causal ? j : 0, n = L - i0;
            /* p[i] = S_ij for i in [i0, L): a dot of K_j with every Q_i */
            scaled_dots(Kd + j * d, Qt + i0, L, d, n, scale, p);
            scaled_dots(Vd + j * d, Gt + i0, L, d, n, 1.0, dp);             /* dP_ij */
            for (int64_t t = 0; t < n; ++t) {
                const int64_t i = i0 + t;
                p[t] = exp(p[t] - m[i]) / l[i];                             /* P_ij  */
                dp[t] = p[t] * (dp[t] - D[i]);                              /* dS_ij */
            }
            weighted_sum(p, Gd + i0 * d, d, n, dV + ((start + j) * H + h) * (int64_t)d);
            weighted_sum(dp, Qd + i0 * d, d, n, acc);
            double* out = dK + ((start + j) * H + h) * (int64_t)d;
            for (int c = 0; c < d; ++c) out[c] = scale * acc[c];
        }
        free(p); free(dp); free(o); free(acc);
    }
    free(Qd); free(Qt); free(Kd); free(Kt); free(Vd); free(Vt); free(Gd); free(Gt);
    free(m); free(l); free(D);
    return 0;
}

int oracle_attn_bwd(const uint16_t* q, const uint16_t* k, const uint16_t* v, const uint16_t* dO,
                    const int32_t* cu, int B, int H, int d, int causal, double scale,
                    double* dQ, double* dK, double* dV)
{
    if (!q || !k || !v || !dO || !cu || B < 0 || H <= 0 || d <= 0) return 1;
    for (int b = 0; b < B; ++b) {
        const int64_t start = cu[b], L = cu[b + 1] - cu[b];
        if (L < 0) return 1;
        if (L == 0) continue;
        for (int h = 0; h < H; ++h) {
            int rc = bwd_slice(q, k, v, dO, start, L, H, h, d, causal, scale, dQ, dK, dV);
            if (rc) return rc;
        }
    }
    return 0;
}

/* O_i, lse_i, dQ_i for the listed rows (relative to the sequence start) of sequence `seq`,
 * head `head`.  Outputs: O_rows, dQ_rows are [n_rows, d]; lse_rows is [n_rows].
 * dO may be NULL, in which case dQ_rows is not written. */
int oracle_attn_rows(const uint16_t* q, const uint16_t* k, const uint16_t* v, const uint16_t* dO,
                     const int32_t* cu, int H, int d, int causal, double scale, int seq, int head,
                     int n_rows, const int32_t* rows, double* O_rows, double* lse_rows,
                     double* dQ_rows)
{
    const int64_t start = cu[seq], L = cu[seq + 1] - cu[seq];
    if (L <= 0 || head < 0 || head >= H) return 1;
    for (int r = 0; r < n_rows; ++r)
        if (rows[r] < 0 || rows[r] >= L) return 1;
    double* Kd = malloc(sizeof(double) * L * d);
    double* Kt = malloc(sizeof(double) * L * d);
    double* Vd = malloc(sizeof(double) * L * d);
    double* Vt = malloc(sizeof(double) * L * d);
    if (!Kd || !Kt || !Vd || !Vt) return 2;
    widen_slice(k, start, L, H, head, d, Kd, Kt);
    widen_slice(v, start, L, H, head, d, Vd, Vt);
#pragma omp parallel
    {
        double* p = malloc(sizeof(double) * L);
        double* dp = malloc(sizeof(double) * L);
        double* qi = malloc(sizeof(double) * d);
        double* gi = malloc(sizeof(double) * d);
        double* acc = malloc(sizeof(double) * d);
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n_rows; ++r) {
            const int64_t i = rows[r], n = visible(i, L, causal);
            double li;
            widen_slice(q, start + i, 1, H, head, d, qi, NULL);
            scaled_dots(qi, Kt, L, d, n, scale, p);
            double mi = softmax_row(p, n, &li);
            double* o = O_rows + (int64_t)r * d;
            weighted_sum(p, Vd, d, n, o);
            lse_rows[r] = mi + log(li);
            if (dO) {
                widen_slice(dO, start + i, 1, H, head, d, gi, NULL);
                double Di = 0.0;
                for (int c = 0; c < d; ++c) Di += gi[c] * o[c];
                scaled_dots(gi, Vt, L, d, n, 1.0, dp);
                for (int64_t j = 0; j < n; ++j) dp[j] = p[j] * (dp[j] - Di);
                weighted_sum(dp, Kd, d, n, acc);
                for (int c = 0; c < d; ++c) dQ_rows[(int64_t)r * d + c] = scale * acc[c];
            }
        }
        free(p); free(dp); free(qi); free(gi); free(acc);
    }
    free(Kd); free(Kt); free(Vd); free(Vt);
    return 0;
}

/* dK_j, dV_j for the listed key columns of sequence `seq`, head `head`; outputs [n_cols, d].
 * Rows that cannot see any listed column (causal: rows before the smallest listed column) are
 * skipped; every other row's m, l, D is computed first, exactly as in the row phase above. */
int oracle_attn_cols(const uint16_t* q, const uint16_t* k, const uint16_t* v, const uint16_t* dO,
                     const int32_t* cu, int H, int d, int causal, double scale, int seq, int head,
                     int n_cols, const int32_t* cols, double* dK_cols, double* dV_cols)
{
    const int64_t start = cu[seq], L = cu[seq + 1] - cu[seq];
    if (L <= 0 || head < 0 || head >= H || n_cols <= 0) return 1;
    int64_t jmin = L;
    for (int r = 0; r < n_cols; ++r) {
        if (cols[r] < 0 || cols[r] >= L) return 1;
        if (cols[r] < jmin) jmin = cols[r];
    }
    const int64_t r0 = causal ? jmin : 0;      /* first row that matters */
    double* Qd = malloc(sizeof(double) * L * d);
    double* Qt = malloc(sizeof(double) * L * d);
    double* Kt = malloc(sizeof(double) * L * d);
    double* Vd = malloc(sizeof(double) * L * d);
    double* Gd = malloc(sizeof(double) * L * d);
    double* Gt = malloc(sizeof(double) * L * d);
    double* m = malloc(sizeof(double) * L);
    double* l = malloc(sizeof(double) * L);
    double* D = malloc(sizeof(double) * L);
    if (!Qd || !Qt || !Kt || !Vd || !Gd || !Gt || !m || !l || !D) return 2;
    widen_slice(q, start, L, H, head, d, Qd, Qt);
    widen_slice(k, start, L, H, head, d, NULL, Kt);
    widen_slice(v, start, L, H, head, d, Vd, NULL);
    widen_slice(dO, start, L, H, head, d, Gd, Gt);
#pragma omp parallel
    {
        double* p = malloc(sizeof(double) * L);
        double* dp = malloc(sizeof(double) * L);
        double* o = malloc(sizeof(double) * d);
        double* kj = malloc(sizeof(double) * d);
        double* vj = malloc(sizeof(double) * d);
        double* acc = malloc(sizeof(double) * d);
#pragma omp for schedule(dynamic, 8)
        for (int64_t i = r0; i < L; ++i) {
            const int64_t n = visible(i, L, causal);
            scaled_dots(Qd + i * d, Kt, L, d, n, scale, p);
            m[i] = softmax_row(p, n, &l[i]);
            weighted_sum(p, Vd, d, n, o);
            double Di = 0.0;
            for (int c = 0; c < d; ++c) Di += Gd[i * d + c] * o[c];
            D[i] = Di;
        }
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n_cols; ++r) {
            const int64_t j = cols[r];
            const int64_t i0 = causal ? j : 0, n = L - i0;
            widen_slice(k, start + j, 1, H, head, d, kj, NULL);
            widen_slice(v, start + j, 1, H, head, d, vj, NULL);
            scaled_dots(kj, Qt + i0, L, d, n, scale, p);
            scaled_dots(vj, Gt + i0, L, d, n, 1.0, dp);
            for (int64_t t = 0; t < n; ++t) {
                const int64_t i = i0 + t;
                p[t] = exp(p[t] - m[i]) / l[i];
                dp[t] = p[t] * (dp[t] - D[i]);
            }
            weighted_sum(p, Gd + i0 * d, d, n, dV_cols + (int64_t)r * d);
            weighted_sum(dp, Qd + i0 * d, d, n, acc);
            for (int c = 0; c < d; ++c) dK_cols[(int64_t)r * d + c] = scale * acc[c];
        }
        free(p); free(dp); free(o); free(kj); free(vj); free(acc);
    }
    free(Qd); free(Qt); free(Kt); free(Vd); free(Gd); free(Gt);
    free(m); free(l); free(D);
    return 0;
}
