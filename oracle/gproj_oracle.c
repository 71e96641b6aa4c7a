/*
 * FP64 CPU oracle for softmax attention forward and its exact vector-Jacobian
 * product (the target every gradient error is measured against).
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call this file;
 * it shares no code with the CUDA kernels and is never tuned for speed.
 *
 * What it computes (Section 3.1, Eq. "row-attention" and Eq. "row-gradients";
 * metric and reference convention: Appendix "Accuracy and Cost", paragraph
 * "Reference and metric"): for one head with BF16 inputs Q, K, V, U=dO of shape
 * [N x d], decoded exactly to FP64, scale alpha, support L_i = {j <= i} (causal)
 * or all j,
 *
 *   s_ij = alpha * sum_c q_ic k_jc          p_ij = exp(s_ij) / sum_{l in L_i} exp(s_il)
 *   LSE_i = ln sum_{l in L_i} exp(s_il)     o_i  = sum_j p_ij v_j
 *   a_ij = sum_c u_ic v_jc                  mu_a,i = sum_j p_ij a_ij
 *   g_ij = p_ij (a_ij - mu_a,i)
 *   dq_i = alpha sum_j g_ij k_j     dk_j = alpha sum_i g_ij q_i     dv_j = sum_i p_ij u_i
 *
 * Outputs stay in FP64 (the paper's references are "uncast").  The max is
 * subtracted before exp only to keep exp in range; it cancels in p.
 *
 * Parity pins live in tests/ (torch float64 autograd, finite differences, a
 * second formulation, closed forms, translation invariants).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_bits_to_f64(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double *decode_tile(const uint16_t *x, size_t n)
{
    double *out = (double *)malloc(n * sizeof(double));
    if (!out) return NULL;
    for (size_t i = 0; i < n; ++i) out[i] = bf16_bits_to_f64(x[i]);
    return out;
}

int gproj_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Query-row quantities for the listed rows of one head.
 *   q,k,v,u : BF16 bit patterns, [N x d], row-major (d fastest)
 *   rows    : nrows query indices in [0,N)
 * Outputs (row r of each corresponds to rows[r]):
 *   O [nrows x d], LSE [nrows], MUA [nrows] (= mu_a, the exact value of the
 *   row statistic D), dQ [nrows x d].
 * Returns 0, or -1 on allocation failure / bad arguments.
 */
int gproj_oracle_head_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v, const uint16_t *u,
                           int N, int d, double alpha, int causal,
                           const int *rows, int nrows,
                           double *O, double *LSE, double *MUA, double *dQ)
{
    if (N <= 0 || d <= 0 || nrows < 0) return -1;
    size_t nd = (size_t)N * (size_t)d;
    double *Q = decode_tile(q, nd), *K = decode_tile(k, nd), *V = decode_tile(v, nd), *U = decode_tile(u, nd);
    int fail = (!Q || !K || !V || !U);

#pragma omp parallel
    {
        double *s = (double *)malloc((size_t)N * sizeof(double));
        double *a = (double *)malloc((size_t)N * sizeof(double));
        if (!s || !a) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 4)
            for (int r = 0; r < nrows; ++r) {
                int i = rows[r];
                int L = causal ? i + 1 : N;
                const double *qi = Q + (size_t)i * d, *ui = U + (size_t)i * d;
                double smax = -INFINITY;
                for (int j = 0; j < L; ++j) {
                    const double *kj = K + (size_t)j * d, *vj = V + (size_t)j * d;
                    double dot = 0.0, av = 0.0;
                    for (int c = 0; c < d; ++c) { dot += qi[c] * kj[c]; av += ui[c] * vj[c]; }
                    s[j] = alpha * dot;
                    a[j] = av;
                    if (s[j] > smax) smax = s[j];
                }
                double Z = 0.0;
                for (int j = 0; j < L; ++j) Z += exp(s[j] - smax);
                double lse = smax + log(Z);
                double mua = 0.0;
                for (int j = 0; j < L; ++j) { s[j] = exp(s[j] - smax) / Z; mua += s[j] * a[j]; }   /* s now holds p */
                double *o = O + (size_t)r * d, *dq = dQ + (size_t)r * d;
                for (int c = 0; c < d; ++c) { o[c] = 0.0; dq[c] = 0.0; }
                for (int j = 0; j < L; ++j) {
                    const double *kj = K + (size_t)j * d, *vj = V + (size_t)j * d;
                    double p = s[j], g = p * (a[j] - mua);
                    for (int c = 0; c < d; ++c) { o[c] += p * vj[c]; dq[c] += g * kj[c]; }
                }
                for (int c = 0; c < d; ++c) dq[c] *= alpha;
                LSE[r] = lse;
                MUA[r] = mua;
            }
        }
        free(s);
        free(a);
    }
    free(Q); free(K); free(V); free(U);
    return fail ? -1 : 0;
}

/*
 * Key-row quantities for the listed keys of one head, given LSE_i and mu_a,i of
 * EVERY query row (from gproj_oracle_head_rows over all rows):
 *   dK [nkeys x d], dV [nkeys x d], row r corresponding to keys[r].
 * p_ij is re-evaluated from its definition as exp(s_ij - LSE_i).
 */
int gproj_oracle_head_keys(const uint16_t *q, const uint16_t *k, const uint16_t *v, const uint16_t *u,
                           int N, int d, double alpha, int causal,
                           const double *LSE, const double *MUA,
                           const int *keys, int nkeys,
                           double *dK, double *dV)
{
    if (N <= 0 || d <= 0 || nkeys < 0) return -1;
    size_t nd = (size_t)N * (size_t)d;
    double *Q = decode_tile(q, nd), *K = decode_tile(k, nd), *V = decode_tile(v, nd), *U = decode_tile(u, nd);
    if (!Q || !K || !V || !U) { free(Q); free(K); free(V); free(U); return -1; }

#pragma omp parallel for schedule(dynamic, 4)
    for (int r = 0; r < nkeys; ++r) {
        int j = keys[r];
        const double *kj = K + (size_t)j * d, *vj = V + (size_t)j * d;
        double *dk = dK + (size_t)r * d, *dv = dV + (size_t)r * d;
        for (int c = 0; c < d; ++c) { dk[c] = 0.0; dv[c] = 0.0; }
        int i0 = causal ? j : 0;
        for (int i = i0; i < N; ++i) {
            const double *qi = Q + (size_t)i * d, *ui = U + (size_t)i * d;
            double dot = 0.0, av = 0.0;
            for (int c = 0; c < d; ++c) { dot += qi[c] * kj[c]; av += ui[c] * vj[c]; }
            double p = exp(alpha * dot - LSE[i]);
            double g = p * (av - MUA[i]);
            for (int c = 0; c < d; ++c) { dk[c] += g * qi[c]; dv[c] += p * ui[c]; }
        }
        for (int c = 0; c < d; ++c) dk[c] *= alpha;
    }
    free(Q); free(K); free(V); free(U);
    return 0;
}

/*
 * Rectangular problems: N_q queries against N_k keys of one head (the paper's synthetic suite lists "unequal lengths" and
 * "empty causal rows", Appendix "Synthetic Numerical Suite"; Algorithm 1 line 14 gives the rule for a row of zero mass).
 * Support of query row i: all keys (causal = 0), or the keys j <= i + (N_k - N_q), i.e. the causal diagonal ends at the
 * LAST query and the LAST key (the alignment of the FlashAttention kernels the paper builds on).  A row whose support is
 * empty has no probabilities: O_i = 0, dq_i = 0, mu_a,i = 0, it contributes to no dk_j / dv_j, and its LSE is reported
 * as +infinity, so that exp(s - LSE) = 0 wherever that row is re-evaluated.
 * These are separate functions; the square ones above are left as they were.
 */
int gproj_oracle_rect_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v, const uint16_t *u,
                           int Nq, int Nk, int d, double alpha, int causal,
                           const int *rows, int nrows,
                           double *O, double *LSE, double *MUA, double *dQ)
{
    if (Nq <= 0 || Nk <= 0 || d <= 0 || nrows < 0) return -1;
    double *Q = decode_tile(q, (size_t)Nq * d), *K = decode_tile(k, (size_t)Nk * d);
    double *V = decode_tile(v, (size_t)Nk * d), *U = decode_tile(u, (size_t)Nq * d);
    int fail = (!Q || !K || !V || !U);
    const int off = Nk - Nq;

#pragma omp parallel
    {
        double *s = (double *)malloc((size_t)Nk * sizeof(double));
        double *a = (double *)malloc((size_t)Nk * sizeof(double));
        if (!s || !a) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 4)
            for (int r = 0; r < nrows; ++r) {
                int i = rows[r];
                int L = causal ? i + off + 1 : Nk;          /* number of supported keys: j = 0 .. L-1 */
                if (L > Nk) L = Nk;
                double *o = O + (size_t)r * d, *dq = dQ + (size_t)r * d;
                for (int c = 0; c < d; ++c) { o[c] = 0.0; dq[c] = 0.0; }
                if (L <= 0) { LSE[r] = INFINITY; MUA[r] = 0.0; continue; }
                const double *qi = Q + (size_t)i * d, *ui = U + (size_t)i * d;
                double smax = -INFINITY;
                for (int j = 0; j < L; ++j) {
                    const double *kj = K + (size_t)j * d, *vj = V + (size_t)j * d;
                    double dot = 0.0, av = 0.0;
                    for (int c = 0; c < d; ++c) { dot += qi[c] * kj[c]; av += ui[c] * vj[c]; }
                    s[j] = alpha * dot;
                    a[j] = av;
                    if (s[j] > smax) smax = s[j];
                }
                double Z = 0.0;
                for (int j = 0; j < L; ++j) Z += exp(s[j] - smax);
                double mua = 0.0;
                for (int j = 0; j < L; ++j) { s[j] = exp(s[j] - smax) / Z; mua += s[j] * a[j]; }   /* s now holds p */
                for (int j = 0; j < L; ++j) {
                    const double *kj = K + (size_t)j * d, *vj = V + (size_t)j * d;
                    double p = s[j], g = p * (a[j] - mua);
                    for (int c = 0; c < d; ++c) { o[c] += p * vj[c]; dq[c] += g * kj[c]; }
                }
                for (int c = 0; c < d; ++c) dq[c] *= alpha;
                LSE[r] = smax + log(Z);
                MUA[r] = mua;
            }
        }
        free(s);
        free(a);
    }
    free(Q); free(K); free(V); free(U);
    return fail ? -1 : 0;
}

int gproj_oracle_rect_keys(const uint16_t *q, const uint16_t *k, const uint16_t *v, const uint16_t *u,
                           int Nq, int Nk, int d, double alpha, int causal,
                           const double *LSE, const double *MUA,
                           const int *keys, int nkeys,
                           double *dK, double *dV)
{
    if (Nq <= 0 || Nk <= 0 || d <= 0 || nkeys < 0) return -1;
    double *Q = decode_tile(q, (size_t)Nq * d), *K = decode_tile(k, (size_t)Nk * d);
    double *V = decode_tile(v, (size_t)Nk * d), *U = decode_tile(u, (size_t)Nq * d);
    if (!Q || !K || !V || !U) { free(Q); free(K); free(V); free(U); return -1; }
    const int off = Nk - Nq;

#pragma omp parallel for schedule(dynamic, 4)
    for (int r = 0; r < nkeys; ++r) {
        int j = keys[r];
        const double *kj = K + (size_t)j * d, *vj = V + (size_t)j * d;
        double *dk = dK + (size_t)r * d, *dv = dV + (size_t)r * d;
        for (int c = 0; c < d; ++c) { dk[c] = 0.0; dv[c] = 0.0; }
        int i0 = causal ? j - off : 0;                      /* first query whose support holds key j */
        if (i0 < 0) i0 = 0;
        for (int i = i0; i < Nq; ++i) {
            const double *qi = Q + (size_t)i * d, *ui = U + (size_t)i * d;
            double dot = 0.0, av = 0.0;
            for (int c = 0; c < d; ++c) { dot += qi[c] * kj[c]; av += ui[c] * vj[c]; }
            double p = exp(alpha * dot - LSE[i]);
            double g = p * (av - MUA[i]);
            for (int c = 0; c < d; ++c) { dk[c] += g * qi[c]; dv[c] += p * ui[c]; }
        }
        for (int c = 0; c < d; ++c) dk[c] *= alpha;
    }
    free(Q); free(K); free(V); free(U);
    return 0;
}
