/*
 * fp64 CPU oracle for the Tensor-Train (TT) embedding gather.  TEST INFRASTRUCTURE ONLY.
 *
 * Only the tests, the smoke check and the benchmark's cpu_baseline / reference arm may call this.
 * It shares no code, header, table or helper with the CUDA library, and the CUDA library never
 * calls it.  It is deliberately plain: one lookup at a time, no sorting, no de-duplication, no
 * prefix sharing, no blocking.  Every function is the definition written out.
 *
 * Data model (paper Sec. 2.1 / 2.4): a table of N rows and D columns is stored as K TT-cores.
 * Core k is the 4-index array G_k[a][i][j][b] with a < r_{k-1}, i < n_k, j < d_k, b < r_k
 * (r_0 = r_K = 1), stored C-contiguous in exactly that index order.  prod(n_k) >= N, prod(d_k) = D.
 *
 * Parity pins (see tests/test_oracle_*.py): dense brute-force definition vs sequential contraction;
 * closed forms (rank-1, all-ones, sum-separable rank-2); exact finite differences for the backward
 * (the loss is linear in every single core entry); library routines (einsum, embedding_bag).
 * The paper's latency tables are "parity unpinned": other hardware, dataset absent.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define TT_MAX_K 8

/* Eq. 1: digit k of row g is floor(g / prod_{j>k} n_j) mod n_k; digit 1 is the most significant. */
void tt_oracle_digits(int64_t g, int K, const int64_t* n, int64_t* digits)
{
    for (int k = 0; k < K; ++k) {
        int64_t suffix = 1;
        for (int j = k + 1; j < K; ++j) suffix *= n[j];
        digits[k] = (g / suffix) % n[k];
    }
}

static inline double core_at(const double* G, const int64_t* n, const int64_t* d, const int64_t* r,
                             int k, int64_t a, int64_t i, int64_t j, int64_t b)
{
    return G[((a * n[k] + i) * d[k] + j) * r[k + 1] + b];
}

static inline int64_t core_off(const int64_t* n, const int64_t* d, const int64_t* r,
                               int k, int64_t a, int64_t i, int64_t j, int64_t b)
{
    return ((a * n[k] + i) * d[k] + j) * r[k + 1] + b;
}

static int64_t max_partial_size(int K, const int64_t* d, const int64_t* r)
{
    int64_t best = 1, rows = 1;
    for (int k = 0; k < K; ++k) {
        rows *= d[k];
        if (rows * r[k + 1] > best) best = rows * r[k + 1];
    }
    return best;
}

/*
 * Sequential contraction (Sec. 3.2, "C = A.B, E = C.D"):
 *   P_1[j1][b]             = G_1[0][i_1][j1][b]
 *   P_k[(p, j)][b]         = sum_a P_{k-1}[p][a] * G_k[a][i_k][j][b]      (p runs over prod_{m<k} d_m)
 * The row is P_K flattened row-major, so the column index is (j_1, .., j_K) with j_1 most significant.
 * `partials` (optional) receives P_1..P_K back to back, each in its own [rows][r_k] layout.
 */
static void row_forward(int K, const int64_t* n, const int64_t* d, const int64_t* r,
                        const double* const* cores, const int64_t* dig,
                        double* P_all, int64_t* P_off, double* E)
{
    int64_t rows = d[0];
    int64_t off = 0;
    P_off[0] = 0;
    for (int64_t j = 0; j < d[0]; ++j)
        for (int64_t b = 0; b < r[1]; ++b)
            P_all[j * r[1] + b] = core_at(cores[0], n, d, r, 0, 0, dig[0], j, b);
    for (int k = 1; k < K; ++k) {
        const double* Pp = P_all + off;
        off += rows * r[k];
        P_off[k] = off;
        double* Pn = P_all + off;
        for (int64_t p = 0; p < rows; ++p)
            for (int64_t j = 0; j < d[k]; ++j)
                for (int64_t b = 0; b < r[k + 1]; ++b) {
                    double s = 0.0;
                    for (int64_t a = 0; a < r[k]; ++a)
                        s += Pp[p * r[k] + a] * core_at(cores[k], n, d, r, k, a, dig[k], j, b);
                    Pn[(p * d[k] + j) * r[k + 1] + b] = s;
                }
        rows *= d[k];
    }
    if (E) {
        const double* PK = P_all + off;
        for (int64_t e = 0; e < rows; ++e) E[e] = PK[e];
    }
}

static int64_t partial_total(int K, const int64_t* d, const int64_t* r)
{
    int64_t tot = 0, rows = 1;
    for (int k = 0; k < K; ++k) { rows *= d[k]; tot += rows * r[k + 1]; }
    return tot;
}

/* One row of the table, D doubles. */
void tt_oracle_row(int K, const int64_t* n, const int64_t* d, const int64_t* r,
                   const double* const* cores, int64_t g, double* E)
{
    int64_t dig[TT_MAX_K], P_off[TT_MAX_K];
    double* P_all = (double*)malloc(sizeof(double) * (size_t)partial_total(K, d, r));
    tt_oracle_digits(g, K, n, dig);
    row_forward(K, n, d, r, cores, dig, P_all, P_off, E);
    free(P_all);
}

/*
 * Pooled forward of ONE table: out[b*out_stride + j] = sum over lookups l in bag b of a_l * row(indices[l])[j]
 * (duplicates counted, empty bag -> zeros).  offsets has B+1 entries.  The paper pools by plain sum (a_l = 1:
 * weights == NULL, mean == 0).  Two extensions follow the usual embedding-bag operator: per-lookup weights
 * (a_l = weights[l]) and mean pooling (a_l = 1 / number of lookups of the bag, invalid ones included).
 * Returns the number of indices outside [0, N) (they contribute nothing).
 */
int64_t tt_oracle_forward(int K, const int64_t* n, const int64_t* d, const int64_t* r, int64_t N,
                          const double* const* cores, const int64_t* indices, const int64_t* offsets,
                          int64_t B, double* out, int64_t out_stride, const double* weights, int mean)
{
    int64_t D = 1;
    for (int k = 0; k < K; ++k) D *= d[k];
    int64_t bad = 0;
    size_t ptot = (size_t)partial_total(K, d, r);
#pragma omp parallel reduction(+ : bad)
    {
        double* P_all = (double*)malloc(sizeof(double) * ptot);
        double* E = (double*)malloc(sizeof(double) * (size_t)D);
        int64_t dig[TT_MAX_K], P_off[TT_MAX_K];
#pragma omp for schedule(dynamic, 16)
        for (int64_t b = 0; b < B; ++b) {
            double* o = out + b * out_stride;
            for (int64_t j = 0; j < D; ++j) o[j] = 0.0;
            const int64_t len = offsets[b + 1] - offsets[b];
            for (int64_t l = offsets[b]; l < offsets[b + 1]; ++l) {
                int64_t g = indices[l];
                if (g < 0 || g >= N) { ++bad; continue; }
                double a = weights ? weights[l] : 1.0;
                if (mean) a /= (double)len;
                tt_oracle_digits(g, K, n, dig);
                row_forward(K, n, d, r, cores, dig, P_all, P_off, E);
                for (int64_t j = 0; j < D; ++j) o[j] += a * E[j];
            }
        }
        free(P_all);
        free(E);
    }
    return bad;
}

/*
 * Backward of ONE table (Sec. 3.2): for every lookup l of bag b, independently,
 *   dP_K = grad_out[b]                                   (shape [D][1])
 *   for k = K..2:  dG_k[a][i_k][j][b'] += sum_p P_{k-1}[p][a] * dP_k[(p,j)][b']       ("dD = C^T.dE")
 *                  dP_{k-1}[p][a]       = sum_{j,b'} dP_k[(p,j)][b'] * G_k[a][i_k][j][b']  ("dC = dE.D^T")
 *   dG_1[0][i_1][j][b'] += dP_1[j][b']
 * No regrouping by shared prefix (Eq. 2) is used here; that the regrouped form agrees is a test.
 * With per-lookup weights or mean pooling (see tt_oracle_forward) dP_K = a_l * grad_out[b].
 * core_grads[k] has the shape of cores[k] and is ACCUMULATED INTO (caller zeroes it).
 * Bags are spread over OpenMP threads; each thread accumulates into a private fp64 copy which is
 * added to core_grads at the end (with one thread this is exactly the lookup order).
 */
int64_t tt_oracle_backward(int K, const int64_t* n, const int64_t* d, const int64_t* r, int64_t N,
                           const double* const* cores, const int64_t* indices, const int64_t* offsets,
                           int64_t B, const double* grad_out, int64_t grad_stride, double* const* core_grads,
                           const double* weights, int mean)
{
    int64_t D = 1;
    for (int k = 0; k < K; ++k) D *= d[k];
    int64_t bad = 0;
    size_t ptot = (size_t)partial_total(K, d, r);
    int64_t pmax = max_partial_size(K, d, r);
    int64_t csize[TT_MAX_K];
    for (int k = 0; k < K; ++k) csize[k] = r[k] * n[k] * d[k] * r[k + 1];
#pragma omp parallel reduction(+ : bad)
    {
        double* P_all = (double*)malloc(sizeof(double) * ptot);
        double* dP = (double*)malloc(sizeof(double) * (size_t)pmax);
        double* dPprev = (double*)malloc(sizeof(double) * (size_t)pmax);
        double* priv[TT_MAX_K];
        for (int k = 0; k < K; ++k) priv[k] = (double*)calloc((size_t)csize[k], sizeof(double));
        int64_t dig[TT_MAX_K], P_off[TT_MAX_K];
#pragma omp for schedule(dynamic, 16)
        for (int64_t b = 0; b < B; ++b) {
            const double* go = grad_out + b * grad_stride;
            const int64_t len = offsets[b + 1] - offsets[b];
            for (int64_t l = offsets[b]; l < offsets[b + 1]; ++l) {
                int64_t g = indices[l];
                if (g < 0 || g >= N) { ++bad; continue; }
                double a = weights ? weights[l] : 1.0;
                if (mean) a /= (double)len;
                tt_oracle_digits(g, K, n, dig);
                row_forward(K, n, d, r, cores, dig, P_all, P_off, NULL);
                for (int64_t e = 0; e < D; ++e) dP[e] = a * go[e];
                int64_t rows = D; /* rows of the partial product after core k */
                for (int k = K - 1; k >= 1; --k) {
                    int64_t prow = rows / d[k]; /* rows of the partial product before core k */
                    const double* Pp = P_all + P_off[k - 1];
                    for (int64_t p = 0; p < prow; ++p)
                        for (int64_t a = 0; a < r[k]; ++a) {
                            double s = 0.0;
                            for (int64_t j = 0; j < d[k]; ++j)
                                for (int64_t bb = 0; bb < r[k + 1]; ++bb) {
                                    double dp = dP[(p * d[k] + j) * r[k + 1] + bb];
                                    priv[k][core_off(n, d, r, k, a, dig[k], j, bb)] += Pp[p * r[k] + a] * dp;
                                    s += dp * core_at(cores[k], n, d, r, k, a, dig[k], j, bb);
                                }
                            dPprev[p * r[k] + a] = s;
                        }
                    double* tmp = dP; dP = dPprev; dPprev = tmp;
                    rows = prow;
                }
                for (int64_t j = 0; j < d[0]; ++j)
                    for (int64_t bb = 0; bb < r[1]; ++bb)
                        priv[0][core_off(n, d, r, 0, 0, dig[0], j, bb)] += dP[j * r[1] + bb];
            }
        }
#pragma omp critical
        {
            for (int k = 0; k < K; ++k)
                for (int64_t i = 0; i < csize[k]; ++i) core_grads[k][i] += priv[k][i];
        }
        for (int k = 0; k < K; ++k) free(priv[k]);
        free(P_all); free(dP); free(dPprev);
    }
    return bad;
}

/*
 * Brute-force definition of the whole table, no intermediate products:
 *   W[i][j] = sum over (a_1..a_{K-1}) of prod_k G_k[a_{k-1}][i_k][j_k][a_k],   a_0 = a_K = 0,
 * for every row i < prod(n) (padding rows included) and column j < D.  Exponential in K; tiny tables only.
 */
void tt_oracle_dense(int K, const int64_t* n, const int64_t* d, const int64_t* r,
                     const double* const* cores, double* W)
{
    int64_t NN = 1, D = 1;
    for (int k = 0; k < K; ++k) { NN *= n[k]; D *= d[k]; }
    int64_t idig[TT_MAX_K], jdig[TT_MAX_K], a[TT_MAX_K + 1];
    for (int64_t i = 0; i < NN; ++i) {
        int64_t rem = i;
        for (int k = K - 1; k >= 0; --k) { idig[k] = rem % n[k]; rem /= n[k]; }
        for (int64_t j = 0; j < D; ++j) {
            rem = j;
            for (int k = K - 1; k >= 0; --k) { jdig[k] = rem % d[k]; rem /= d[k]; }
            double total = 0.0;
            for (int k = 0; k <= K; ++k) a[k] = 0;
            for (;;) {
                double prod = 1.0;
                for (int k = 0; k < K; ++k)
                    prod *= core_at(cores[k], n, d, r, k, a[k], idig[k], jdig[k], a[k + 1]);
                total += prod;
                int k = K - 1; /* odometer over a_1..a_{K-1} */
                while (k >= 1) {
                    if (++a[k] < r[k]) break;
                    a[k] = 0;
                    --k;
                }
                if (k < 1) break;
            }
            W[i * D + j] = total;
        }
    }
}

/* Plain SGD: G <- G - lr * dG, elementwise. */
void tt_oracle_sgd(double* G, const double* dG, int64_t count, double lr)
{
    for (int64_t i = 0; i < count; ++i) G[i] = G[i] - lr * dG[i];
}
