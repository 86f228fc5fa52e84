/*
 * Memoised fp64 CPU oracle for the Tensor-Train (TT) embedding gather.  TEST INFRASTRUCTURE ONLY.
 *
 * The plain oracle (tt_oracle.c) rebuilds a row for every lookup; at 10^8 lookups that takes hours.  This file
 * computes the same plain definition with two tables keyed by row id and nothing else:
 *   forward   each DISTINCT row of the batch is built once (sequential slice products, Sec. 3.2) and kept; a
 *             bag's output is the sum of the kept rows of its lookups, in lookup order;
 *   backward  the output gradient is first summed per distinct row (dE_u = sum over the lookups of row u of
 *             a_l * grad_out[bag(l)], in lookup order), then the per-lookup backward chain of Sec. 3.2 runs once
 *             per distinct row with dE_u in place of one lookup's gradient.  The chain is linear in that
 *             gradient, so the result is the per-lookup sum exactly (up to fp64 rounding order).
 * There is no prefix sharing, no Eq. 2 regrouping, no blocking: rows are independent of one another.  It shares
 * no code with the CUDA library nor with tt_oracle.c (its own digit split, its own products), so the two
 * oracles check each other: the tests compare them on tiny, medium and sub-sampled full-size inputs.
 *
 * Same data model as tt_oracle.c: core k is G_k[a][i][j][b] (a < r_{k-1}, i < n_k, j < d_k, b < r_k), C-contiguous
 * in that order, fp64; r_0 = r_K = 1; indices int64 of ONE table, offsets int64 [B + 1].
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MEMO_MAX_K 8

typedef struct {
    int K;
    int64_t n[MEMO_MAX_K], d[MEMO_MAX_K], r[MEMO_MAX_K + 1];
    int64_t D;
    int64_t psize[MEMO_MAX_K];   /* doubles in P_k (k 0-based: after core k): d_0 .. d_k rows times r_{k+1} */
    int64_t poff[MEMO_MAX_K];    /* where P_k starts in a scratch block */
    int64_t ptotal;
    int64_t slice_max;           /* largest r_k * d_k * r_{k+1} */
} shape_t;

static void shape_init(shape_t* s, int K, const int64_t* n, const int64_t* d, const int64_t* r)
{
    s->K = K;
    s->D = 1;
    s->ptotal = 0;
    s->slice_max = 1;
    int64_t rows = 1;
    for (int k = 0; k < K; ++k) {
        s->n[k] = n[k]; s->d[k] = d[k]; s->r[k] = r[k];
        rows *= d[k];
        s->psize[k] = rows * r[k + 1];
        s->poff[k] = s->ptotal;
        s->ptotal += s->psize[k];
        if (r[k] * d[k] * r[k + 1] > s->slice_max) s->slice_max = r[k] * d[k] * r[k + 1];
    }
    s->r[K] = r[K];
    s->D = rows;
}

/* Eq. 1, most significant digit first: peel the digits off from the last one. */
static void split_row(const shape_t* s, int64_t g, int64_t* dig)
{
    for (int k = s->K - 1; k >= 0; --k) {
        dig[k] = g % s->n[k];
        g /= s->n[k];
    }
}

/* S[a][j][b] = G_k[a][i][j][b]: the slice digit i selects, copied out so that the products below walk memory in order */
static void take_slice(const shape_t* s, const double* G, int k, int64_t i, double* S)
{
    const int64_t ra = s->r[k], nk = s->n[k], inner = s->d[k] * s->r[k + 1];
    for (int64_t a = 0; a < ra; ++a)
        memcpy(S + a * inner, G + (a * nk + i) * inner, sizeof(double) * (size_t)inner);
}

/* all partial products of one row: P_0 = slice of core 0; P_k[(p, j)][b] = sum_a P_{k-1}[p][a] * S_k[a][j][b] */
static void row_partials(const shape_t* s, const double* const* cores, const int64_t* dig, double* P, double* S)
{
    take_slice(s, cores[0], 0, dig[0], P + s->poff[0]);
    int64_t rows = s->d[0];
    for (int k = 1; k < s->K; ++k) {
        const int64_t ra = s->r[k], inner = s->d[k] * s->r[k + 1];
        const double* Pp = P + s->poff[k - 1];
        double* Pn = P + s->poff[k];
        take_slice(s, cores[k], k, dig[k], S);
        for (int64_t p = 0; p < rows; ++p) {
            double* o = Pn + p * inner;
            for (int64_t x = 0; x < inner; ++x) o[x] = 0.0;
            for (int64_t a = 0; a < ra; ++a) {
                const double pa = Pp[p * ra + a];
                const double* sa = S + a * inner;
                for (int64_t x = 0; x < inner; ++x) o[x] += pa * sa[x];
            }
        }
        rows *= s->d[k];
    }
}

/*
 * Distinct rows of the batch in first-seen order.  slot_of[l] = position of indices[l] in that order, or -1 for an
 * id outside [0, N).  Returns the number of distinct rows; *rows_out (malloc'ed) lists them.  A direct-address
 * table over the row-id domain: N ints.
 */
static int64_t distinct_rows(int64_t N, const int64_t* indices, int64_t L, int32_t* slot_of, int64_t** rows_out, int64_t* bad)
{
    int32_t* where = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
    int64_t* rows = (int64_t*)malloc(sizeof(int64_t) * (size_t)(L > 0 ? L : 1));
    for (int64_t g = 0; g < N; ++g) where[g] = -1;
    int64_t U = 0;
    *bad = 0;
    for (int64_t l = 0; l < L; ++l) {
        const int64_t g = indices[l];
        if (g < 0 || g >= N) { slot_of[l] = -1; ++*bad; continue; }
        if (where[g] < 0) { where[g] = (int32_t)U; rows[U++] = g; }
        slot_of[l] = where[g];
    }
    free(where);
    *rows_out = rows;
    return U;
}

/* pooled forward of ONE table; same arguments and return value as tt_oracle_forward */
int64_t tt_memo_forward(int K, const int64_t* n, const int64_t* d, const int64_t* r, int64_t N,
                        const double* const* cores, const int64_t* indices, const int64_t* offsets,
                        int64_t B, double* out, int64_t out_stride, const double* weights, int mean)
{
    shape_t s;
    shape_init(&s, K, n, d, r);
    const int64_t L = offsets[B], D = s.D;
    int32_t* slot_of = (int32_t*)malloc(sizeof(int32_t) * (size_t)(L > 0 ? L : 1));
    int64_t* rows = NULL;
    int64_t bad = 0;
    const int64_t U = distinct_rows(N, indices, L, slot_of, &rows, &bad);
    double* kept = (double*)malloc(sizeof(double) * (size_t)(U > 0 ? U : 1) * (size_t)D);
#pragma omp parallel
    {
        double* P = (double*)malloc(sizeof(double) * (size_t)s.ptotal);
        double* S = (double*)malloc(sizeof(double) * (size_t)s.slice_max);
        int64_t dig[MEMO_MAX_K];
#pragma omp for schedule(static)
        for (int64_t u = 0; u < U; ++u) {
            split_row(&s, rows[u], dig);
            row_partials(&s, cores, dig, P, S);
            memcpy(kept + u * D, P + s.poff[K - 1], sizeof(double) * (size_t)D);   /* P_K is the row, row-major over (j_1..j_K) */
        }
        free(P);
        free(S);
#pragma omp for schedule(static)
        for (int64_t b = 0; b < B; ++b) {
            double* o = out + b * out_stride;
            for (int64_t j = 0; j < D; ++j) o[j] = 0.0;
            const int64_t len = offsets[b + 1] - offsets[b];
            for (int64_t l = offsets[b]; l < offsets[b + 1]; ++l) {
                if (slot_of[l] < 0) continue;
                double a = weights ? weights[l] : 1.0;
                if (mean) a /= (double)len;
                const double* e = kept + (int64_t)slot_of[l] * D;
                for (int64_t j = 0; j < D; ++j) o[j] += a * e[j];
            }
        }
    }
    free(kept);
    free(rows);
    free(slot_of);
    return bad;
}

/* backward of ONE table; same arguments and return value as tt_oracle_backward (core_grads is accumulated into) */
int64_t tt_memo_backward(int K, const int64_t* n, const int64_t* d, const int64_t* r, int64_t N,
                         const double* const* cores, const int64_t* indices, const int64_t* offsets,
                         int64_t B, const double* grad_out, int64_t grad_stride, double* const* core_grads,
                         const double* weights, int mean)
{
    shape_t s;
    shape_init(&s, K, n, d, r);
    const int64_t L = offsets[B], D = s.D;
    int32_t* slot_of = (int32_t*)malloc(sizeof(int32_t) * (size_t)(L > 0 ? L : 1));
    int64_t* rows = NULL;
    int64_t bad = 0;
    const int64_t U = distinct_rows(N, indices, L, slot_of, &rows, &bad);
    /* lookups of every distinct row, in lookup order: count, prefix sum, fill */
    int64_t* start = (int64_t*)calloc((size_t)U + 2, sizeof(int64_t));
    int64_t* who = (int64_t*)malloc(sizeof(int64_t) * (size_t)(L > 0 ? L : 1));
    int32_t* bag_of = (int32_t*)malloc(sizeof(int32_t) * (size_t)(L > 0 ? L : 1));
    for (int64_t b = 0; b < B; ++b)
        for (int64_t l = offsets[b]; l < offsets[b + 1]; ++l) bag_of[l] = (int32_t)b;
    for (int64_t l = 0; l < L; ++l)
        if (slot_of[l] >= 0) ++start[slot_of[l] + 2];
    for (int64_t u = 0; u < U; ++u) start[u + 2] += start[u + 1];   /* start[u + 1] = first position of row u */
    for (int64_t l = 0; l < L; ++l)
        if (slot_of[l] >= 0) who[start[slot_of[l] + 1]++] = l;      /* afterwards start[u + 1] = end of row u = start of u + 1 */
    /* now row u owns who[start[u] .. start[u + 1]) */
    int64_t csize[MEMO_MAX_K];
    for (int k = 0; k < K; ++k) csize[k] = r[k] * n[k] * d[k] * r[k + 1];
#pragma omp parallel
    {
        double* P = (double*)malloc(sizeof(double) * (size_t)s.ptotal);
        double* S = (double*)malloc(sizeof(double) * (size_t)s.slice_max);
        double* dS = (double*)malloc(sizeof(double) * (size_t)s.slice_max);
        double* dPa = (double*)malloc(sizeof(double) * (size_t)s.ptotal);
        double* dPb = (double*)malloc(sizeof(double) * (size_t)s.ptotal);
        double* priv[MEMO_MAX_K];
        for (int k = 0; k < K; ++k) priv[k] = (double*)calloc((size_t)csize[k], sizeof(double));
        int64_t dig[MEMO_MAX_K];
#pragma omp for schedule(dynamic, 64)
        for (int64_t u = 0; u < U; ++u) {
            /* dE_u: the gradients of the bags that looked row u up, added in lookup order */
            double* dP = dPa;
            double* dPn = dPb;
            for (int64_t j = 0; j < D; ++j) dP[j] = 0.0;
            for (int64_t q = start[u]; q < start[u + 1]; ++q) {
                const int64_t l = who[q], b = bag_of[l];
                double a = weights ? weights[l] : 1.0;
                if (mean) a /= (double)(offsets[b + 1] - offsets[b]);
                const double* go = grad_out + b * grad_stride;
                for (int64_t j = 0; j < D; ++j) dP[j] += a * go[j];
            }
            split_row(&s, rows[u], dig);
            row_partials(&s, cores, dig, P, S);
            /* k = K-1 .. 1:  dG_k[a][i_k][j][b] += sum_p P_{k-1}[p][a] dP_k[(p,j)][b];  dP_{k-1}[p][a] = sum_{j,b} dP_k[(p,j)][b] G_k[a][i_k][j][b] */
            int64_t prow = D;
            for (int k = K - 1; k >= 1; --k) {
                const int64_t ra = r[k], inner = d[k] * r[k + 1], nk = n[k];
                prow /= d[k];
                const double* Pp = P + s.poff[k - 1];
                take_slice(&s, cores[k], k, dig[k], S);
                for (int64_t x = 0; x < ra * inner; ++x) dS[x] = 0.0;
                for (int64_t p = 0; p < prow; ++p) {
                    const double* dp = dP + p * inner;
                    for (int64_t a = 0; a < ra; ++a) {
                        const double pa = Pp[p * ra + a];
                        const double* sa = S + a * inner;
                        double* da = dS + a * inner;
                        double acc = 0.0;
                        for (int64_t x = 0; x < inner; ++x) {
                            da[x] += pa * dp[x];
                            acc += dp[x] * sa[x];
                        }
                        dPn[p * ra + a] = acc;
                    }
                }
                for (int64_t a = 0; a < ra; ++a) {
                    double* g = priv[k] + (a * nk + dig[k]) * inner;
                    for (int64_t x = 0; x < inner; ++x) g[x] += dS[a * inner + x];
                }
                double* tmp = dP; dP = dPn; dPn = tmp;
            }
            {   /* dG_1[0][i_1][j][b] += dP_1[j][b] */
                const int64_t inner = d[0] * r[1];
                double* g = priv[0] + dig[0] * inner;
                for (int64_t x = 0; x < inner; ++x) g[x] += dP[x];
            }
        }
#pragma omp critical
        {
            for (int k = 0; k < K; ++k)
                for (int64_t i = 0; i < csize[k]; ++i) core_grads[k][i] += priv[k][i];
        }
        for (int k = 0; k < K; ++k) free(priv[k]);
        free(P); free(S); free(dS); free(dPa); free(dPb);
    }
    free(bag_of);
    free(who);
    free(start);
    free(rows);
    free(slot_of);
    return bad;
}
