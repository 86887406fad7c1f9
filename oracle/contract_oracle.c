/*
 * CPU oracle for sparse tensor-network contractions.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain reference that the CUDA library is checked against.  Only the
 * test-suite, the smoke check and the benchmark's CPU-baseline leg may call it; no product
 * code path links or loads it.  It shares no code, header, table or helper with the CUDA path.
 *
 * What it computes (paper Sec. 2.1, "Tensor contractions" and "Tensor networks"): a network
 * R = T1 x T2 x ... x Tn assigns to every tuple of external indices the sum, over all values of
 * the contraction indices, of the product of the operands, where a sparse operand contributes
 * only at its stored coordinates.  The direct evaluation is the single loop nest of Fig. 2(b):
 * one loop per index, one multiply-accumulate statement.  Here that loop nest is written over
 * the COO nonzeros of the sparse operand(s) and the full range of the dense indices.  No
 * contraction tree, no intermediate tensor and no CSF structure is used: the method under
 * test reaches exactly this value (up to rounding order), so the definition is the oracle.
 *
 * Every function returns two arrays in double precision: S, the sum of the terms, and A, the
 * sum of their absolute values.  Parity tests accept |gpu - S| <= tol * A per element.
 * Inputs given in single precision are widened exactly by the caller.
 *
 * Threads: nonzeros are first bucketed by their output row i (a counting pass), then rows are
 * distributed over OpenMP threads, so no two threads touch the same output row.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Bucket nonzero ids by row: start[r]..start[r+1] indexes `ids`, ids inside a row keep input order. */
static int bucket_by_row(int64_t nnz, const int32_t *row, int64_t n_rows, int64_t **start_out, int64_t **ids_out) {
    int64_t *start = (int64_t *)calloc((size_t)n_rows + 1, sizeof(int64_t));
    int64_t *ids = (int64_t *)malloc((size_t)(nnz > 0 ? nnz : 1) * sizeof(int64_t));
    int64_t *fill = (int64_t *)malloc((size_t)(n_rows > 0 ? n_rows : 1) * sizeof(int64_t));
    if (!start || !ids || !fill) { free(start); free(ids); free(fill); return -1; }
    for (int64_t e = 0; e < nnz; ++e) {
        if (row[e] < 0 || row[e] >= n_rows) { free(start); free(ids); free(fill); return -2; }
        start[row[e] + 1]++;
    }
    for (int64_t r = 0; r < n_rows; ++r) start[r + 1] += start[r];
    for (int64_t r = 0; r < n_rows; ++r) fill[r] = start[r];
    for (int64_t e = 0; e < nnz; ++e) ids[fill[row[e]]++] = e;
    free(fill);
    *start_out = start;
    *ids_out = ids;
    return 0;
}

/*
 * TTMc, order 3 (paper Sec. 5.3):  Y[i,a,b] = sum_{j,k} X[i,j,k] * U[j,a] * V[k,b].
 * U is Nj x Ra, V is Nk x Rb, row-major.  S and A are Ni x Ra x Rb, row-major, overwritten.
 */
int oracle_ttmc3(int64_t nnz, const int32_t *ci, const int32_t *cj, const int32_t *ck, const double *x,
                 const double *U, int64_t Ra, const double *V, int64_t Rb, int64_t Ni,
                 double *S, double *A) {
    int64_t *start, *ids;
    int rc = bucket_by_row(nnz, ci, Ni, &start, &ids);
    if (rc) return rc;
    memset(S, 0, (size_t)(Ni * Ra * Rb) * sizeof(double));
    memset(A, 0, (size_t)(Ni * Ra * Rb) * sizeof(double));
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < Ni; ++i) {
        double *Si = S + i * Ra * Rb, *Ai = A + i * Ra * Rb;
        for (int64_t q = start[i]; q < start[i + 1]; ++q) {
            int64_t e = ids[q];
            const double *u = U + (int64_t)cj[e] * Ra;
            const double *v = V + (int64_t)ck[e] * Rb;
            for (int64_t a = 0; a < Ra; ++a)
                for (int64_t b = 0; b < Rb; ++b) {
                    double term = x[e] * u[a] * v[b];
                    Si[a * Rb + b] += term;
                    Ai[a * Rb + b] += fabs(term);
                }
        }
    }
    free(start); free(ids);
    return 0;
}

/*
 * TTMc, order 4:  Y[i,a,b,c] = sum_{j,k,l} X[i,j,k,l] * U[j,a] * V[k,b] * W[l,c].
 */
int oracle_ttmc4(int64_t nnz, const int32_t *ci, const int32_t *cj, const int32_t *ck, const int32_t *cl,
                 const double *x, const double *U, int64_t Ra, const double *V, int64_t Rb,
                 const double *W, int64_t Rc, int64_t Ni, double *S, double *A) {
    int64_t *start, *ids;
    int rc = bucket_by_row(nnz, ci, Ni, &start, &ids);
    if (rc) return rc;
    int64_t slab = Ra * Rb * Rc;
    memset(S, 0, (size_t)(Ni * slab) * sizeof(double));
    memset(A, 0, (size_t)(Ni * slab) * sizeof(double));
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < Ni; ++i) {
        double *Si = S + i * slab, *Ai = A + i * slab;
        for (int64_t q = start[i]; q < start[i + 1]; ++q) {
            int64_t e = ids[q];
            const double *u = U + (int64_t)cj[e] * Ra;
            const double *v = V + (int64_t)ck[e] * Rb;
            const double *w = W + (int64_t)cl[e] * Rc;
            for (int64_t a = 0; a < Ra; ++a)
                for (int64_t b = 0; b < Rb; ++b)
                    for (int64_t c = 0; c < Rc; ++c) {
                        double term = x[e] * u[a] * v[b] * w[c];
                        Si[(a * Rb + b) * Rc + c] += term;
                        Ai[(a * Rb + b) * Rc + c] += fabs(term);
                    }
        }
    }
    free(start); free(ids);
    return 0;
}

/*
 * MTTKRP, order 3 (paper Sec. 5.2):  A'[i,r] = sum_{j,k} X[i,j,k] * B[j,r] * C[k,r].
 */
int oracle_mttkrp3(int64_t nnz, const int32_t *ci, const int32_t *cj, const int32_t *ck, const double *x,
                   const double *B, const double *C, int64_t R, int64_t Ni, double *S, double *A) {
    int64_t *start, *ids;
    int rc = bucket_by_row(nnz, ci, Ni, &start, &ids);
    if (rc) return rc;
    memset(S, 0, (size_t)(Ni * R) * sizeof(double));
    memset(A, 0, (size_t)(Ni * R) * sizeof(double));
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < Ni; ++i) {
        for (int64_t q = start[i]; q < start[i + 1]; ++q) {
            int64_t e = ids[q];
            const double *b = B + (int64_t)cj[e] * R;
            const double *c = C + (int64_t)ck[e] * R;
            for (int64_t r = 0; r < R; ++r) {
                double term = x[e] * b[r] * c[r];
                S[i * R + r] += term;
                A[i * R + r] += fabs(term);
            }
        }
    }
    free(start); free(ids);
    return 0;
}

/* Neumaier's compensated addition: (sum, comp) += term; the result is sum + comp. */
static inline void comp_add(double *sum, double *comp, double term) {
    double t = *sum + term;
    if (fabs(*sum) >= fabs(term)) *comp += (*sum - t) + term;
    else                          *comp += (term - t) + *sum;
    *sum = t;
}

/*
 * Two-contraction network (paper Sec. 1):  Z[i,m] = sum_{j,k,l} U[i,j,k] * V[j,l] * W[k,l,m].
 * U and W are sparse (COO), V is dense Nj x Nl row-major.  A term exists for every pair of a
 * U nonzero (i,j,k) and a W nonzero (k',l,m) with k' = k.  W's nonzeros are bucketed by k so the
 * matching pairs can be enumerated; the sum itself is the plain triple product.
 * With ~1e4..1e5 terms per output a naive double sum could err by a few 1e-12 * A, which is the
 * test tolerance, so the accumulation is compensated.
 */
int oracle_network(int64_t nnzU, const int32_t *ui, const int32_t *uj, const int32_t *uk, const double *uval,
                   const double *V, int64_t Nl,
                   int64_t nnzW, const int32_t *wk, const int32_t *wl, const int32_t *wm, const double *wval,
                   int64_t Ni, int64_t Nk, int64_t Nm, double *S, double *A) {
    int64_t *ustart, *uids, *wstart, *wids;
    int rc = bucket_by_row(nnzU, ui, Ni, &ustart, &uids);
    if (rc) return rc;
    rc = bucket_by_row(nnzW, wk, Nk, &wstart, &wids);
    if (rc) { free(ustart); free(uids); return rc; }
    for (int64_t e = 0; e < nnzU; ++e)
        if (uk[e] < 0 || uk[e] >= Nk) { free(ustart); free(uids); free(wstart); free(wids); return -2; }
    memset(S, 0, (size_t)(Ni * Nm) * sizeof(double));
    memset(A, 0, (size_t)(Ni * Nm) * sizeof(double));
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < Ni; ++i) {
        if (ustart[i] == ustart[i + 1]) continue;
        double *cs = (double *)calloc((size_t)Nm, sizeof(double));
        double *ca = (double *)calloc((size_t)Nm, sizeof(double));
        if (!cs || !ca) { failed = 1; free(cs); free(ca); continue; }
        double *Si = S + i * Nm, *Ai = A + i * Nm;
        for (int64_t q = ustart[i]; q < ustart[i + 1]; ++q) {
            int64_t e = uids[q];
            const double *vrow = V + (int64_t)uj[e] * Nl;
            int64_t k = uk[e];
            for (int64_t p = wstart[k]; p < wstart[k + 1]; ++p) {
                int64_t f = wids[p];
                double term = uval[e] * vrow[wl[f]] * wval[f];
                comp_add(&Si[wm[f]], &cs[wm[f]], term);
                comp_add(&Ai[wm[f]], &ca[wm[f]], fabs(term));
            }
        }
        for (int64_t m = 0; m < Nm; ++m) { Si[m] += cs[m]; Ai[m] += ca[m]; }
        free(cs); free(ca);
    }
    free(ustart); free(uids); free(wstart); free(wids);
    return failed ? -1 : 0;
}
