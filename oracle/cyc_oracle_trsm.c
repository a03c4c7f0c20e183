/*
 * CPU oracle for the block lower-triangular solve  L X = B
 *
 *      X_i = TRSM( L_ii ,  B_i - sum_{j<i} GEMM(L_ij, X_j) )
 *
 * (Section "Multiple Iteration Spaces"; recurrences of Figure
 * "deps-tri-solve": a triangular space of streamed GEMM updates and a
 * diagonal space of small triangular solves, joined by the interface maps
 * Phi_1 and Phi_2.)
 *
 * THIS IS TEST INFRASTRUCTURE.  A plain, slow evaluator used only to check
 * the GPU library and to report a CPU baseline.  It shares no code, header,
 * table or helper with the CUDA path and must never be called from the
 * product path.
 *
 * L is [n][n] row-major fp32; only i >= j is read.  B is [n][m] row-major
 * fp32 (m right-hand sides), X is [n][m] row-major fp64.  Tiles are T x T
 * (T x m for X and B); the last tile may be ragged.  All arithmetic is fp64
 * (the paper does not fix a precision), multiply and add/subtract as
 * separate rounded operations, no reassociation.
 *
 * Modes
 *   literal    every point of the two iteration spaces holds its own values:
 *              (i,j)^tri_Xb is received from (i-1,j)^tri, or from the
 *              diagonal point (j,j) when i = j+1 (Phi_2); (i,j)^tri_Xa is
 *              received from (i,j-1)^tri (zero at j = 0), updated by the tile
 *              product and forwarded along j; the diagonal point (ii,ii)
 *              receives the end-of-row accumulator (Phi_1) and solves.  The
 *              copy invariant (i,j)_Xb == X_j is asserted.  Small sizes only.
 *   collapsed  reads X_j in place (justified by the copy invariant) and keeps
 *              one accumulator per row; same order of operations; columns of
 *              B are independent and are split over threads.
 *
 * Order of operations for one entry X[r][c], r in block row i:
 *   xa = 0;  for j = 0..i-1, for k in block j increasing:  xa += L[r][k]*X[k][c]
 *   s  = B[r][c] - xa;  for k in block i, k < r increasing:  s -= L[r][k]*X[k][c]
 *   X[r][c] = s / L[r][r]
 *
 * Build:  gcc -O2 -fno-fast-math -ffp-contract=off -shared -fPIC -pthread
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORT_OK 0
#define ORT_BAD_ARG 1
#define ORT_NO_MEM 2
#define ORT_COPY_INVARIANT 3 /* (i,j)_Xb != X_j */

static int64_t imin(int64_t a, int64_t b) { return a < b ? a : b; }

/* ------------------------------------------------------------------ */
/* tile operations, columns [c0,c1) of the right-hand sides            */
/* ------------------------------------------------------------------ */

/* Xa <- Xa + GEMM(L_ij, Xb):  Xa is [rows_i][w], Xb is [rows_j][w]    */
static void tile_gemm(const float *L, int64_t n, int64_t r0, int64_t rows_i, int64_t k0, int64_t rows_j, const double *Xb,
                      double *Xa, int64_t w) {
    for (int64_t r = 0; r < rows_i; ++r)
        for (int64_t k = 0; k < rows_j; ++k) {
            double l = (double)L[(r0 + r) * n + (k0 + k)];
            for (int64_t c = 0; c < w; ++c) {
                double p = l * Xb[k * w + c];
                Xa[r * w + c] = Xa[r * w + c] + p;
            }
        }
}

/* X <- TRSM(L_ii, Bi - Xa): forward substitution inside the tile      */
static void tile_trsm(const float *L, int64_t n, int64_t r0, int64_t rows, const double *Bi_minus_Xa, double *X, int64_t w) {
    for (int64_t r = 0; r < rows; ++r) {
        double d = (double)L[(r0 + r) * n + (r0 + r)];
        for (int64_t c = 0; c < w; ++c) {
            double s = Bi_minus_Xa[r * w + c];
            for (int64_t k = 0; k < r; ++k) {
                double p = (double)L[(r0 + r) * n + (r0 + k)] * X[k * w + c];
                s = s - p;
            }
            X[r * w + c] = s / d;
        }
    }
}

/* ------------------------------------------------------------------ */
/* literal: every point of the two spaces holds its own copies         */
/* ------------------------------------------------------------------ */
static int trsm_literal(int64_t n, int64_t m, int64_t T, const float *L, const float *B, double *X) {
    int64_t nb = (n + T - 1) / T;
    size_t tile = (size_t)T * (size_t)m;
    /* Xb[i*nb+j], Xa[i*nb+j] for tri points i > j; Xd[ii] for diagonal points */
    double **Xb = (double **)calloc((size_t)(nb * nb), sizeof(double *));
    double **Xa = (double **)calloc((size_t)(nb * nb), sizeof(double *));
    double **Xd = (double **)calloc((size_t)nb, sizeof(double *));
    double *rhs = (double *)malloc(sizeof(double) * tile);
    int rc = ORT_OK;
    if (!Xb || !Xa || !Xd || !rhs) rc = ORT_NO_MEM;
    for (int64_t i = 0; i < nb && !rc; ++i) {
        int64_t r0 = i * T, rows_i = imin(T, n - r0);
        for (int64_t j = 0; j < i && !rc; ++j) { /* triangular space, i > j */
            int64_t k0 = j * T, rows_j = imin(T, n - k0);
            double *xb = (double *)malloc(sizeof(double) * tile), *xa = (double *)malloc(sizeof(double) * tile);
            if (!xb || !xa) { free(xb); free(xa); rc = ORT_NO_MEM; break; }
            Xb[i * nb + j] = xb;
            Xa[i * nb + j] = xa;
            /* vertical broadcast in column j; the first point below the diagonal is seeded by (j,j)^diag (Phi_2) */
            const double *from = (i == j + 1) ? Xd[j] : Xb[(i - 1) * nb + j];
            memcpy(xb, from, sizeof(double) * (size_t)rows_j * (size_t)m);
            for (int64_t e = 0; e < rows_j * m; ++e)
                if (!(xb[e] == Xd[j][e]) && !(xb[e] != xb[e] && Xd[j][e] != Xd[j][e])) rc = ORT_COPY_INVARIANT;
            /* accumulator received from the west neighbour, zero at the west boundary */
            if (j == 0) for (int64_t e = 0; e < rows_i * m; ++e) xa[e] = 0.0;
            else memcpy(xa, Xa[i * nb + (j - 1)], sizeof(double) * (size_t)rows_i * (size_t)m);
            tile_gemm(L, n, r0, rows_i, k0, rows_j, xb, xa, m);
        }
        if (rc) break;
        /* diagonal space: read the end of row i of the triangular space (Phi_1), solve, publish */
        double *xd = (double *)malloc(sizeof(double) * tile);
        if (!xd) { rc = ORT_NO_MEM; break; }
        Xd[i] = xd;
        for (int64_t r = 0; r < rows_i; ++r)
            for (int64_t c = 0; c < m; ++c) {
                double xa = (i == 0) ? 0.0 : Xa[i * nb + (i - 1)][r * m + c];
                rhs[r * m + c] = (double)B[(r0 + r) * m + c] - xa;
            }
        tile_trsm(L, n, r0, rows_i, rhs, xd, m);
        memcpy(X + r0 * m, xd, sizeof(double) * (size_t)rows_i * (size_t)m);
    }
    if (Xb) for (int64_t e = 0; e < nb * nb; ++e) free(Xb[e]);
    if (Xa) for (int64_t e = 0; e < nb * nb; ++e) free(Xa[e]);
    if (Xd) for (int64_t e = 0; e < nb; ++e) free(Xd[e]);
    free(Xb); free(Xa); free(Xd); free(rhs);
    return rc;
}

/* ------------------------------------------------------------------ */
/* collapsed: one accumulator per row, X read in place                 */
/* ------------------------------------------------------------------ */
typedef struct {
    int64_t n, m, T, c0, c1;
    const float *L, *B;
    double *X;
    int rc;
} trsm_job;

static void *trsm_collapsed_worker(void *p) {
    trsm_job *jb = (trsm_job *)p;
    int64_t n = jb->n, m = jb->m, T = jb->T, c0 = jb->c0, w = jb->c1 - jb->c0;
    int64_t nb = (n + T - 1) / T;
    double *xa = (double *)malloc(sizeof(double) * (size_t)w);
    if (!xa) { jb->rc = ORT_NO_MEM; return NULL; }
    for (int64_t i = 0; i < nb; ++i) {
        int64_t r0 = i * T, r1 = imin(n, r0 + T);
        for (int64_t r = r0; r < r1; ++r) {
            const float *Lr = jb->L + r * n;
            double *Xr = jb->X + r * m + c0;
            for (int64_t c = 0; c < w; ++c) xa[c] = 0.0;
            for (int64_t k = 0; k < r0; ++k) { /* blocks j = 0..i-1, k increasing */
                double l = (double)Lr[k];
                const double *Xk = jb->X + k * m + c0;
                for (int64_t c = 0; c < w; ++c) {
                    double pr = l * Xk[c];
                    xa[c] = xa[c] + pr;
                }
            }
            for (int64_t c = 0; c < w; ++c) xa[c] = (double)jb->B[r * m + c0 + c] - xa[c]; /* B_i - Xa */
            for (int64_t k = r0; k < r; ++k) { /* inside the diagonal tile */
                double l = (double)Lr[k];
                const double *Xk = jb->X + k * m + c0;
                for (int64_t c = 0; c < w; ++c) {
                    double pr = l * Xk[c];
                    xa[c] = xa[c] - pr;
                }
            }
            double d = (double)Lr[r];
            for (int64_t c = 0; c < w; ++c) Xr[c] = xa[c] / d;
        }
    }
    free(xa);
    jb->rc = ORT_OK;
    return NULL;
}

static int trsm_collapsed(int64_t n, int64_t m, int64_t T, const float *L, const float *B, double *X, int nthreads) {
    if (nthreads > m) nthreads = (int)m;
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    trsm_job *jobs = (trsm_job *)malloc(sizeof(trsm_job) * (size_t)nthreads);
    if (!th || !jobs) { free(th); free(jobs); return ORT_NO_MEM; }
    for (int t = 0; t < nthreads; ++t) {
        trsm_job jb = {n, m, T, m * t / nthreads, m * (t + 1) / nthreads, L, B, X, ORT_OK};
        jobs[t] = jb;
        if (nthreads == 1) trsm_collapsed_worker(&jobs[t]);
        else pthread_create(&th[t], NULL, trsm_collapsed_worker, &jobs[t]);
    }
    int rc = ORT_OK;
    for (int t = 0; t < nthreads; ++t) {
        if (nthreads > 1) pthread_join(th[t], NULL);
        if (jobs[t].rc) rc = jobs[t].rc;
    }
    free(th); free(jobs);
    return rc;
}

/* mode 0 = literal, 1 = collapsed */
int cyc_oracle_block_trsm(int mode, int64_t n, int64_t m, int64_t T, const float *L, const float *B, double *X, int nthreads) {
    if (n <= 0 || m <= 0 || T <= 0 || !L || !B || !X || nthreads < 1) return ORT_BAD_ARG;
    if (mode == 0) return trsm_literal(n, m, T, L, B, X);
    if (mode == 1) return trsm_collapsed(n, m, T, L, B, X, nthreads);
    return ORT_BAD_ARG;
}

/* For the tolerance checks, in fp64, for the columns listed in cols[ncols] of a candidate solution Xc ([n][m] fp32):
 *   R[r][q] = B[r][c] - sum_{k<=r} L[r][k] Xc[k][c]          the residual
 *   S[r][q] = |B[r][c]| + sum_{k<=r} |L[r][k]| |Xc[k][c]|     its scale                                   */
int cyc_oracle_trsm_residual(int64_t n, int64_t m, const float *L, const float *B, const float *Xc, const int64_t *cols,
                             int64_t ncols, double *R, double *S) {
    if (n <= 0 || m <= 0 || !L || !B || !Xc || !cols || ncols <= 0 || !R || !S) return ORT_BAD_ARG;
    for (int64_t q = 0; q < ncols; ++q)
        if (cols[q] < 0 || cols[q] >= m) return ORT_BAD_ARG;
    for (int64_t r = 0; r < n; ++r)
        for (int64_t q = 0; q < ncols; ++q) {
            int64_t c = cols[q];
            double acc = 0.0, s = fabs((double)B[r * m + c]);
            for (int64_t k = 0; k <= r; ++k) {
                double l = (double)L[r * n + k], x = (double)Xc[k * m + c];
                acc += l * x;
                s += fabs(l) * fabs(x);
            }
            R[r * ncols + q] = (double)B[r * m + c] - acc;
            S[r * ncols + q] = s;
        }
    return ORT_OK;
}
