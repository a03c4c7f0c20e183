/*
 * CPU oracle for the Cholesky recurrences.
 *
 * Scalar form (Figure "Representative recurrences", "Cholesky (lower L)"):
 *
 *      L_ii = sqrt( A_ii - sum_{k<i} L_ik^2 )
 *      L_ij = ( A_ij - sum_{k<j} L_ik L_jk ) / L_jj          j < i
 *
 * Tiled form (Section "Simulated Cholesky and Flash Attention", paragraph
 * "Cholesky Recurrence"), A partitioned into b x b tiles, for each panel j:
 *
 *      A_jj^(j) = A_jj - sum_{k<j} SYRK(L_jk)          L_jj = CHOL(A_jj^(j))
 *      A_ij^(j) = A_ij - sum_{k<j} GEMM(L_ik, L_jk)    L_ij = TRSM(A_ij^(j), L_jj)     i > j
 *
 * read as SYRK(X) = X X^T, GEMM(X, Y) = X Y^T, TRSM(S, L_jj) = the solution X
 * of X L_jj^T = S, and CHOL = the scalar form applied inside the tile.
 *
 * THIS IS TEST INFRASTRUCTURE.  A plain, slow evaluator used only to check
 * the GPU library and to report a CPU baseline.  It shares no code, header,
 * table or helper with the CUDA path and must never be called from the
 * product path.
 *
 * A is [n][n] row-major fp32; only entries with i >= j are read (the matrix is
 * symmetric; the upper triangle may hold anything).  L is [n][n] row-major
 * fp64; entries above the diagonal are set to zero.  All arithmetic is fp64
 * (the paper fixes no precision), multiply and add/subtract as separate rounded
 * operations, no reassociation; sqrt and division are the C library's
 * (correctly rounded).  A non-positive pivot is not an error: sqrt of a
 * negative number gives NaN, which then spreads, as the formula says.
 *
 * Order of operations for one entry L[i][j] (j <= i), tile edge b, panel of j = J:
 *   s = A[i][j];  for k = 0 .. J*b-1 increasing (tile by tile): s -= L[i][k]*L[j][k]
 *   then, inside panel J, for k = J*b .. j-1 increasing:       s -= L[i][k]*L[j][k]
 *   L[i][j] = (i == j) ? sqrt(s) : s / L[j][j]
 * The scalar mode is the same chain with one tile covering everything.  The two
 * modes therefore perform the same operations in the same order and agree bit
 * for bit; they differ in how the work is walked (entry by entry along a row /
 * tile by tile with explicit tile buffers), which is what the tests compare.
 *
 * Build:  gcc -O2 -fno-fast-math -ffp-contract=off -shared -fPIC -pthread
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_BAD_ARG 1
#define ORC_NO_MEM 2

static int64_t imin(int64_t a, int64_t b) { return a < b ? a : b; }

/* ------------------------------------------------------------------ */
/* scalar form: row by row, entry by entry                             */
/* ------------------------------------------------------------------ */
static int chol_scalar(int64_t n, const float *A, double *L) {
    for (int64_t i = 0; i < n; ++i) {
        for (int64_t j = 0; j <= i; ++j) {
            double s = (double)A[i * n + j];
            for (int64_t k = 0; k < j; ++k) s = s - L[i * n + k] * L[j * n + k];
            if (i == j) L[i * n + i] = sqrt(s);           /* L_ii = sqrt(A_ii - sum L_ik^2) */
            else L[i * n + j] = s / L[j * n + j];         /* L_ij = (A_ij - sum L_ik L_jk) / L_jj */
        }
        for (int64_t j = i + 1; j < n; ++j) L[i * n + j] = 0.0;
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* tile operations on explicit tile buffers S[rows][cols]              */
/* ------------------------------------------------------------------ */

/* S <- S - X Y^T : X is rows x kk at L[r0..][k0..], Y is cols x kk at L[c0..][k0..]; SYRK when r0 == c0 */
static void tile_update(const double *L, int64_t n, int64_t r0, int64_t rows, int64_t c0, int64_t cols, int64_t k0, int64_t kk,
                        double *S, int64_t lds) {
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            double s = S[r * lds + c];
            for (int64_t k = 0; k < kk; ++k) s = s - L[(r0 + r) * n + k0 + k] * L[(c0 + c) * n + k0 + k];
            S[r * lds + c] = s;
        }
}

/* CHOL: the scalar recurrence inside a tile, in place on the lower triangle of S[rows][rows] */
static void tile_chol(double *S, int64_t rows, int64_t lds) {
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j <= i; ++j) {
            double s = S[i * lds + j];
            for (int64_t k = 0; k < j; ++k) s = s - S[i * lds + k] * S[j * lds + k];
            S[i * lds + j] = (i == j) ? sqrt(s) : s / S[j * lds + j];
        }
}

/* TRSM: X L_jj^T = S, row by row, in place; Ljj[cols][cols] lower triangular */
static void tile_trsm_right(const double *Ljj, int64_t ldl, double *S, int64_t rows, int64_t cols, int64_t lds) {
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            double s = S[r * lds + c];
            for (int64_t k = 0; k < c; ++k) s = s - S[r * lds + k] * Ljj[c * ldl + k];
            S[r * lds + c] = s / Ljj[c * ldl + c];
        }
}

/* ------------------------------------------------------------------ */
/* tiled form: panel by panel                                          */
/* ------------------------------------------------------------------ */
typedef struct {
    int64_t n, b, J, i_first, i_step, tiles;
    const float *A;
    double *L;
    int rc;
} panel_job_t;

/* one tile (I, J), I >= J: gather A_IJ, subtract the updates of panels k < J in increasing k, then CHOL or TRSM */
static int do_tile(int64_t n, int64_t b, int64_t I, int64_t J, const float *A, double *L) {
    const int64_t r0 = I * b, rows = imin(b, n - r0), c0 = J * b, cols = imin(b, n - c0);
    double *S = (double *)malloc(sizeof(double) * (size_t)(rows * cols));
    if (!S) return ORC_NO_MEM;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c)
            S[r * cols + c] = (r0 + r >= c0 + c) ? (double)A[(r0 + r) * n + c0 + c] : 0.0;   /* lower triangle of A only */
    for (int64_t k = 0; k < J; ++k)   /* SYRK(L_Jk) on the diagonal, GEMM(L_Ik, L_Jk) below it */
        tile_update(L, n, r0, rows, c0, cols, k * b, b, S, cols);
    if (I == J) {
        tile_chol(S, rows, cols);
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t c = 0; c < cols; ++c) L[(r0 + r) * n + c0 + c] = (c <= r) ? S[r * cols + c] : 0.0;
    } else {
        tile_trsm_right(L + c0 * n + c0, n, S, rows, cols, cols);
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t c = 0; c < cols; ++c) L[(r0 + r) * n + c0 + c] = S[r * cols + c];
    }
    free(S);
    return ORC_OK;
}

static void *panel_worker(void *p) {
    panel_job_t *jb = (panel_job_t *)p;
    for (int64_t I = jb->i_first; I < jb->tiles; I += jb->i_step) {
        const int rc = do_tile(jb->n, jb->b, I, jb->J, jb->A, jb->L);
        if (rc) jb->rc = rc;
    }
    return NULL;
}

static int chol_tiled(int64_t n, int64_t b, const float *A, double *L, int nthreads) {
    const int64_t tiles = (n + b - 1) / b;
    for (int64_t i = 0; i < n; ++i)
        for (int64_t j = i + 1; j < n; ++j) L[i * n + j] = 0.0;
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    panel_job_t *jobs = (panel_job_t *)malloc(sizeof(panel_job_t) * (size_t)nthreads);
    if (!th || !jobs) { free(th); free(jobs); return ORC_NO_MEM; }
    int rc = ORC_OK;
    for (int64_t J = 0; J < tiles && rc == ORC_OK; ++J) {
        rc = do_tile(n, b, J, J, A, L);   /* the diagonal tile first: every tile below needs L_JJ */
        if (rc) break;
        /* the tiles below the diagonal of panel J are independent of one another */
        for (int t = 0; t < nthreads; ++t) {
            jobs[t].n = n; jobs[t].b = b; jobs[t].J = J; jobs[t].i_first = J + 1 + t; jobs[t].i_step = nthreads;
            jobs[t].tiles = tiles; jobs[t].A = A; jobs[t].L = L; jobs[t].rc = ORC_OK;
            if (nthreads == 1) panel_worker(&jobs[t]);
            else pthread_create(&th[t], NULL, panel_worker, &jobs[t]);
        }
        for (int t = 0; t < nthreads; ++t) {
            if (nthreads > 1) pthread_join(th[t], NULL);
            if (jobs[t].rc) rc = jobs[t].rc;
        }
    }
    free(th);
    free(jobs);
    return rc;
}

/* mode 0: scalar form; mode 1: tiled form with tile edge b */
int cyc_oracle_cholesky(int mode, int64_t n, int64_t b, const float *A, double *L, int nthreads) {
    if (n < 1 || !A || !L || (mode != 0 && mode != 1)) return ORC_BAD_ARG;
    if (mode == 0) return chol_scalar(n, A, L);
    if (b < 1) return ORC_BAD_ARG;
    if (nthreads < 1) nthreads = 1;
    return chol_tiled(n, b, A, L, nthreads);
}

/*
 * Residual of a candidate factor Lc (fp32, lower triangle read) for the listed rows:
 *   R[q][j] = A[i][j] - sum_{k<=j} Lc[i][k] Lc[j][k],   Sc[q][j] = sum_{k<=j} |Lc[i][k]| |Lc[j][k]|,   i = rows[q], j <= i
 * in fp64; entries with j > i are set to zero.
 */
int cyc_oracle_cholesky_residual(int64_t n, const float *A, const float *Lc, const int64_t *rows, int64_t nrows, double *R,
                                 double *Sc) {
    if (n < 1 || !A || !Lc || !rows || !R || !Sc) return ORC_BAD_ARG;
    for (int64_t q = 0; q < nrows; ++q) {
        const int64_t i = rows[q];
        if (i < 0 || i >= n) return ORC_BAD_ARG;
        for (int64_t j = 0; j < n; ++j) {
            double acc = 0.0, sc = 0.0;
            if (j <= i) {
                for (int64_t k = 0; k <= j; ++k) {
                    const double p = (double)Lc[i * n + k] * (double)Lc[j * n + k];
                    acc = acc + p;
                    sc = sc + fabs(p);
                }
                R[q * n + j] = (double)A[i * n + j] - acc;
                Sc[q * n + j] = sc;
            } else {
                R[q * n + j] = 0.0;
                Sc[q * n + j] = 0.0;
            }
        }
    }
    return ORC_OK;
}
