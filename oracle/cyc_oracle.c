/*
 * CPU oracle for the weight-stationary systolic matrix-multiply recurrence
 *
 *      [i,k]_C <- [i,k-1]_C + [i,k]_W * [i,k]_B          (Section "Space-time
 *      Mappings of Dataflow Recurrences", weight-stationary program)
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, literal evaluator used
 * only to check the GPU library and to report a CPU baseline.  It shares no
 * code, header, table or helper with the CUDA path and must never be called
 * from the product path.
 *
 * Modes
 *   literal    every cell (i,k) runs the per-cell program of Figure "perPE":
 *              load W once, then for each time step j receive/inject B,
 *              receive/zero the partial sum, multiply-accumulate, send B south,
 *              send C east or export C_ij.  Sends and receives go through
 *              explicit one-slot channels so a missing or duplicate send is an
 *              error, and the copy invariant (i,j,k)_B == B_kj is asserted.
 *   wavefront  the same cells driven by a global clock with unit link latency;
 *              cell (i,k) handles time step j at tick t = i + j + k
 *              (Section "Timing"), operands must have been produced at t-1.
 *   os_cannon  the output-stationary program of the same section (i,j in
 *              space, k in time) -- a different schedule of the same base
 *              recurrence C_ij = sum_k A_ik B_kj.
 *   collapsed  reads B_kj directly (justified by the copy invariant) and
 *              keeps the increasing-k order of every C_ij; loop order i,k,j;
 *              rows split over threads.  Used for the large configurations.
 *   points     the explicit-reduction recurrence (i,j,k)_C <- (i,j,k-1)_C +
 *              A_ik B_kj, (i,j,0)_C <- 0 (Section "Explicit Reduction
 *              Dimensions") for single outputs (i,j).
 *
 * Arithmetic.  dtype 0: fp32 in, fp32 accumulate.  dtype 1: bf16 in (widened
 * exactly to fp32), fp32 accumulate.  dtype 2: int8 in (sign-extended), int32
 * accumulate.  Round-to-nearest-even.  `fma` = 0 evaluates the multiply and
 * the add as two rounded operations (the statement as printed); `fma` = 1
 * evaluates them as one fused multiply-add (one rounding).  The paper does
 * not say which; both are offered.  The fp rounding variant is therefore
 * "parity unpinned" by the paper; everything else is pinned by the tests.
 *
 * Index base.  Cells are k = 0 .. K-1 and cell k = 0 computes 0 + W*B as the
 * boxes (.,0) of Figure "perPE" show.
 *
 * Build:  gcc -O2 -fno-fast-math -ffp-contract=off -shared -fPIC -pthread
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define CYC_ORACLE_F32 0
#define CYC_ORACLE_BF16_F32 1
#define CYC_ORACLE_I8_I32 2

/* error codes returned by the walkers */
#define ORC_OK 0
#define ORC_BAD_ARG 1
#define ORC_NO_MEM 2
#define ORC_COPY_INVARIANT 3 /* (i,j,k)_B != B_kj */
#define ORC_CHANNEL 4        /* recv without send, or send into a full slot */
#define ORC_TIMING 5         /* operand not produced at tick t-1 */

/* ------------------------------------------------------------------ */
/* element access: widen the stored type to the arithmetic type        */
/* ------------------------------------------------------------------ */

static float bf16_to_f32(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16; /* bf16 is the top half of an fp32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* widen an [rows][cols] operand (row stride rs, column stride cs, in
 * elements) to a dense row-major array of the arithmetic type */
static float *widen_f(int dtype, const void *src, int64_t rows, int64_t cols, int64_t rs, int64_t cs) {
    float *dst = (float *)malloc(sizeof(float) * (size_t)rows * (size_t)cols);
    if (!dst) return NULL;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            int64_t at = r * rs + c * cs;
            dst[r * cols + c] = (dtype == CYC_ORACLE_F32) ? ((const float *)src)[at] : bf16_to_f32(((const uint16_t *)src)[at]);
        }
    return dst;
}

static int32_t *widen_i(const void *src, int64_t rows, int64_t cols, int64_t rs, int64_t cs) {
    int32_t *dst = (int32_t *)malloc(sizeof(int32_t) * (size_t)rows * (size_t)cols);
    if (!dst) return NULL;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) dst[r * cols + c] = (int32_t)((const int8_t *)src)[r * rs + c * cs];
    return dst;
}

/* the cell's arithmetic statement  c_out = c_in + w * b  */
static inline float mac_f(float cin, float w, float b, int fma) {
    if (fma) return fmaf(w, b, cin); /* one rounding */
    float p = w * b;                 /* two roundings (no contraction: -ffp-contract=off) */
    return cin + p;
}
static inline int32_t mac_i(int32_t cin, int32_t w, int32_t b) { return cin + w * b; }

/* ------------------------------------------------------------------ */
/* statement counters for the nine per-cell programs                   */
/* ------------------------------------------------------------------ */
/* cell type = 3*row_class + col_class ; row_class 0: i==0, 1: interior, 2: i==i_end (and i!=0)
 *                                       col_class 0: k==0, 1: interior, 2: k==k_end (and k!=0)
 * (a 1-row grid is classed as row 0, a 1-column grid as column 0)
 * counters per cell type, in this order:                                   */
enum { ST_LOAD_W = 0, ST_INJECT_B, ST_RECV_B, ST_ZERO_C, ST_RECV_C, ST_MAC, ST_SEND_B, ST_SEND_C, ST_EXPORT_C, ST_COUNT };

static int cell_type(int64_t i, int64_t k, int64_t M, int64_t K) {
    int rc = (i == 0) ? 0 : (i == M - 1 ? 2 : 1);
    int cc = (k == 0) ? 0 : (k == K - 1 ? 2 : 1);
    return 3 * rc + cc;
}

/* ------------------------------------------------------------------ */
/* the walkers, written once per arithmetic type                       */
/* ------------------------------------------------------------------ */
#define T float
#define SUF(x) x##_f
#define MAC(cin, w, b) mac_f((cin), (w), (b), fma)
#include "cyc_oracle_walkers.inc"
#undef T
#undef SUF
#undef MAC

#define T int32_t
#define SUF(x) x##_i
#define MAC(cin, w, b) mac_i((cin), (w), (b))
#include "cyc_oracle_walkers.inc"
#undef T
#undef SUF
#undef MAC

/* ------------------------------------------------------------------ */
/* public entry points (ctypes)                                        */
/* ------------------------------------------------------------------ */
/* A is [M][K] row-major.  B is [K][N] row-major, or, with b_col_major != 0,
 * stored as [N][K] (element B_kj at B[j*K + k]).  C is [M][N] row-major,
 * float for dtype 0/1, int32 for dtype 2.                              */

static int widen_inputs(int dtype, int64_t M, int64_t N, int64_t K, const void *A, const void *B, int b_col_major, void **Aw,
                        void **Bw) {
    if (M <= 0 || N <= 0 || K <= 0 || !A || !B) return ORC_BAD_ARG;
    int64_t brs = b_col_major ? 1 : N, bcs = b_col_major ? K : 1;
    if (dtype == CYC_ORACLE_I8_I32) {
        *Aw = widen_i(A, M, K, K, 1);
        *Bw = widen_i(B, K, N, brs, bcs);
    } else if (dtype == CYC_ORACLE_F32 || dtype == CYC_ORACLE_BF16_F32) {
        *Aw = widen_f(dtype, A, M, K, K, 1);
        *Bw = widen_f(dtype, B, K, N, brs, bcs);
    } else
        return ORC_BAD_ARG;
    if (!*Aw || !*Bw) {
        free(*Aw);
        free(*Bw);
        return ORC_NO_MEM;
    }
    return ORC_OK;
}

/* mode: 0 literal, 1 wavefront, 2 os_cannon.  `counts` (may be NULL) receives
 * 9*ST_COUNT statement counters for the literal and wavefront modes.       */
int cyc_oracle_walk(int mode, int dtype, int64_t M, int64_t N, int64_t K, const void *A, const void *B, int b_col_major,
                    void *C, int fma, int64_t *counts) {
    void *Aw = NULL, *Bw = NULL;
    int rc = widen_inputs(dtype, M, N, K, A, B, b_col_major, &Aw, &Bw);
    if (rc) return rc;
    if (!C) rc = ORC_BAD_ARG;
    else if (dtype == CYC_ORACLE_I8_I32) {
        if (mode == 0) rc = ws_literal_i(M, N, K, Aw, Bw, C, fma, counts);
        else if (mode == 1) rc = ws_wavefront_i(M, N, K, Aw, Bw, C, fma, counts);
        else if (mode == 2) rc = os_cannon_i(M, N, K, Aw, Bw, C, fma);
        else rc = ORC_BAD_ARG;
    } else {
        if (mode == 0) rc = ws_literal_f(M, N, K, Aw, Bw, C, fma, counts);
        else if (mode == 1) rc = ws_wavefront_f(M, N, K, Aw, Bw, C, fma, counts);
        else if (mode == 2) rc = os_cannon_f(M, N, K, Aw, Bw, C, fma);
        else rc = ORC_BAD_ARG;
    }
    free(Aw);
    free(Bw);
    return rc;
}

/* collapsed mode on a list of rows: Crows is [nrows][N]; rows == NULL means
 * rows 0 .. nrows-1.  nthreads >= 1.                                      */
typedef struct {
    int dtype, fma;
    int64_t N, K;
    const void *Aw, *Bw;
    const int64_t *rows;
    void *Crows;
    int64_t r0, r1;
} collapsed_job;

static void *collapsed_worker(void *p) {
    collapsed_job *jb = (collapsed_job *)p;
    if (jb->dtype == CYC_ORACLE_I8_I32)
        ws_collapsed_rows_i(jb->N, jb->K, (const int32_t *)jb->Aw, (const int32_t *)jb->Bw, jb->rows, jb->r0, jb->r1,
                            (int32_t *)jb->Crows, jb->fma);
    else
        ws_collapsed_rows_f(jb->N, jb->K, (const float *)jb->Aw, (const float *)jb->Bw, jb->rows, jb->r0, jb->r1,
                            (float *)jb->Crows, jb->fma);
    return NULL;
}

int cyc_oracle_collapsed_rows(int dtype, int64_t M, int64_t N, int64_t K, const void *A, const void *B, int b_col_major,
                              const int64_t *rows, int64_t nrows, void *Crows, int fma, int nthreads) {
    if (nrows <= 0 || !Crows || nthreads < 1) return ORC_BAD_ARG;
    if (rows)
        for (int64_t r = 0; r < nrows; ++r)
            if (rows[r] < 0 || rows[r] >= M) return ORC_BAD_ARG;
    if (!rows && nrows > M) return ORC_BAD_ARG;
    void *Aw = NULL, *Bw = NULL;
    int rc = widen_inputs(dtype, M, N, K, A, B, b_col_major, &Aw, &Bw);
    if (rc) return rc;
    if (nthreads > nrows) nthreads = (int)nrows;
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    collapsed_job *jobs = (collapsed_job *)malloc(sizeof(collapsed_job) * (size_t)nthreads);
    if (!th || !jobs) {
        free(th); free(jobs); free(Aw); free(Bw);
        return ORC_NO_MEM;
    }
    for (int t = 0; t < nthreads; ++t) {
        collapsed_job jb = {dtype, fma, N, K, Aw, Bw, rows, Crows, nrows * t / nthreads, nrows * (t + 1) / nthreads};
        jobs[t] = jb;
        if (nthreads == 1) collapsed_worker(&jobs[t]);
        else pthread_create(&th[t], NULL, collapsed_worker, &jobs[t]);
    }
    if (nthreads > 1)
        for (int t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
    free(th); free(jobs); free(Aw); free(Bw);
    return ORC_OK;
}

/* single outputs: out[p] = (ii[p], jj[p], k_end)_C ; float or int32 per dtype.
 * Reads the stored operands in place (no widened copy), so it is usable on the
 * largest configurations.                                                   */
int cyc_oracle_points(int dtype, int64_t M, int64_t N, int64_t K, const void *A, const void *B, int b_col_major,
                      const int64_t *ii, const int64_t *jj, int64_t npts, void *out, int fma) {
    if (M <= 0 || N <= 0 || K <= 0 || !A || !B || !ii || !jj || !out || npts < 0) return ORC_BAD_ARG;
    int64_t brs = b_col_major ? 1 : N, bcs = b_col_major ? K : 1;
    for (int64_t p = 0; p < npts; ++p) {
        int64_t i = ii[p], j = jj[p];
        if (i < 0 || i >= M || j < 0 || j >= N) return ORC_BAD_ARG;
        if (dtype == CYC_ORACLE_I8_I32) {
            int32_t c = 0; /* (i,j,0)_C <- 0 */
            for (int64_t k = 0; k < K; ++k)
                c = mac_i(c, (int32_t)((const int8_t *)A)[i * K + k], (int32_t)((const int8_t *)B)[k * brs + j * bcs]);
            ((int32_t *)out)[p] = c;
        } else if (dtype == CYC_ORACLE_F32) {
            float c = 0.0f;
            for (int64_t k = 0; k < K; ++k) c = mac_f(c, ((const float *)A)[i * K + k], ((const float *)B)[k * brs + j * bcs], fma);
            ((float *)out)[p] = c;
        } else if (dtype == CYC_ORACLE_BF16_F32) {
            float c = 0.0f;
            for (int64_t k = 0; k < K; ++k)
                c = mac_f(c, bf16_to_f32(((const uint16_t *)A)[i * K + k]), bf16_to_f32(((const uint16_t *)B)[k * brs + j * bcs]),
                          fma);
            ((float *)out)[p] = c;
        } else
            return ORC_BAD_ARG;
    }
    return ORC_OK;
}

/* For the tolerance checks: S_ij = sum_k |A_ik||B_kj| and the exact-product
 * double-precision sum R_ij = sum_k A_ik B_kj, for the listed rows (or single
 * points when jj != NULL: then S and R are [npts]).                          */
static double load_d(int dtype, const void *p, int64_t at) {
    if (dtype == CYC_ORACLE_F32) return (double)((const float *)p)[at];
    if (dtype == CYC_ORACLE_BF16_F32) return (double)bf16_to_f32(((const uint16_t *)p)[at]);
    return (double)((const int8_t *)p)[at];
}

int cyc_oracle_abs_sum_points(int dtype, int64_t M, int64_t N, int64_t K, const void *A, const void *B, int b_col_major,
                              const int64_t *ii, const int64_t *jj, int64_t npts, double *S, double *R) {
    if (M <= 0 || N <= 0 || K <= 0 || !A || !B || !ii || !jj || npts < 0) return ORC_BAD_ARG;
    if (dtype < 0 || dtype > 2) return ORC_BAD_ARG;
    int64_t brs = b_col_major ? 1 : N, bcs = b_col_major ? K : 1;
    for (int64_t p = 0; p < npts; ++p) {
        int64_t i = ii[p], j = jj[p];
        if (i < 0 || i >= M || j < 0 || j >= N) return ORC_BAD_ARG;
        double s = 0.0, r = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double a = load_d(dtype, A, i * K + k), b = load_d(dtype, B, k * brs + j * bcs);
            s += fabs(a) * fabs(b);
            r += a * b;
        }
        if (S) S[p] = s;
        if (R) R[p] = r;
    }
    return ORC_OK;
}

typedef struct {
    int dtype;
    int64_t N, K, brs, bcs;
    const void *A, *B;
    const int64_t *rows;
    double *S, *R;
    int64_t r0, r1;
} abs_job;

static void *abs_worker(void *p) {
    abs_job *jb = (abs_job *)p;
    for (int64_t r = jb->r0; r < jb->r1; ++r) {
        int64_t i = jb->rows ? jb->rows[r] : r;
        double *s = jb->S ? jb->S + r * jb->N : NULL, *q = jb->R ? jb->R + r * jb->N : NULL;
        for (int64_t j = 0; j < jb->N; ++j) {
            if (s) s[j] = 0.0;
            if (q) q[j] = 0.0;
        }
        for (int64_t k = 0; k < jb->K; ++k) {
            double a = load_d(jb->dtype, jb->A, i * jb->K + k);
            for (int64_t j = 0; j < jb->N; ++j) {
                double b = load_d(jb->dtype, jb->B, k * jb->brs + j * jb->bcs);
                if (s) s[j] += fabs(a) * fabs(b);
                if (q) q[j] += a * b;
            }
        }
    }
    return NULL;
}

int cyc_oracle_abs_sum_rows(int dtype, int64_t M, int64_t N, int64_t K, const void *A, const void *B, int b_col_major,
                            const int64_t *rows, int64_t nrows, double *S, double *R, int nthreads) {
    if (M <= 0 || N <= 0 || K <= 0 || !A || !B || nrows <= 0 || nthreads < 1) return ORC_BAD_ARG;
    if (dtype < 0 || dtype > 2) return ORC_BAD_ARG;
    if (rows)
        for (int64_t r = 0; r < nrows; ++r)
            if (rows[r] < 0 || rows[r] >= M) return ORC_BAD_ARG;
    if (!rows && nrows > M) return ORC_BAD_ARG;
    if (nthreads > nrows) nthreads = (int)nrows;
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    abs_job *jobs = (abs_job *)malloc(sizeof(abs_job) * (size_t)nthreads);
    if (!th || !jobs) {
        free(th); free(jobs);
        return ORC_NO_MEM;
    }
    for (int t = 0; t < nthreads; ++t) {
        abs_job jb = {dtype, N, K, b_col_major ? 1 : N, b_col_major ? K : 1, A, B, rows, S, R, nrows * t / nthreads,
                      nrows * (t + 1) / nthreads};
        jobs[t] = jb;
        if (nthreads == 1) abs_worker(&jobs[t]);
        else pthread_create(&th[t], NULL, abs_worker, &jobs[t]);
    }
    if (nthreads > 1)
        for (int t = 0; t < nthreads; ++t) pthread_join(th[t], NULL);
    free(th); free(jobs);
    return ORC_OK;
}

int cyc_oracle_statement_count(void) { return ST_COUNT; }
