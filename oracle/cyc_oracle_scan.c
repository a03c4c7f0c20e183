/*
 * CPU oracle for the prefix-sum recurrence (Figure "Representative
 * recurrences"):
 *
 *     P_i = P_{i-1} + A_i
 *
 * The paper leaves the start implicit; it is read as P_{-1} = 0, so that
 * P_0 = A_0 (the inclusive prefix sum).  The recurrence is walked literally:
 * one addition per element, in increasing i, each step reading the value the
 * previous step produced.
 *
 * THIS IS TEST INFRASTRUCTURE.  A plain, slow evaluator used only to check
 * the GPU library and to report a CPU baseline.  It shares no code, header,
 * table or helper with the CUDA path and must never be called from the
 * product path.
 *
 * Three arithmetics:
 *   f64   fp32 inputs widened exactly, the running value kept in fp64 (the paper
 *         fixes no precision); also returns S_i = sum_{k<=i} |A_k| in fp64, the
 *         scale of the tolerance checks
 *   f32   the same walk with the running value in fp32 (one rounding per step):
 *         what the recurrence gives when evaluated in the data's own precision
 *   i32   two's-complement 32-bit integers, wrapping (computed on unsigned
 *         words, where wrap-around is defined)
 * `rows` independent sequences of length n, row r starting at element
 * r * stride of A and of P.
 *
 * Build:  gcc -O2 -fno-fast-math -ffp-contract=off -shared -fPIC
 */
#include <math.h>
#include <stdint.h>

#define ORS_OK 0
#define ORS_BAD_ARG 1

int cyc_oracle_prefix_sum_f64(int64_t rows, int64_t n, int64_t stride, const float *A, double *P, double *S) {
    if (rows < 0 || n < 0 || stride < n || !A || !P) return ORS_BAD_ARG;
    for (int64_t r = 0; r < rows; ++r) {
        double prev = 0.0;   /* P_{-1} */
        double scale = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            const double a = (double)A[r * stride + i];
            prev = prev + a;             /* P_i = P_{i-1} + A_i */
            P[r * stride + i] = prev;
            if (S) {
                scale = scale + fabs(a);
                S[r * stride + i] = scale;
            }
        }
    }
    return ORS_OK;
}

int cyc_oracle_prefix_sum_f32(int64_t rows, int64_t n, int64_t stride, const float *A, float *P) {
    if (rows < 0 || n < 0 || stride < n || !A || !P) return ORS_BAD_ARG;
    for (int64_t r = 0; r < rows; ++r) {
        volatile float prev = 0.0f;      /* volatile: every step is rounded to fp32 */
        for (int64_t i = 0; i < n; ++i) {
            prev = prev + A[r * stride + i];
            P[r * stride + i] = prev;
        }
    }
    return ORS_OK;
}

int cyc_oracle_prefix_sum_i32(int64_t rows, int64_t n, int64_t stride, const int32_t *A, int32_t *P) {
    if (rows < 0 || n < 0 || stride < n || !A || !P) return ORS_BAD_ARG;
    for (int64_t r = 0; r < rows; ++r) {
        uint32_t prev = 0u;
        for (int64_t i = 0; i < n; ++i) {
            prev = prev + (uint32_t)A[r * stride + i];
            P[r * stride + i] = (int32_t)prev;
        }
    }
    return ORS_OK;
}
