/*
 * CPU oracle for the FlashAttention-2 recurrence (Section "Simulated Cholesky
 * and Flash Attention", paragraph "FlashAttention-2 Recurrence"):
 *
 *   S_{i,J_t} = alpha Q_i K_{J_t}^T ,           alpha = 1 / sqrt(d)
 *   mh_i^(t)  = max( m_i^(t-1), max S_{i,J_t} )
 *   l_i^(t)   = exp(m_i^(t-1) - mh_i^(t)) l_i^(t-1) + sum_{j in J_t} exp(S_ij - mh_i^(t))
 *   o_i^(t)   = exp(m_i^(t-1) - mh_i^(t)) o_i^(t-1) + sum_{j in J_t} exp(S_ij - mh_i^(t)) V_j
 *   m_i^(t)   = mh_i^(t) ,      O_i = o_i^(T) / l_i^(T)
 *
 * with m^(0) = -inf, l^(0) = 0, o^(0) = 0 (the paper leaves the initial state
 * implicit; these are the values for which the first step reduces to a plain
 * softmax over the first tile).
 *
 * THIS IS TEST INFRASTRUCTURE.  A plain, slow evaluator used only to check
 * the GPU library and to report a CPU baseline.  It shares no code, header,
 * table or helper with the CUDA path and must never be called from the
 * product path.
 *
 * Q is [N][d], K and V are [M][d], all row-major fp32 (bf16 inputs are widened
 * by the caller); keys are processed in tiles J_t of `tile` consecutive rows
 * (the last one may be shorter).  All arithmetic is fp64 with the C library's
 * exp; the paper fixes no precision.  Outputs: O [N][d]; optionally the final
 * states m [N] and l [N], and A [N][d] = sum_j softmax_ij |V_jd| (the scale of
 * the tolerance checks).  Rows of Q are independent and are split over threads.
 *
 * Build:  gcc -O2 -fno-fast-math -ffp-contract=off -shared -fPIC -pthread
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>

#define ORF_OK 0
#define ORF_BAD_ARG 1
#define ORF_NO_MEM 2

typedef struct {
    int64_t N, M, d, tile, i0, i1;
    const float *Q, *K, *V;
    double *O, *m_out, *l_out, *A;
    int rc;
} fa2_job;

static void *fa2_worker(void *p) {
    fa2_job *jb = (fa2_job *)p;
    int64_t M = jb->M, d = jb->d, T = jb->tile;
    double alpha = 1.0 / sqrt((double)d);
    double *S = (double *)malloc(sizeof(double) * (size_t)T);
    double *o = (double *)malloc(sizeof(double) * (size_t)d);
    double *a = (double *)malloc(sizeof(double) * (size_t)d);
    if (!S || !o || !a) { free(S); free(o); free(a); jb->rc = ORF_NO_MEM; return NULL; }
    for (int64_t i = jb->i0; i < jb->i1; ++i) {
        const float *q = jb->Q + i * d;
        double m = -INFINITY, l = 0.0;
        for (int64_t c = 0; c < d; ++c) { o[c] = 0.0; a[c] = 0.0; }
        for (int64_t j0 = 0; j0 < M; j0 += T) { /* tile J_t */
            int64_t j1 = j0 + T < M ? j0 + T : M;
            double mh = m;
            for (int64_t j = j0; j < j1; ++j) {
                const float *k = jb->K + j * d;
                double s = 0.0;
                for (int64_t c = 0; c < d; ++c) s += (double)q[c] * (double)k[c];
                S[j - j0] = alpha * s;
                if (S[j - j0] > mh) mh = S[j - j0];
            }
            double carry = exp(m - mh); /* exp(-inf) = 0 on the first tile */
            l = carry * l;
            for (int64_t c = 0; c < d; ++c) { o[c] = carry * o[c]; a[c] = carry * a[c]; }
            for (int64_t j = j0; j < j1; ++j) {
                double e = exp(S[j - j0] - mh);
                const float *v = jb->V + j * d;
                l += e;
                for (int64_t c = 0; c < d; ++c) {
                    o[c] += e * (double)v[c];
                    a[c] += e * fabs((double)v[c]);
                }
            }
            m = mh;
        }
        for (int64_t c = 0; c < d; ++c) {
            jb->O[i * d + c] = o[c] / l;
            if (jb->A) jb->A[i * d + c] = a[c] / l;
        }
        if (jb->m_out) jb->m_out[i] = m;
        if (jb->l_out) jb->l_out[i] = l;
    }
    free(S); free(o); free(a);
    jb->rc = ORF_OK;
    return NULL;
}

int cyc_oracle_fa2(int64_t N, int64_t M, int64_t d, int64_t tile, const float *Q, const float *K, const float *V, double *O,
                   double *m_out, double *l_out, double *A, int nthreads) {
    if (N <= 0 || M <= 0 || d <= 0 || tile <= 0 || !Q || !K || !V || !O || nthreads < 1) return ORF_BAD_ARG;
    if (nthreads > N) nthreads = (int)N;
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)nthreads);
    fa2_job *jobs = (fa2_job *)malloc(sizeof(fa2_job) * (size_t)nthreads);
    if (!th || !jobs) { free(th); free(jobs); return ORF_NO_MEM; }
    for (int t = 0; t < nthreads; ++t) {
        fa2_job jb = {N, M, d, tile, N * t / nthreads, N * (t + 1) / nthreads, Q, K, V, O, m_out, l_out, A, ORF_OK};
        jobs[t] = jb;
        if (nthreads == 1) fa2_worker(&jobs[t]);
        else pthread_create(&th[t], NULL, fa2_worker, &jobs[t]);
    }
    int rc = ORF_OK;
    for (int t = 0; t < nthreads; ++t) {
        if (nthreads > 1) pthread_join(th[t], NULL);
        if (jobs[t].rc) rc = jobs[t].rc;
    }
    free(th); free(jobs);
    return rc;
}
