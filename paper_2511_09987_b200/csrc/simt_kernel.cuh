// General kernel: every C_ij is one dependent chain  acc <- acc + A_ik * B_kj,
// k = 0, 1, ..., K-1, starting from zero -- the partial sum of the recurrence
// walking east through the cells (i,0), (i,1), ... of its row.  fp32 chains use
// a fused multiply-add (one rounding per cell).  The chain never leaves the
// thread's registers, so the "forward C east" step of the per-cell programs
// costs nothing.
//
// CTA = 128 x 128 block of C (cells of 128 rows i x all k, time steps j of 128
// columns), 256 threads, 8 x 8 outputs per thread; A and B k-slabs of depth 16
// staged through shared memory (B_kj read once per CTA and reused by all 128
// rows = the copy of B southwards along i).  Any shape, any alignment, both B
// layouts, any batch.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace cyc {

struct SimtParams {
    const void* A;
    const void* B;
    void* C;
    int M, N, K;
    long long sA, sB, sC;  // batch strides, elements
    long long lda;         // row pitch of A, elements (K when A is dense)
    long long b_sk, b_sj;  // element B_kj at B[k*b_sk + j*b_sj]
    int tiles_m, tiles_n;
};

constexpr int SIMT_BM = 128, SIMT_BN = 128, SIMT_BK = 16, SIMT_THREADS = 256;

template <typename TIn, typename TAcc>
__device__ __forceinline__ TAcc simt_widen(TIn v);
template <>
__device__ __forceinline__ float simt_widen<float, float>(float v) { return v; }
template <>
__device__ __forceinline__ float simt_widen<__nv_bfloat16, float>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <>
__device__ __forceinline__ int simt_widen<int8_t, int>(int8_t v) { return static_cast<int>(v); }

__device__ __forceinline__ float simt_mac(float acc, float a, float b) { return fmaf(a, b, acc); }
__device__ __forceinline__ int simt_mac(int acc, int a, int b) { return acc + a * b; }

// VEC: fp32 only; A, B, C 16-byte aligned, K % 4 == 0, N % 4 == 0, B row-major.
template <typename TIn, typename TAcc, bool VEC>
__global__ void __launch_bounds__(SIMT_THREADS, 2) simt_recurrence_kernel(const SimtParams p) {
    __shared__ __align__(16) TAcc As[2][SIMT_BK][SIMT_BM];
    __shared__ __align__(16) TAcc Bs[2][SIMT_BK][SIMT_BN];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    long long t = blockIdx.x;
    const int tn = static_cast<int>(t % p.tiles_n);
    t /= p.tiles_n;
    const int tm = static_cast<int>(t % p.tiles_m);
    const long long batch = t / p.tiles_m;
    const int m0 = tm * SIMT_BM, n0 = tn * SIMT_BN;

    const TIn* __restrict__ A = static_cast<const TIn*>(p.A) + batch * p.sA;
    const TIn* __restrict__ B = static_cast<const TIn*>(p.B) + batch * p.sB;
    TAcc* __restrict__ C = static_cast<TAcc*>(p.C) + batch * p.sC;
    const int M = p.M, N = p.N, K = p.K;

    // staging registers for the next k-slab: 8 elements of A and 8 of B per thread
    TAcc ra[8], rb[8];

    auto load_slab = [&](int k0) {
        if constexpr (VEC) {
            // A: 128 rows x 16 k = 512 float4; thread -> rows (tid>>2) and (tid>>2)+64, k quad (tid&3)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = (tid >> 2) + 64 * h, kq = (tid & 3) * 4;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (m0 + r < M && k0 + kq < K) v = *reinterpret_cast<const float4*>(A + static_cast<long long>(m0 + r) * p.lda + k0 + kq);
                ra[4 * h + 0] = v.x; ra[4 * h + 1] = v.y; ra[4 * h + 2] = v.z; ra[4 * h + 3] = v.w;
            }
            // B: 16 k x 128 j = 512 float4; thread -> k rows (tid>>5) and (tid>>5)+8, j quad (tid&31)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int kr = (tid >> 5) + 8 * h, jq = (tid & 31) * 4;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (k0 + kr < K && n0 + jq < N) v = *reinterpret_cast<const float4*>(B + static_cast<long long>(k0 + kr) * N + n0 + jq);
                rb[4 * h + 0] = v.x; rb[4 * h + 1] = v.y; rb[4 * h + 2] = v.z; rb[4 * h + 3] = v.w;
            }
        } else {
            // element-wise, fully guarded; A: element e -> row e/16, k e%16 ; B: element e -> k e/128, j e%128
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int idx = tid + e * SIMT_THREADS;
                const int r = idx >> 4, kk = idx & 15;
                TAcc v = TAcc(0);
                if (m0 + r < M && k0 + kk < K) v = simt_widen<TIn, TAcc>(A[static_cast<long long>(m0 + r) * p.lda + k0 + kk]);
                ra[e] = v;
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int idx = tid + e * SIMT_THREADS;
                int kk, j;
                if (p.b_sj == 1) { kk = idx >> 7; j = idx & 127; }   // row-major B: consecutive threads along j
                else { kk = idx & 15; j = idx >> 4; }                // column-major B: consecutive threads along k
                TAcc v = TAcc(0);
                if (k0 + kk < K && n0 + j < N) v = simt_widen<TIn, TAcc>(B[static_cast<long long>(k0 + kk) * p.b_sk + static_cast<long long>(n0 + j) * p.b_sj]);
                rb[e] = v;
            }
        }
    };
    auto store_slab = [&](int buf) {
        if constexpr (VEC) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = (tid >> 2) + 64 * h, kq = (tid & 3) * 4;
#pragma unroll
                for (int q = 0; q < 4; ++q) As[buf][kq + q][r] = ra[4 * h + q];
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int kr = (tid >> 5) + 8 * h, jq = (tid & 31) * 4;
                *reinterpret_cast<float4*>(&Bs[buf][kr][jq]) = make_float4(rb[4 * h + 0], rb[4 * h + 1], rb[4 * h + 2], rb[4 * h + 3]);
            }
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int idx = tid + e * SIMT_THREADS;
                As[buf][idx & 15][idx >> 4] = ra[e];
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int idx = tid + e * SIMT_THREADS;
                if (p.b_sj == 1) Bs[buf][idx >> 7][idx & 127] = rb[e];
                else Bs[buf][idx & 15][idx >> 4] = rb[e];
            }
        }
    };

    // [i,0-1]_C = 0: every chain starts from zero
    TAcc acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = TAcc(0);

    const int nslabs = (K + SIMT_BK - 1) / SIMT_BK;
    load_slab(0);
    store_slab(0);
    __syncthreads();
    for (int s = 0; s < nslabs; ++s) {
        const int buf = s & 1;
        if (s + 1 < nslabs) load_slab((s + 1) * SIMT_BK);
        const int kmax = min(SIMT_BK, K - s * SIMT_BK);  // never run a chain past k_end (keeps -0/+0 and NaN semantics exact)
        if (kmax == SIMT_BK) {
#pragma unroll
            for (int kk = 0; kk < SIMT_BK; ++kk) {
                TAcc a[8], b[8];
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        a[4 * h + q] = As[buf][kk][64 * h + ty * 4 + q];
                        b[4 * h + q] = Bs[buf][kk][64 * h + tx * 4 + q];
                    }
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = simt_mac(acc[i][j], a[i], b[j]);
            }
        } else {
            for (int kk = 0; kk < kmax; ++kk) {
                TAcc a[8], b[8];
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        a[4 * h + q] = As[buf][kk][64 * h + ty * 4 + q];
                        b[4 * h + q] = Bs[buf][kk][64 * h + tx * 4 + q];
                    }
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = simt_mac(acc[i][j], a[i], b[j]);
            }
        }
        if (s + 1 < nslabs) {
            store_slab(buf ^ 1);
            __syncthreads();
        }
    }

    // C_ij <- [i,k_end]_C
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = m0 + 64 * (i >> 2) + ty * 4 + (i & 3);
        if (r >= M) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int c = n0 + 64 * h + tx * 4;
            TAcc* dst = C + static_cast<long long>(r) * N + c;
            if constexpr (VEC) {
                if (c < N) *reinterpret_cast<float4*>(dst) = make_float4(acc[i][4 * h + 0], acc[i][4 * h + 1], acc[i][4 * h + 2], acc[i][4 * h + 3]);
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (c + q < N) dst[q] = acc[i][4 * h + q];
            }
        }
    }
}

// Small problems (fewer 128 x 128 tiles than half the SMs): 64 x 64 tiles, 4 x 4 outputs per
// thread, so that more SMs take part and the per-thread chain work shrinks.  Same chains, same
// order, same bits; element-wise guarded loads (any shape, any alignment).
constexpr int SIMT_S_BM = 64, SIMT_S_BN = 64, SIMT_S_BK = 64;  // a deep slab: one round trip to memory per 64 k

template <typename TIn, typename TAcc>
__global__ void __launch_bounds__(SIMT_THREADS) simt_recurrence_small_kernel(const SimtParams p) {
    __shared__ __align__(16) TAcc As[SIMT_S_BK][SIMT_S_BM + 4];
    __shared__ __align__(16) TAcc Bs[SIMT_S_BK][SIMT_S_BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    long long t = blockIdx.x;
    const int tn = static_cast<int>(t % p.tiles_n);
    t /= p.tiles_n;
    const int tm = static_cast<int>(t % p.tiles_m);
    const long long batch = t / p.tiles_m;
    const int m0 = tm * SIMT_S_BM, n0 = tn * SIMT_S_BN;
    const TIn* __restrict__ A = static_cast<const TIn*>(p.A) + batch * p.sA;
    const TIn* __restrict__ B = static_cast<const TIn*>(p.B) + batch * p.sB;
    TAcc* __restrict__ C = static_cast<TAcc*>(p.C) + batch * p.sC;
    const int M = p.M, N = p.N, K = p.K;

    TAcc acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = TAcc(0);  // [i,0-1]_C = 0

    for (int k0 = 0; k0 < K; k0 += SIMT_S_BK) {
        // 64 x 64 elements of A and of B: sixteen of each per thread, all loads issued before the first use
        TAcc ra[16], rb[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const int idx = tid + e * SIMT_THREADS;
            const int r = idx >> 6, kk = idx & 63;
            ra[e] = TAcc(0);
            if (m0 + r < M && k0 + kk < K) ra[e] = simt_widen<TIn, TAcc>(A[static_cast<long long>(m0 + r) * p.lda + k0 + kk]);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const int idx = tid + e * SIMT_THREADS;
            int kk, j;
            if (p.b_sj == 1) { kk = idx >> 6; j = idx & 63; }
            else { kk = idx & 63; j = idx >> 6; }
            rb[e] = TAcc(0);
            if (k0 + kk < K && n0 + j < N) rb[e] = simt_widen<TIn, TAcc>(B[static_cast<long long>(k0 + kk) * p.b_sk + static_cast<long long>(n0 + j) * p.b_sj]);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const int idx = tid + e * SIMT_THREADS;
            As[idx & 63][idx >> 6] = ra[e];
            if (p.b_sj == 1) Bs[idx >> 6][idx & 63] = rb[e];
            else Bs[idx & 63][idx >> 6] = rb[e];
        }
        __syncthreads();
        const int kmax = min(SIMT_S_BK, K - k0);  // never run a chain past k_end
        for (int kk = 0; kk < kmax; ++kk) {
            TAcc a[4], b[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                a[q] = As[kk][ty * 4 + q];
                b[q] = Bs[kk][tx * 4 + q];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = simt_mac(acc[i][j], a[i], b[j]);
        }
        __syncthreads();
    }
    // C_ij <- [i,k_end]_C
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = m0 + ty * 4 + i;
        if (r >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = n0 + tx * 4 + j;
            if (c < N) C[static_cast<long long>(r) * N + c] = acc[i][j];
        }
    }
}

}  // namespace cyc
