// Diagonal space of the block lower-triangular solve L X = B (Figure "deps-tri-solve"):
//
//      (ii,ii)_Xa <- end of row ii of the triangular space          (interface map Phi_1)
//      (ii,ii)_X  <- TRSM( L_ii , B_ii - (ii,ii)_Xa ),   X_ii <- (ii,ii)_X
//
// The triangular space (the GEMM updates sum_j L_ij X_j) runs on the recurrence-matmul kernels; its end-of-row
// accumulator reaches this kernel as up to 32 partial-sum planes W_l (one per level of the recursive split of the
// block rows), summed here in increasing l.
//
// One CTA solves one diagonal tile (rows <= 256) for 32 right-hand-side columns; lane = column, so every shared-memory
// access of the right-hand side is conflict-free and every global access of B, W, X is a 128-byte row segment.
// The tile is processed in sub-blocks of 32 rows:
//   update   rows of the sub-block  -=  L[sub-block rows][earlier rows of the tile] * X[earlier rows]   (8 warps x 4 rows)
//   solve    the 32 x 32 triangle by a column sweep in registers (warp 0): x_k = s_k / L_kk, s_r -= L_rk x_k for r > k
// The L panel of the next sub-block is fetched with cp.async while the current one is processed.  Entries of L above
// the diagonal are never used.  x_k is formed as s_k * (1 / L_kk) with a correctly rounded reciprocal.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace cyc {

struct TrsmDiagParams {
    const float* L;   // [n][n] row-major
    const float* B;   // [n][m]
    float* X;         // [n][m]; may be B
    const float* W;   // planes [levels][n][m] of partial sums; not read when mask == 0
    long long plane;  // n * m
    int n, m;
    int r0, rows;     // the tile: rows [r0, r0 + rows), rows <= TRSM_T_MAX
    unsigned mask;    // bit l set: plane l holds a partial sum for these rows
};

constexpr int TRSM_T_MAX = 256, TRSM_CW = 32, TRSM_SB = 32, TRSM_THREADS = 256;
constexpr int TRSM_LP_PITCH = TRSM_T_MAX + 4;  // floats; rows stay 16-byte aligned, row starts fall in different banks
constexpr int TRSM_LT_PITCH = TRSM_SB + 4;
constexpr int TRSM_SMEM_BYTES =
    (TRSM_T_MAX * TRSM_CW + 2 * TRSM_SB * TRSM_LP_PITCH + TRSM_SB * TRSM_LT_PITCH + TRSM_SB) * static_cast<int>(sizeof(float));

__device__ __forceinline__ void trsm_cp_async4(float* dst_smem, const float* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem))), "l"(src)
                 : "memory");
}
__device__ __forceinline__ void trsm_cp_async16(float* dst_smem, const float* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem))), "l"(src)
                 : "memory");
}
__device__ __forceinline__ void trsm_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void trsm_cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__global__ void __launch_bounds__(TRSM_THREADS) trsm_diag_kernel(const TrsmDiagParams p) {
    extern __shared__ __align__(16) float trsm_smem[];
    float(*Xs)[TRSM_CW] = reinterpret_cast<float(*)[TRSM_CW]>(trsm_smem);                     // right-hand side, then X
    float* Lp_base = trsm_smem + TRSM_T_MAX * TRSM_CW;                                        // two panels
    float(*Lt)[TRSM_LT_PITCH] = reinterpret_cast<float(*)[TRSM_LT_PITCH]>(Lp_base + 2 * TRSM_SB * TRSM_LP_PITCH);
    float* dinv = reinterpret_cast<float*>(Lt) + TRSM_SB * TRSM_LT_PITCH;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c = blockIdx.x * TRSM_CW + lane;
    const bool col_ok = c < p.m;

    // panel of sub-block sb: rows [s0, s0+32) of the tile, tile columns [0, s0+32); rows past the tile are zero.
    // Warp w fetches rows w, w+8, w+16, w+24; 16-byte copies when every row of L starts on a 16-byte boundary.
    const bool vec_ok = (reinterpret_cast<uintptr_t>(p.L) % 16 == 0) && (p.n % 4 == 0) && (p.r0 % 4 == 0);
    auto issue_panel = [&](int s0, int buf) {
        float* Lp = Lp_base + buf * TRSM_SB * TRSM_LP_PITCH;
        const int width = s0 + TRSM_SB;
#pragma unroll
        for (int i = 0; i < TRSM_SB / 8; ++i) {
            const int r = warp + 8 * i;
            float* dst = Lp + r * TRSM_LP_PITCH;
            const float* src = p.L + static_cast<long long>(p.r0 + s0 + r) * p.n + p.r0;
            const bool row_ok = s0 + r < p.rows;
            for (int k = 4 * lane; k < width; k += 128) {
                if (row_ok && vec_ok && k + 4 <= p.rows) {
                    trsm_cp_async16(dst + k, src + k);
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (row_ok && k + q < p.rows) trsm_cp_async4(dst + k + q, src + k + q);
                        else dst[k + q] = 0.f;
                    }
                }
            }
        }
        trsm_cp_async_commit();
    };
    issue_panel(0, 0);

    // right-hand side of the tile: B_ii - Xa, Xa = the partial-sum planes in increasing level.  Eight rows per warp
    // at a time, all their loads in flight together.
    for (int rb = 0; rb < TRSM_T_MAX; rb += 64) {
        float v[8], xa[8];
        long long at[8];
        bool ok[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = rb + 8 * i + warp;
            ok[i] = r < p.rows && col_ok;
            at[i] = static_cast<long long>(p.r0 + r) * p.m + c;
            v[i] = ok[i] ? __ldg(p.B + at[i]) : 0.f;
            xa[i] = 0.f;
        }
        unsigned mk = p.mask;
        for (int l = 0; mk; ++l, mk >>= 1) {
            if (!(mk & 1u)) continue;
            const float* Wl = p.W + l * p.plane;
            float w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i] = ok[i] ? __ldg(Wl + at[i]) : 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) xa[i] += w[i];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) Xs[rb + 8 * i + warp][lane] = v[i] - xa[i];
    }

    for (int s0 = 0, sb = 0; s0 < p.rows; s0 += TRSM_SB, ++sb) {
        const int buf = sb & 1;
        float* Lp = Lp_base + buf * TRSM_SB * TRSM_LP_PITCH;
        trsm_cp_async_wait_all();
        __syncthreads();  // panel sb complete; rows < s0 of Xs final; the other panel buffer and Lt free again
        if (s0 + TRSM_SB < p.rows) issue_panel(s0 + TRSM_SB, buf ^ 1);

        // diagonal 32 x 32 block transposed (strictly lower part only) and the reciprocals of its diagonal
        for (int idx = tid; idx < TRSM_SB * TRSM_SB; idx += TRSM_THREADS) {
            const int r = idx >> 5, k = idx & 31;
            Lt[k][r] = (r > k) ? Lp[r * TRSM_LP_PITCH + s0 + k] : 0.f;
        }
        if (tid < TRSM_SB) dinv[tid] = (s0 + tid < p.rows) ? 1.0f / Lp[tid * TRSM_LP_PITCH + s0 + tid] : 1.0f;

        // update: rows s0 + 4*warp .. +3  -=  L[row][0..s0) . X[0..s0)
        if (s0 > 0) {
            float acc[4][2] = {};  // two partial sums per row (even and odd pairs of k): eight independent chains
            const float* lrow = Lp + (4 * warp) * TRSM_LP_PITCH;
#pragma unroll 2
            for (int k = 0; k < s0; k += 4) {
                const float x0 = Xs[k][lane], x1 = Xs[k + 1][lane], x2 = Xs[k + 2][lane], x3 = Xs[k + 3][lane];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 l = *reinterpret_cast<const float4*>(lrow + i * TRSM_LP_PITCH + k);
                    acc[i][0] = fmaf(l.x, x0, acc[i][0]);
                    acc[i][1] = fmaf(l.y, x1, acc[i][1]);
                    acc[i][0] = fmaf(l.z, x2, acc[i][0]);
                    acc[i][1] = fmaf(l.w, x3, acc[i][1]);
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) Xs[s0 + 4 * warp + i][lane] -= acc[i][0] + acc[i][1];
        }
        __syncthreads();  // updated right-hand side, Lt and dinv visible to warp 0

        if (warp == 0) {
            float s[TRSM_SB];
#pragma unroll
            for (int r = 0; r < TRSM_SB; ++r) s[r] = Xs[s0 + r][lane];
            const float my_dinv = dinv[lane];
            float4 lnext[TRSM_SB / 4];  // column k+1 of the triangle (row k+1 of Lt), fetched while column k is applied
#pragma unroll
            for (int g = 0; g < TRSM_SB / 4; ++g) lnext[g] = *reinterpret_cast<const float4*>(&Lt[0][4 * g]);
#pragma unroll
            for (int k = 0; k < TRSM_SB; ++k) {
                float4 l[TRSM_SB / 4];
#pragma unroll
                for (int g = 0; g < TRSM_SB / 4; ++g) l[g] = lnext[g];
                if (k + 1 < TRSM_SB) {
#pragma unroll
                    for (int g = (k + 2) / 4; g < TRSM_SB / 4; ++g) lnext[g] = *reinterpret_cast<const float4*>(&Lt[k + 1][4 * g]);
                }
                const float xk = s[k] * __shfl_sync(0xffffffffu, my_dinv, k);
                s[k] = xk;
#pragma unroll
                for (int g = (k + 1) / 4; g < TRSM_SB / 4; ++g) {  // entries with r <= k are zero in Lt and skipped here
                    if (4 * g + 0 > k) s[4 * g + 0] = fmaf(-l[g].x, xk, s[4 * g + 0]);
                    if (4 * g + 1 > k) s[4 * g + 1] = fmaf(-l[g].y, xk, s[4 * g + 1]);
                    if (4 * g + 2 > k) s[4 * g + 2] = fmaf(-l[g].z, xk, s[4 * g + 2]);
                    if (4 * g + 3 > k) s[4 * g + 3] = fmaf(-l[g].w, xk, s[4 * g + 3]);
                }
            }
#pragma unroll
            for (int r = 0; r < TRSM_SB; ++r) {
                Xs[s0 + r][lane] = s[r];
                if (s0 + r < p.rows && col_ok) p.X[static_cast<long long>(p.r0 + s0 + r) * p.m + c] = s[r];
            }
        }
    }
}

}  // namespace cyc
