// Diagonal space of the block lower-triangular solve L X = B (Figure "deps-tri-solve"):
//
//      (ii,ii)_Xa <- end of row ii of the triangular space          (interface map Phi_1)
//      (ii,ii)_X  <- TRSM( L_ii , B_ii - (ii,ii)_Xa ),   X_ii <- (ii,ii)_X
//
// The triangular space (the GEMM updates sum_j L_ij X_j) runs on the recurrence-matmul kernels; its end-of-row
// accumulator reaches this kernel as up to 32 partial-sum planes W_l (one per level of the recursive split of the
// block rows), summed here in increasing l.
//
// One CTA solves one diagonal tile (rows <= 256) for 32 right-hand-side columns (8 when the columns are few); lane = column, so every shared-memory
// access of the right-hand side is conflict-free and every global access of B, W, X is a 128-byte row segment.
// The lower triangle of the tile is brought into shared memory once, as 32 x 32 blocks (cp.async; 144 KB for a full
// tile).  The tile is then processed in sub-blocks of 32 rows, with one step of look-ahead so that the sequential part
// overlaps the bulk of the arithmetic:
//   solve(s)     warps 0-3 (eight columns each, four lanes per column): the 32 x 32 triangle of sub-block s by a
//                column sweep in registers, rows pre-scaled by the reciprocal of their diagonal entry:
//                x_r = s_r / L_rr - sum_{k<r} (L_rk / L_rr) x_k
//   trailing(s)  the twelve other warps, at the same time: rows below sub-block s  -=  L[rows][sub-block s-1] * x_(s-1)
//                (a warp takes 16 rows x 32 columns, a lane one column of them)
//   next(s+1)    eight warps: rows of sub-block s+1  -=  L[rows][sub-block s] * x_s; the other eight prepare its triangle
// Every row receives its updates in increasing column order.  Entries of L above the diagonal are never used.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "ptx.cuh"

namespace cyc {

struct TrsmDiagParams {
    const float* L;   // [n][n] row-major
    const float* B;   // right-hand side: entry (tile row r, column c) at B[r * b_r + c * b_c]
    float* X;         // solution, entry (r, c) at X[r * x_r + c * x_c]; may be B
    const float* W;   // planes of partial sums, entry (r, c) of plane l at W[l * plane + r * w_r + c * w_c]; not read when mask == 0
    long long plane;
    long long b_r, b_c, x_r, x_c, w_r, w_c;  // element strides: (m, 1) for row-major [rows][m]; (1, pitch) when the
                                             // right-hand sides are the rows of a row-major matrix (X L^T = B)
    int n, m;         // order of L; number of right-hand-side columns
    int r0, rows;     // the tile of L: rows and columns [r0, r0 + rows), rows <= TRSM_T_MAX
    unsigned mask;    // bit l set: plane l holds a partial sum for these rows
};

constexpr int TRSM_T_MAX = 256, TRSM_CW = 32, TRSM_CW_NARROW = 8, TRSM_SB = 32, TRSM_THREADS = 512, TRSM_WARPS = TRSM_THREADS / 32;
constexpr int TRSM_NSB = TRSM_T_MAX / TRSM_SB;            // sub-blocks per tile
constexpr int TRSM_BLK = TRSM_SB * TRSM_SB;               // floats per 32 x 32 block of L
constexpr int TRSM_NBLK = TRSM_NSB * (TRSM_NSB + 1) / 2;  // blocks on and below the diagonal
constexpr int TRSM_LT_PITCH = TRSM_SB + 4;
constexpr int TRSM_SMEM_BYTES =   // sized for the wider form
    (TRSM_T_MAX * TRSM_CW + TRSM_NBLK * TRSM_BLK + TRSM_SB * TRSM_LT_PITCH + TRSM_SB) * static_cast<int>(sizeof(float));

__device__ __forceinline__ void trsm_cp_async4(float* dst_smem, const float* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem))), "l"(src)
                 : "memory");
}
__device__ __forceinline__ void trsm_cp_async16(float* dst_smem, const float* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem))), "l"(src)
                 : "memory");
}
__device__ __forceinline__ void trsm_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void trsm_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// block (bi, bj), bj <= bi, of the tile's lower triangle; element (r, k) of a block at [r * 32 + k]
__device__ __forceinline__ int trsm_block(int bi, int bj) { return (bi * (bi + 1) / 2 + bj) * TRSM_BLK; }

// One warp:  xdst[0..ROWS)[0..CW)  -=  Lrows[0..ROWS)[0..32) . xsrc[0..32)[0..CW)
// (Lrows: ROWS consecutive rows of one 32 x 32 block; xsrc: the 32 solved rows; xdst: the ROWS rows to update).
// A lane owns one column: it keeps its column of x in registers and walks down rows; with CW = 32 a lane takes every
// row, with CW = 8 the four lanes of a column take every fourth row each.  The entries of L are the same address in all
// lanes of a row group (one 16-byte broadcast per four values of k), so a multiply-add costs a quarter of the
// shared-memory traffic of a register patch per lane, and every access of x is conflict-free.
template <int ROWS, int CW>
__device__ __forceinline__ void trsm_apply(const float* __restrict__ lrows, float (*xsrc)[CW], float (*xdst)[CW], int lane) {
    constexpr int G = 32 / CW;   // row groups per warp
    static_assert(ROWS % (4 * G) == 0, "a lane takes its rows four at a time");
    const int col = lane % CW, g = lane / CW;
    float xr[TRSM_SB];
#pragma unroll
    for (int k = 0; k < TRSM_SB; ++k) xr[k] = xsrc[k][col];
#pragma unroll 1
    for (int i = 0; i < ROWS; i += 4 * G) {   // four rows per lane at a time: four independent chains of multiply-adds
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int k = 0; k < TRSM_SB; k += 4) {
            float4 l[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) l[r] = *reinterpret_cast<const float4*>(lrows + (i + g + G * r) * TRSM_SB + k);
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[r] = fmaf(l[r].x, xr[k], acc[r]);
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[r] = fmaf(l[r].y, xr[k + 1], acc[r]);
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[r] = fmaf(l[r].z, xr[k + 2], acc[r]);
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[r] = fmaf(l[r].w, xr[k + 3], acc[r]);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) xdst[i + g + G * r][col] -= acc[r];
    }
}

// wait until at most `pending` of this thread's cp.async groups are still in flight (pending = 0 .. TRSM_NSB - 1)
__device__ __forceinline__ void trsm_wait_pending(int pending) {
    switch (pending) {
        case 0: trsm_cp_async_wait<0>(); break;
        case 1: trsm_cp_async_wait<1>(); break;
        case 2: trsm_cp_async_wait<2>(); break;
        case 3: trsm_cp_async_wait<3>(); break;
        case 4: trsm_cp_async_wait<4>(); break;
        case 5: trsm_cp_async_wait<5>(); break;
        case 6: trsm_cp_async_wait<6>(); break;
        default: trsm_cp_async_wait<7>(); break;
    }
}

// CW = right-hand-side columns per CTA: 32, or 8 when there are so few columns that 32 per CTA would leave most SMs idle
// (a CTA's arithmetic shrinks with CW, its chain of dependent steps does not, so narrow CTAs pay only then).
template <int CW>
__global__ void __launch_bounds__(TRSM_THREADS, 1) trsm_diag_kernel(const TrsmDiagParams p) {
    static_assert(CW == 32 || CW == 8, "32 or 8 columns per CTA");
    constexpr int G = 32 / CW;   // lanes per column in the updates and in the load of the right-hand side
    extern __shared__ __align__(16) float trsm_smem[];
    float(*Xs)[CW] = reinterpret_cast<float(*)[CW]>(trsm_smem);  // right-hand side, then X
    float* Lb = trsm_smem + TRSM_T_MAX * CW;                     // the blocks of L
    float(*Lt)[TRSM_LT_PITCH] = reinterpret_cast<float(*)[TRSM_LT_PITCH]>(Lb + TRSM_NBLK * TRSM_BLK);
    float* dinv = reinterpret_cast<float*>(Lt) + TRSM_SB * TRSM_LT_PITCH;

    // launched with programmatic stream serialisation: only the launch itself overlaps the previous kernel
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c = blockIdx.x * CW + lane % CW;   // this lane's column in the load of the right-hand side
    const bool col_ok = c < p.m;
    const int nsb = (p.rows + TRSM_SB - 1) / TRSM_SB;

    // Column block j of the triangle (tile rows [32 j, 32 nsb), tile columns [32 j, 32 j + 32)) is one cp.async group:
    // step s of the loop below needs the column blocks up to s only, so the later ones arrive behind the arithmetic.
    // Rows and columns past the tile are zero.  16-byte copies when every row of L starts on a 16-byte boundary.
    const bool vec_ok = (reinterpret_cast<uintptr_t>(p.L) % 16 == 0) && (p.n % 4 == 0) && (p.r0 % 4 == 0);
    for (int j = 0; j < nsb; ++j) {
        const int chunks = (nsb - j) * TRSM_SB * (TRSM_SB / 4);
        for (int idx = tid; idx < chunks; idx += TRSM_THREADS) {
            const int t = j * TRSM_SB + (idx >> 3), k = j * TRSM_SB + 4 * (idx & 7);
            float* dst = Lb + trsm_block(t >> 5, j) + (t & 31) * TRSM_SB + 4 * (idx & 7);
            const float* src = p.L + static_cast<long long>(p.r0 + t) * p.n + p.r0 + k;
            const bool row_ok = t < p.rows;
            if (row_ok && vec_ok && k + 4 <= p.rows) {
                trsm_cp_async16(dst, src);
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (row_ok && k + q < p.rows) trsm_cp_async4(dst + q, src + q);
                    else dst[q] = 0.f;
                }
            }
        }
        trsm_cp_async_commit();
    }

    // right-hand side of the tile: B_ii - Xa, Xa = the partial-sum planes in increasing level.  A thread holds all its
    // rows (of one column) at once, so that the loads of a whole plane -- two planes at a time -- are in flight
    // together: the planes come from DRAM, and this prologue is all latency.
    {
        constexpr int RPT = TRSM_T_MAX / (TRSM_WARPS * G);  // rows per thread: row (TRSM_WARPS * i + warp) * G + lane / CW
        const int rsub = warp * G + lane / CW;
        float v[RPT], xa[RPT];
        unsigned okm = 0;
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            const int r = TRSM_WARPS * G * i + rsub;
            const bool ok = r < p.rows && col_ok;
            okm |= static_cast<unsigned>(ok) << i;
            v[i] = ok ? __ldg(p.B + r * p.b_r + c * p.b_c) : 0.f;
            xa[i] = 0.f;
        }
        const long long wcol = c * p.w_c;
        unsigned mk = p.mask;
        while (mk) {
            const int l0 = __ffs(mk) - 1;
            mk &= mk - 1;
            const int l1 = mk ? __ffs(mk) - 1 : -1;
            if (l1 >= 0) mk &= mk - 1;
            const float* W0 = p.W + l0 * p.plane + wcol;
            const float* W1 = p.W + (l1 >= 0 ? l1 : l0) * p.plane + wcol;
            float w0[RPT], w1[RPT];
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const bool ok = (okm >> i) & 1u;
                const long long at = (TRSM_WARPS * G * i + rsub) * p.w_r;
                w0[i] = ok ? __ldg(W0 + at) : 0.f;
                w1[i] = (ok && l1 >= 0) ? __ldg(W1 + at) : 0.f;
            }
#pragma unroll
            for (int i = 0; i < RPT; ++i) xa[i] = (xa[i] + w0[i]) + w1[i];
        }
#pragma unroll
        for (int i = 0; i < RPT; ++i) Xs[TRSM_WARPS * G * i + rsub][lane % CW] = v[i] - xa[i];
    }

    // Diagonal block s prepared for the column sweep: every row r scaled by 1 / L_rr (so that the sweep needs no
    // multiplication by the reciprocal inside its dependent chain), strictly lower part, transposed; dinv = 1 / L_rr.
    // Done by the upper half of the warps.
    auto build_lt = [&](int s) {
        if (warp < TRSM_WARPS / 2) return;
        const float* d = Lb + trsm_block(s, s);
        const int k = lane;
        float diag[4], low[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {  // rows (warp - 8) + 8 i: one row per warp and pass, lane = column
            const int r = warp - TRSM_WARPS / 2 + (TRSM_WARPS / 2) * i;
            diag[i] = d[r * TRSM_SB + r];
            low[i] = d[r * TRSM_SB + k];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = warp - TRSM_WARPS / 2 + (TRSM_WARPS / 2) * i;
            const float rinv = (s * TRSM_SB + r < p.rows) ? 1.0f / diag[i] : 1.0f;
            Lt[k][r] = (r > k) ? low[i] * rinv : 0.f;
            if (k == 0) dinv[r] = rinv;
        }
    };

    trsm_wait_pending(nsb - 1);  // column block 0 (this thread's copies; the barrier below covers the other threads')
    __syncthreads();
    build_lt(0);
    __syncthreads();

    for (int s = 0; s < nsb; ++s) {
        const int s0 = s * TRSM_SB;
        if (warp < CW / 8) {
            // ---- solve(s): x_r = (s_r - sum_{k<r} L_rk x_k) / L_rr evaluated as s_r/L_rr - sum_k (L_rk/L_rr) x_k.
            // ---- Four warps, one per scheduler, eight columns each; a column is shared by four lanes that hold eight
            // ---- consecutive rows each, so a step of the sweep is one shuffle (x_k from the lane that owns row k)
            // ---- and eight multiply-adds per lane -- a quarter of the instructions a single warp would issue, and
            // ---- the dependent chain of 32 steps is the shuffle and one multiply-add long.  The multipliers of step
            // ---- k + 4 are fetched while step k is applied: the other warps keep shared memory busy.
            const int cl = 8 * warp + (lane >> 2), q = lane & 3;   // column of the CTA's 32; row group
            constexpr int AHEAD = 4;
            float sv[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) sv[i] = Xs[s0 + 8 * q + i][cl] * dinv[8 * q + i];
            float4 la[AHEAD][2];   // Lt[k][8 q .. 8 q + 7] for the next steps
#pragma unroll
            for (int a = 0; a < AHEAD; ++a) {
                la[a][0] = *reinterpret_cast<const float4*>(&Lt[a][8 * q]);
                la[a][1] = *reinterpret_cast<const float4*>(&Lt[a][8 * q + 4]);
            }
#pragma unroll
            for (int k = 0; k < TRSM_SB; ++k) {
                const float4 l0 = la[k % AHEAD][0], l1 = la[k % AHEAD][1];
                if (k + AHEAD < TRSM_SB) {
                    la[k % AHEAD][0] = *reinterpret_cast<const float4*>(&Lt[k + AHEAD][8 * q]);
                    la[k % AHEAD][1] = *reinterpret_cast<const float4*>(&Lt[k + AHEAD][8 * q + 4]);
                }
                const float xk = __shfl_sync(0xffffffffu, sv[k & 7], (lane & ~3) | (k >> 3));
                // only rows r > k take part (a finished row must not meet an infinite or NaN x_k): all eight rows of
                // the lanes past the owner of row k, the rows after it in the owner itself
                const bool past = q > (k >> 3), from = q >= (k >> 3);
                const float lv[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (i > (k & 7) ? from : past) sv[i] = fmaf(-lv[i], xk, sv[i]);
            }
            const int cx = blockIdx.x * CW + cl;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = s0 + 8 * q + i;
                Xs[r][cl] = sv[i];
                if (r < p.rows && cx < p.m) p.X[r * p.x_r + cx * p.x_c] = sv[i];
            }
        } else if (warp >= 4 && s >= 1 && s + 1 < nsb) {
            // ---- trailing(s): rows below sub-block s, sixteen per warp at a time, with x of sub-block s-1: the other
            // ---- twelve warps
            const int tasks = (nsb - s - 1) * (TRSM_SB / 16);
            for (int g = warp - 4; g < tasks; g += 12) {
                const int t = s0 + TRSM_SB + 16 * g;  // first tile row of the task
                trsm_apply<16, CW>(Lb + trsm_block(t >> 5, s - 1) + (t & 31) * TRSM_SB, &Xs[s0 - TRSM_SB], &Xs[t], lane);
            }
        }
        if (s + 1 < nsb) trsm_wait_pending(nsb - 2 - s);  // column block s+1
        __syncthreads();  // x of sub-block s final; rows below it carry every update up to x of s-1
        if (s + 1 < nsb) {
            // ---- next(s+1): the 32 rows of the next sub-block with x of sub-block s (four rows per lane: eight warps with
            // ---- 32 columns, two with 8 -- this step is on the critical path, so it is spread thin); its triangle is
            // ---- prepared by warps 8-15 meanwhile
            constexpr int NR = 4 * G;   // rows per warp: four per lane
            if (warp < TRSM_SB / NR)
                trsm_apply<NR, CW>(Lb + trsm_block(s + 1, s) + (NR * warp) * TRSM_SB, &Xs[s0], &Xs[s0 + TRSM_SB + NR * warp], lane);
            build_lt(s + 1);
            __syncthreads();
        }
    }
}

}  // namespace cyc
