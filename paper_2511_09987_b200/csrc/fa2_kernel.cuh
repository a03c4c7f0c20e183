// FlashAttention-2 recurrence (Section "Simulated Cholesky and Flash Attention"):
//
//   S_{i,J_t} = alpha Q_i K_{J_t}^T,  mh = max(m, max S),  l <- e^{m-mh} l + sum_j e^{S_ij-mh},
//   o <- e^{m-mh} o + sum_j e^{S_ij-mh} V_j,  m <- mh,   O_i = o / l,     alpha = 1/sqrt(d)
//
// The paper assigns one query tile to one processing element, which alternates matrix products with elementwise
// updates of its own state.  Here that element is a CTA: it keeps a 128-row query tile in shared memory for its whole
// life and walks the key tiles J_t (128 keys each):
//   warp 0      TMA producer: Q once, then K_t and V_t into two buffers each (K_t is released as soon as S_t is done)
//   warp 1      one thread issues tcgen05 MMAs:  S_t = Q K_t^T  (fp32, in tensor memory, two buffers) and
//               U_t = P_t V_t (fp32, tensor memory, two buffers), P_t = e^{S_t - mh} in bf16 read from TENSOR memory:
//               the row threads write P_t over the first 64 columns of the buffer S_t came in ("in place"), so P is
//               double-buffered with S and never passes through shared memory
//   warps 2-9   two threads per query row (= one TMEM lane; warps 2-5 take keys 0-63 of the tile and the first half of
//               the d columns, warps 6-9 the rest): running maximum (the two partial maxima meet through shared memory),
//               P_t, partial normaliser, and the running output o <- e^{m-mh} o + U_t in registers
// S_{t+1} is issued before U_t, so the tensor core works on the next scores while the row threads exponentiate, and
// the exponentials of tile t do not wait for the product of tile t-1.
// Exponentials are 2^x on the scores scaled by alpha*log2(e).  bf16 inputs, fp32 output.  Every wait is bounded.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ptx.cuh"
#include "umma_kernel.cuh"

namespace cyc {

constexpr int FA2_THREADS = 320, FA2_BM = 128, FA2_BN = 128;

struct Fa2Params {
    float* O;          // [batch][N][D] fp32
    int N, M;          // queries, keys
    int tiles_q;       // ceil(N / 128)
    float scale_log2;  // alpha * log2(e)
    int* status;       // device status word
};

struct Fa2Ctl {
    uint64_t q_full;
    uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];
    uint64_t s_full[2], sp_free[2];   // scores ready / buffer free again (its P has been consumed)
    uint64_t p_ready[2], pv_done[2];  // P written over the scores / U complete
    uint32_t tmem_base;
    volatile int abort;
    float row_max[2][2][FA2_BM];  // [tile parity][half][row]: partial maxima of the two threads of a row
    float row_sum[2][FA2_BM];     // [half][row]: partial normalisers, exchanged once at the end
};

template <int D>
struct Fa2Smem {
    static constexpr int SLAB = 128 * 128;            // 128 rows x 128 bytes (64 bf16)
    static constexpr int Q_BYTES = (D / 64) * SLAB;   // K-major A operand of S
    static constexpr int K_BYTES = (D / 64) * SLAB;   // K-major B operand of S
    static constexpr int V_BYTES = (D / 64) * SLAB;   // MN-major B operand of U: D/64 chunks of 128 keys x 128 bytes of d
    static constexpr int STAGE_BYTES = K_BYTES + V_BYTES;
    static constexpr int TOTAL = Q_BYTES + 2 * STAGE_BYTES + 4096 + 1024;  // + control block + alignment slack
};

__device__ __forceinline__ bool fa2_wait(uint64_t* bar, uint32_t parity, Fa2Ctl* ctl, int* status, int where) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (ctl->abort) return false;
        if (clock64() - t0 > UMMA_WAIT_CYCLES) {
            ctl->abort = 1;
            atomicExch(status, 0x300 | where);
            return false;
        }
    }
    return true;
}

__device__ __forceinline__ float fa2_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// D[tmem] (+)= A[tmem] * B[smem], bf16 operands, one CTA
__device__ __forceinline__ void fa2_umma_tmem_a(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns from registers: thread t of the warp writes lane (base_lane + t)
__device__ __forceinline__ void fa2_tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
        "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
        "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void fa2_tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <int D>
__global__ void __launch_bounds__(FA2_THREADS, 1)
fa2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
           const Fa2Params p) {
    using Sm = Fa2Smem<D>;
    static_assert(D == 64 || D == 128, "head dimension 64 or 128");
    constexpr uint32_t TMEM_COLS = 512;                 // S0 | S1 | U0 | U1  (128 + 128 + D + D columns)
    constexpr uint32_t COL_S0 = 0, COL_U = 256;
    constexpr uint32_t IDESC_S = umma_instr_desc(1, 1, false, FA2_BM, FA2_BN);
    constexpr uint32_t IDESC_U = umma_instr_desc(1, 1, true, FA2_BM, D);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* sQ = smem;
    uint8_t* sKV = sQ + Sm::Q_BYTES;
    Fa2Ctl* ctl = reinterpret_cast<Fa2Ctl*>(sKV + 2 * Sm::STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x / p.tiles_q, qt = blockIdx.x - b * p.tiles_q;
    const int n0 = qt * FA2_BM;
    const int T = (p.M + FA2_BN - 1) / FA2_BN;  // key tiles

    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) {
        ptx::mbar_init(&ctl->q_full, 1);
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&ctl->k_full[s], 1);
            ptx::mbar_init(&ctl->k_empty[s], 1);
            ptx::mbar_init(&ctl->v_full[s], 1);
            ptx::mbar_init(&ctl->v_empty[s], 1);
            ptx::mbar_init(&ctl->s_full[s], 1);
            ptx::mbar_init(&ctl->sp_free[s], 1);
            ptx::mbar_init(&ctl->p_ready[s], 8);
            ptx::mbar_init(&ctl->pv_done[s], 1);
        }
        ctl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmQ);
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmV);
    }
    if (warp == 1) {
        ptx::tmem_alloc<1>(&ctl->tmem_base, TMEM_COLS);
        ptx::tmem_relinquish<1>();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::grid_dependency_wait();  // the set-up above may overlap the previous kernel; nothing it wrote is read before it ends
            ptx::mbar_arrive_expect_tx(&ctl->q_full, Sm::Q_BYTES);
#pragma unroll
            for (int kb = 0; kb < D / 64; ++kb) ptx::tma_load_3d(sQ + kb * Sm::SLAB, &tmQ, &ctl->q_full, kb * 64, n0, b);
            // K_t is free again as soon as S_t has been computed, V_t only after U_t: separate barriers, so that the
            // next keys are on their way one whole tile earlier than the next values
            int issued_k = 0, issued_v = 0;
            bool ok = true;
            for (int t = 0; t < T; ++t) {
                const int st = t & 1;
                const uint32_t ph = (t >> 1) & 1;
                uint8_t* sK = sKV + st * Sm::STAGE_BYTES;
                uint8_t* sV = sK + Sm::K_BYTES;
                if (!fa2_wait(&ctl->k_empty[st], ph ^ 1, ctl, p.status, 1)) { ok = false; break; }
                ptx::mbar_arrive_expect_tx(&ctl->k_full[st], Sm::K_BYTES);
#pragma unroll
                for (int kb = 0; kb < D / 64; ++kb)
                    ptx::tma_load_3d(sK + kb * Sm::SLAB, &tmK, &ctl->k_full[st], kb * 64, t * FA2_BN, b);  // keys x 64 of d
                ++issued_k;
                if (!fa2_wait(&ctl->v_empty[st], ph ^ 1, ctl, p.status, 8)) { ok = false; break; }
                ptx::mbar_arrive_expect_tx(&ctl->v_full[st], Sm::V_BYTES);
#pragma unroll
                for (int kb = 0; kb < D / 64; ++kb)
                    ptx::tma_load_3d(sV + kb * Sm::SLAB, &tmV, &ctl->v_full[st], kb * 64, t * FA2_BN, b);  // keys x d-chunk kb
                ++issued_v;
            }
            if (!ok) {
                // leave no copy in flight: wait (bounded) for the loads already issued
                const long long t0 = clock64();
                while (!ptx::mbar_try_wait(&ctl->q_full, 0) && clock64() - t0 < UMMA_WAIT_CYCLES) {}
                for (int u = issued_k - 1; u >= 0 && u >= issued_k - 2; --u) {
                    const long long t1 = clock64();
                    while (!ptx::mbar_try_wait(&ctl->k_full[u & 1], (u >> 1) & 1) && clock64() - t1 < UMMA_WAIT_CYCLES) {}
                }
                for (int u = issued_v - 1; u >= 0 && u >= issued_v - 2; --u) {
                    const long long t1 = clock64();
                    while (!ptx::mbar_try_wait(&ctl->v_full[u & 1], (u >> 1) & 1) && clock64() - t1 < UMMA_WAIT_CYCLES) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t aQ = ptx::smem_u32(sQ);
            bool ok = fa2_wait(&ctl->q_full, 0, ctl, p.status, 2);
            // U_u = P_u V_u : A = P in tensor memory (row = lane, two keys per 32-bit column, 16 keys = 8 columns per
            // MMA), B = V (MN-major: 128-byte rows of d, 8-key groups 1024 B apart, next 64 columns of d one slab on)
            auto issue_u = [&](int u) -> bool {
                const int su = u & 1;
                const uint32_t pu = (u >> 1) & 1;
                if (!fa2_wait(&ctl->v_full[su], pu, ctl, p.status, 9)) return false;
                if (!fa2_wait(&ctl->p_ready[su], pu, ctl, p.status, 3)) return false;
                ptx::tc_fence_after();
                const uint32_t aV = ptx::smem_u32(sKV + su * Sm::STAGE_BYTES + Sm::K_BYTES);
#pragma unroll
                for (int k = 0; k < FA2_BN / 16; ++k) {
                    const uint64_t bdesc = umma_smem_desc(aV + k * (16 * 128), Sm::SLAB, 1024);
                    fa2_umma_tmem_a(tmem_base + COL_U + su * D, tmem_base + COL_S0 + su * FA2_BN + k * 8, bdesc, IDESC_U, k != 0 ? 1u : 0u);
                }
                ptx::umma_commit(&ctl->pv_done[su]);
                ptx::umma_commit(&ctl->v_empty[su]);
                ptx::umma_commit(&ctl->sp_free[su]);
                return true;
            };
            for (int t = 0; t < T && ok; ++t) {
                const int st = t & 1;
                const uint32_t ph = (t >> 1) & 1;
                if (!fa2_wait(&ctl->k_full[st], ph, ctl, p.status, 4)) { ok = false; break; }
                if (!fa2_wait(&ctl->sp_free[st], ph ^ 1, ctl, p.status, 5)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t aK = ptx::smem_u32(sKV + st * Sm::STAGE_BYTES);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {  // S_t = Q K_t^T, both K-major
                    const uint32_t off = (k >> 2) * Sm::SLAB + (k & 3) * 32;
                    ptx::umma<KIND_BF16, 1>(tmem_base + COL_S0 + st * FA2_BN, umma_smem_desc(aQ + off, 16, 1024),
                                            umma_smem_desc(aK + off, 16, 1024), IDESC_S, k != 0 ? 1u : 0u);
                }
                ptx::umma_commit(&ctl->s_full[st]);
                ptx::umma_commit(&ctl->k_empty[st]);
                if (t > 0) ok = issue_u(t - 1);
            }
            if (ok) issue_u(T - 1);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ row threads: two per query row
        constexpr int HD = D / 2;               // d columns of the running output per thread
        constexpr int HN = FA2_BN / 2;          // keys of a tile per thread
        const int q = warp & 3;                 // TMEM lane quarter this warp may access
        const int half = (warp - 2) >> 2;       // 0: keys 0-63, d columns 0..HD ; 1: the rest
        const int r = q * 32 + lane;            // row of the query tile
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        float m = -INFINITY, l = 0.f, carry_prev = 0.f;
        float o[HD];
#pragma unroll
        for (int c = 0; c < HD; ++c) o[c] = 0.f;
        bool ok = true;
        // the two warps that share a lane quarter meet at a named barrier of their own
        auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + q) : "memory"); };
        // o <- carry o + U_u  (U_u complete in its tensor-memory buffer: pv_done[u & 1] has completed its phase)
        auto fold = [&](int u) {
            ptx::tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < HD; c0 += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(lane_addr + COL_U + (u & 1) * D + half * HD + c0, v);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int g = 0; g < 32; ++g) o[c0 + g] = fmaf(o[c0 + g], carry_prev, __uint_as_float(v[g]));
            }
        };
        // Both threads of a row pass the named barrier exactly once per key tile and once after the loop, whatever
        // happens: a thread whose wait ran out keeps walking the loop (doing nothing else) so that its partner is never
        // left alone at the barrier.
        for (int t = 0; t < T; ++t) {
            const int st = t & 1;
            if (ok) ok = fa2_wait(&ctl->s_full[st], (t >> 1) & 1, ctl, p.status, 7);
            ptx::tc_fence_after();
            const uint32_t s_addr = lane_addr + COL_S0 + st * FA2_BN + half * HN;
            const int valid = min(FA2_BN, p.M - t * FA2_BN) - half * HN;  // keys of this thread's half that exist
            // this thread's 64 scores: with the short running output (d = 64) they stay in registers from the maximum
            // to the exponentials; with the long one (d = 128) they pass through 32 registers, the first 32 read twice
            constexpr bool KEEP = (D == 64);
            uint32_t sc[HN];  // scores (KEEP) / the packed exponentials in its first half
            uint32_t tmp[KEEP ? 1 : 32];
            float mx = -INFINITY;
            if (ok) {
                if constexpr (KEEP) {
                    ptx::tmem_ld_32x32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
                    ptx::tmem_ld_32x32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sc[32]));
                    ptx::tmem_ld_wait();
                    if (valid < HN) {  // only the last tile can be ragged
#pragma unroll
                        for (int g = 0; g < HN; ++g)
                            if (g >= valid) sc[g] = 0xff800000u;  // a key that does not exist: -inf, weight 0
                    }
#pragma unroll
                    for (int g = 0; g < HN; ++g) mx = fmaxf(mx, __uint_as_float(sc[g]));
                } else {
#pragma unroll
                    for (int c0 = 0; c0 < HN; c0 += 32) {
                        ptx::tmem_ld_32x32(s_addr + c0, *reinterpret_cast<uint32_t(*)[32]>(&tmp[0]));
                        ptx::tmem_ld_wait();
                        if (valid < HN) {
#pragma unroll
                            for (int g = 0; g < 32; ++g)
                                if (c0 + g >= valid) tmp[g] = 0xff800000u;
                        }
#pragma unroll
                        for (int g = 0; g < 32; ++g) mx = fmaxf(mx, __uint_as_float(tmp[g]));
                    }
                }
            }
            ctl->row_max[st][half][r] = mx;
            pair_sync();
            if (ctl->abort) ok = false;
            if (!ok) continue;
            mx = fmaxf(mx, ctl->row_max[st][half ^ 1][r]);
            const float m_new = fmaxf(m, mx * p.scale_log2);
            const float carry = fa2_exp2(m - m_new);  // 2^(-inf) = 0 on the first tile
            // P_t = 2^(S scale - m_new) as bf16, two keys per 32-bit word (the lower key in the lower half), row sum in fp32
            float lsum = 0.f;
            if constexpr (KEEP) {
#pragma unroll
                for (int g = 0; g < HN; g += 2) {
                    const float p0 = fa2_exp2(fmaf(__uint_as_float(sc[g]), p.scale_log2, -m_new));
                    const float p1 = fa2_exp2(fmaf(__uint_as_float(sc[g + 1]), p.scale_log2, -m_new));
                    lsum += p0 + p1;
                    __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                    sc[g >> 1] = *reinterpret_cast<uint32_t*>(&h);  // word g/2 <= g: nothing still needed is overwritten
                }
            } else {
                // the scores of keys 32-63 are still in `tmp` from the pass for the maximum: they go first, and only
                // keys 0-31 are read from tensor memory a second time
#pragma unroll
                for (int c0 = HN - 32; c0 >= 0; c0 -= 32) {
                    if (c0 != HN - 32) {
                        ptx::tmem_ld_32x32(s_addr + c0, *reinterpret_cast<uint32_t(*)[32]>(&tmp[0]));
                        ptx::tmem_ld_wait();
                        if (valid < HN) {
#pragma unroll
                            for (int g = 0; g < 32; ++g)
                                if (c0 + g >= valid) tmp[g] = 0xff800000u;
                        }
                    }
#pragma unroll
                    for (int g = 0; g < 32; g += 2) {
                        const float p0 = fa2_exp2(fmaf(__uint_as_float(tmp[g]), p.scale_log2, -m_new));
                        const float p1 = fa2_exp2(fmaf(__uint_as_float(tmp[g + 1]), p.scale_log2, -m_new));
                        lsum += p0 + p1;
                        __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                        sc[(c0 + g) >> 1] = *reinterpret_cast<uint32_t*>(&h);
                    }
                }
                // No second barrier: P goes to columns 0-63 of the buffer.  Columns 32-63 held this row's scores of
                // keys 32-63, which their owner (half 0) took from registers above; the scores read a second time sit
                // in columns 0-31 (half 0, overwritten only by its own store below) and 64-95 (half 1, never overwritten).
            }
            l = fmaf(l, carry, lsum);
            m = m_new;
            // over the first 64 columns of the buffer the scores came in: keys 64 half .. + 63 are columns 32 half .. + 31
            fa2_tmem_st_32x32(lane_addr + COL_S0 + st * FA2_BN + half * (HN / 2), *reinterpret_cast<uint32_t(*)[32]>(&sc[0]));
            fa2_tmem_st_wait();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->p_ready[st]);
            // with P_t handed over, fold the previous tile's product (in the other U buffer) into the running output
            if (t > 0) {
                if (!fa2_wait(&ctl->pv_done[(t - 1) & 1], ((t - 1) >> 1) & 1, ctl, p.status, 6)) { ok = false; continue; }
                fold(t - 1);
            }
            carry_prev = carry;
        }
        if (ok) ok = fa2_wait(&ctl->pv_done[(T - 1) & 1], ((T - 1) >> 1) & 1, ctl, p.status, 10);
        if (ok) fold(T - 1);
        // the normaliser of a row is the sum of its two partial ones
        ctl->row_sum[half][r] = l;
        pair_sync();
        if (ok && !ctl->abort && n0 + r < p.N) {
            const float inv = 1.0f / (l + ctl->row_sum[half ^ 1][r]);
            float* dst = p.O + (static_cast<long long>(b) * p.N + n0 + r) * D + half * HD;
#pragma unroll
            for (int c = 0; c < HD; c += 4)
                *reinterpret_cast<float4*>(dst + c) = make_float4(o[c] * inv, o[c + 1] * inv, o[c + 2] * inv, o[c + 3] * inv);
        }
        ptx::tc_fence_before();
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc<1>(tmem_base, TMEM_COLS);
    }
}

}  // namespace cyc
