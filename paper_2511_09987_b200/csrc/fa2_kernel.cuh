// FlashAttention-2 recurrence (Section "Simulated Cholesky and Flash Attention"):
//
//   S_{i,J_t} = alpha Q_i K_{J_t}^T,  mh = max(m, max S),  l <- e^{m-mh} l + sum_j e^{S_ij-mh},
//   o <- e^{m-mh} o + sum_j e^{S_ij-mh} V_j,  m <- mh,   O_i = o / l,     alpha = 1/sqrt(d)
//
// The paper assigns a query tile to a processing element, which alternates matrix products with elementwise updates
// of its own state.  Here a CTA owns TWO 128-row query tiles of one problem and walks the key tiles J_t (128 keys
// each) once for both, so that the tensor core always has the other tile's product to run while one tile's rows
// exponentiate, and K_t / V_t are fetched once for 256 queries:
//   warps 0-3, 4-7  row threads of query tile 0 / 1: one thread per query row (= one TMEM lane).  Per key tile: running
//                   maximum, P_t = e^{S_t - m} as bf16 written over the first 64 columns of the buffer S_t came in,
//                   partial normaliser l.
//   warps 8-11      output keepers: the running output o lives in tensor memory and the second product accumulates
//                   into it in place; when a row's maximum has grown, its keeper thread rescales the row of o before
//                   the product of that key tile is issued; after the last key tile they write O = o / l.
//   warp 12         TMA producer: both Q tiles once, then K_t and V_t into two buffers each.
//   warp 13         one thread issues the tcgen05 MMAs, in the order  U0_t, S0_{t+1}, U1_t, S1_{t+1}  (U = P V).
// The maximum a row's exponentials refer to is only moved when the true running maximum exceeds it by more than 2^8:
// the recurrence's result does not depend on which reference is used (the same factor multiplies o and l), the
// exponentials stay below 2^8 in bf16 / fp32, and the rescale of o, a read-modify-write of tensor memory, becomes rare.
// Exponentials are 2^x on the scores scaled by alpha*log2(e).  bf16 inputs, fp32 output.  Every wait is bounded.
//
// Sliced tail.  The grid's last, partial round of CTAs would leave most SMs idle for a whole pass over the keys.  The
// host may therefore cut each (problem, 256 queries) unit of that round into 2 to 4 parts by key range, one CTA each.
// A part keeps its own (m, l, o); the recurrence is associative in these triples,
//   (m, l, o) = (max(m_a, m_b), l_a 2^(m_a-m) + l_b 2^(m_b-m), o_a 2^(m_a-m) + o_b 2^(m_b-m)),
// so each warp of row threads writes its 32 rows' triple to scratch, counts itself in, and the last part to arrive for
// those rows folds all parts together in part order (the same bits whichever part arrives last) and writes O.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ptx.cuh"
#include "umma_kernel.cuh"

namespace cyc {

constexpr int FA2_THREADS = 512, FA2_BM = 128, FA2_BN = 128;
constexpr int FA2_ROWS = 2 * FA2_BM;        // query rows per CTA
constexpr float FA2_RESCALE_LOG2 = 8.0f;    // the reference maximum of a row moves only when it is exceeded by more than 2^8

struct Fa2Params {
    float* O;          // [batch][N][D] fp32
    int N, M;          // queries, keys
    int tiles_q;       // ceil(N / 256)
    float scale_log2;  // alpha * log2(e)
    int* status;       // device status word
    // sliced tail: CTAs [0, full_units) take a whole unit each; after them come tail_parts CTAs per remaining unit
    int full_units;      // = batch * tiles_q when there is no tail
    int tail_parts;      // 0 (no tail) or 2..4
    float* tail_ws;      // [tail unit][part][query tile][row warp] slots of fa2_tail_slot_floats(D) floats
    int* tail_counters;  // [tail unit][query tile][warp], zero between launches
};
constexpr int FA2_TAIL_MAX_PARTS = 4;
// the partial state of one warp's 32 rows: 32 x D of o, then 32 m, then 32 l
__host__ __device__ constexpr int fa2_tail_slot_floats(int d) { return 32 * d + 64; }

struct Fa2Ctl {
    uint64_t q_full;
    uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];
    // per query tile: scores ready / P written / rescale decided / o ready for the product / product done / l final
    uint64_t s_full[2], p_ready[2], corr_req[2], o_ready[2], pv_done[2], l_done[2];
    uint32_t tmem_base;
    volatile int abort;
    int need[2][4];            // [query tile][warp]: some row of the warp asks for a rescale at this key tile
    float factor[2][FA2_BM];   // [query tile][row]: what to multiply the row of o by
    float row_l[2][FA2_BM];    // [query tile][row]: final normaliser
};

template <int D>
struct Fa2Smem {
    static constexpr int SLAB = 128 * 128;            // 128 rows x 128 bytes (64 bf16)
    static constexpr int Q_BYTES = (D / 64) * SLAB;   // one query tile, K-major A operand of S
    static constexpr int K_BYTES = (D / 64) * SLAB;   // K-major B operand of S
    static constexpr int V_BYTES = (D / 64) * SLAB;   // MN-major B operand of U: D/64 chunks of 128 keys x 128 bytes of d
    static constexpr int STAGE_BYTES = K_BYTES + V_BYTES;
    static constexpr int TOTAL = 2 * Q_BYTES + 2 * STAGE_BYTES + 4096 + 1024;  // + control block + alignment slack
};
static_assert(sizeof(Fa2Ctl) <= 4096, "control block");

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
__device__ __forceinline__ void fa2_umma_tmem_a(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate, uint32_t leader) {
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "setp.ne.b32 q, %5, 0;\n"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(leader)
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

// Register split.  The block is launched with 512 x 128 registers; the four warps that hold the producer and the MMA
// issuer drop to 64 each and the keepers to 96, which lets the two groups of row threads grow to 176:
// 2 * 128 * 176 + 128 * 96 + 128 * 64 = 65536 (no spills with this split).  (A split that asked for more than the launch holds would wait forever;
// the host refuses to launch if the kernel was not compiled to 128 registers per thread.)
constexpr int FA2_REGS_ROW = 176, FA2_REGS_KEEPER = 96, FA2_REGS_OTHER = 64, FA2_REGS_LAUNCH = 128;
static_assert(FA2_REGS_ROW % 8 == 0 && FA2_REGS_KEEPER % 8 == 0 && FA2_REGS_OTHER % 8 == 0, "setmaxnreg takes multiples of 8");
static_assert(2 * 128 * FA2_REGS_ROW + 128 * FA2_REGS_KEEPER + 128 * FA2_REGS_OTHER <= FA2_THREADS * FA2_REGS_LAUNCH, "register split");
template <int N>
__device__ __forceinline__ void fa2_regs_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void fa2_regs_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
__device__ __forceinline__ float fa2_max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

template <int D>
__global__ void __launch_bounds__(FA2_THREADS, 1)
fa2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
           const Fa2Params p) {
    using Sm = Fa2Smem<D>;
    static_assert(D == 64 || D == 128, "head dimension 64 or 128");
    constexpr uint32_t TMEM_COLS = 512;                 // S0 | S1 | o0 | o1  (128 + 128 + D + D columns)
    constexpr uint32_t COL_S = 0, COL_O = 256;
    constexpr uint32_t IDESC_S = umma_instr_desc(1, 1, false, FA2_BM, FA2_BN);
    constexpr uint32_t IDESC_U = umma_instr_desc(1, 1, true, FA2_BM, D);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* sQ = smem;                       // two query tiles
    uint8_t* sKV = sQ + 2 * Sm::Q_BYTES;
    Fa2Ctl* ctl = reinterpret_cast<Fa2Ctl*>(sKV + 2 * Sm::STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // which unit (problem, 256 queries) and which key tiles [kt0, kt0 + T) of it this CTA walks
    int unit = blockIdx.x, part = -1, kt0 = 0;
    int T = (p.M + FA2_BN - 1) / FA2_BN;
    if (static_cast<int>(blockIdx.x) >= p.full_units) {
        const int x = blockIdx.x - p.full_units;
        unit = p.full_units + x / p.tail_parts;
        part = x - (unit - p.full_units) * p.tail_parts;
        kt0 = static_cast<int>(static_cast<long long>(T) * part / p.tail_parts);
        T = static_cast<int>(static_cast<long long>(T) * (part + 1) / p.tail_parts) - kt0;
    }
    const int b = unit / p.tiles_q, qt = unit - b * p.tiles_q;
    const int n0 = qt * FA2_ROWS;
    const int ntq = (n0 + FA2_BM < p.N) ? 2 : 1;        // query tiles of this CTA that hold rows of the problem

    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) {
        ptx::mbar_init(&ctl->q_full, 1);
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&ctl->k_full[s], 1);
            ptx::mbar_init(&ctl->k_empty[s], 1);
            ptx::mbar_init(&ctl->v_full[s], 1);
            ptx::mbar_init(&ctl->v_empty[s], 1);
            ptx::mbar_init(&ctl->s_full[s], 1);
            ptx::mbar_init(&ctl->p_ready[s], 4);
            ptx::mbar_init(&ctl->corr_req[s], 4);
            ptx::mbar_init(&ctl->o_ready[s], 4);
            ptx::mbar_init(&ctl->pv_done[s], 1);
            ptx::mbar_init(&ctl->l_done[s], 4);
        }
        ctl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmQ);
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmV);
    }
    if (warp == 13) {
        ptx::tmem_alloc<1>(&ctl->tmem_base, TMEM_COLS);
        ptx::tmem_relinquish<1>();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp >= 12) {
      fa2_regs_dec<FA2_REGS_OTHER>();
      if (warp == 12) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            ptx::grid_dependency_wait();  // the set-up above may overlap the previous kernel; nothing it wrote is read before it ends
            ptx::mbar_arrive_expect_tx(&ctl->q_full, ntq * Sm::Q_BYTES);
            for (int i = 0; i < ntq; ++i)
#pragma unroll
                for (int kb = 0; kb < D / 64; ++kb)
                    ptx::tma_load_3d(sQ + i * Sm::Q_BYTES + kb * Sm::SLAB, &tmQ, &ctl->q_full, kb * 64, n0 + i * FA2_BM, b);
            // K_t is free again as soon as the scores of both query tiles have been computed, V_t only after both
            // second products: separate barriers, so that the next keys are on their way one tile earlier
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
                    ptx::tma_load_3d(sK + kb * Sm::SLAB, &tmK, &ctl->k_full[st], kb * 64, (kt0 + t) * FA2_BN, b);  // keys x 64 of d
                ++issued_k;
                if (!fa2_wait(&ctl->v_empty[st], ph ^ 1, ctl, p.status, 8)) { ok = false; break; }
                ptx::mbar_arrive_expect_tx(&ctl->v_full[st], Sm::V_BYTES);
#pragma unroll
                for (int kb = 0; kb < D / 64; ++kb)
                    ptx::tma_load_3d(sV + kb * Sm::SLAB, &tmV, &ctl->v_full[st], kb * 64, (kt0 + t) * FA2_BN, b);  // keys x d-chunk kb
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
      } else if (warp == 13) {
        // ------------------------------------------------------------ MMA issuer: the whole warp walks the loop (waits
        // ------------------------------------------------------------ included), one elected lane issues
        {
            const uint32_t leader = ptx::elect_one();
            bool ok = fa2_wait(&ctl->q_full, 0, ctl, p.status, 2);
            // The issuing thread shares its scheduler with busy row warps, and an MMA of this size runs for only 64 clocks:
            // every instruction between two MMAs counts.  Descriptors are built once; a k-step only adds its byte offset
            // (in 16-byte units) to the address field, which cannot carry out of its 14 bits below 256 KB.
            uint64_t dQ[2], dK[2], dV[2];
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                dQ[x] = umma_smem_desc(ptx::smem_u32(sQ + x * Sm::Q_BYTES), 16, 1024);
                dK[x] = umma_smem_desc(ptx::smem_u32(sKV + x * Sm::STAGE_BYTES), 16, 1024);
                dV[x] = umma_smem_desc(ptx::smem_u32(sKV + x * Sm::STAGE_BYTES + Sm::K_BYTES), Sm::SLAB, 1024);
            }
            // S_i(t) = Q_i K_t^T, both operands K-major, into the score buffer of query tile i
            auto issue_s = [&](int i, int t) {
                const uint64_t q0 = dQ[i], k0 = dK[t & 1];
                const uint32_t d_s = tmem_base + COL_S + i * FA2_BN;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    constexpr uint32_t dummy = 0; (void)dummy;
                    const uint64_t off = static_cast<uint64_t>(((k >> 2) * Sm::SLAB + (k & 3) * 32) >> 4);
                    ptx::umma_elect<KIND_BF16>(d_s, q0 + off, k0 + off, IDESC_S, k != 0 ? 1u : 0u, leader);
                }
                ptx::umma_commit_elect(&ctl->s_full[i], leader);
            };
            // o_i (+)= P_i(t) V_t : A = P in tensor memory (row = lane, two keys per 32-bit column, 16 keys = 8 columns
            // per MMA), B = V (MN-major: 128-byte rows of d, 8-key groups 1024 B apart, next 64 columns of d one slab on)
            auto issue_u = [&](int i, int t) {
                const uint64_t v0 = dV[t & 1];
                const uint32_t d_o = tmem_base + COL_O + i * D, a_p = tmem_base + COL_S + i * FA2_BN;
#pragma unroll
                for (int k = 0; k < FA2_BN / 16; ++k)
                    fa2_umma_tmem_a(d_o, a_p + k * 8, v0 + static_cast<uint64_t>((k * 16 * 128) >> 4), IDESC_U, (t | k) != 0 ? 1u : 0u, leader);
                ptx::umma_commit_elect(&ctl->pv_done[i], leader);
            };
            if (ok) ok = fa2_wait(&ctl->k_full[0], 0, ctl, p.status, 4);
            if (ok) {
                ptx::tc_fence_after();
                for (int i = 0; i < ntq; ++i) issue_s(i, 0);
                ptx::umma_commit_elect(&ctl->k_empty[0], leader);
            }
            for (int t = 0; t < T && ok; ++t) {
                const int st = t & 1;
                if (!fa2_wait(&ctl->v_full[st], (t >> 1) & 1, ctl, p.status, 9)) { ok = false; break; }
                for (int i = 0; i < ntq && ok; ++i) {
                    if (!fa2_wait(&ctl->p_ready[i], t & 1, ctl, p.status, 3)) { ok = false; break; }
                    if (!fa2_wait(&ctl->o_ready[i], t & 1, ctl, p.status, 5)) { ok = false; break; }
                    ptx::tc_fence_after();
                    issue_u(i, t);
                    if (i == ntq - 1) ptx::umma_commit_elect(&ctl->v_empty[st], leader);
                    if (t + 1 < T) {
                        // the next scores of this query tile go to the buffer its P was just read from: the tensor core
                        // runs the MMAs of one thread in issue order
                        if (i == 0 && !fa2_wait(&ctl->k_full[(t + 1) & 1], ((t + 1) >> 1) & 1, ctl, p.status, 4)) { ok = false; break; }
                        ptx::tc_fence_after();
                        issue_s(i, t + 1);
                        if (i == ntq - 1) ptx::umma_commit_elect(&ctl->k_empty[(t + 1) & 1], leader);
                    }
                }
            }
        }
        __syncwarp();
      }
    } else if (warp < 8) {
        fa2_regs_inc<FA2_REGS_ROW>();
        // ------------------------------------------------------------ row threads: one per query row
        const int i = warp >> 2;                 // query tile
        const int q = warp & 3;                  // TMEM lane quarter this warp may access
        const int r = q * 32 + lane;             // row of the query tile
        if (i < ntq) {
            const uint32_t s_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + COL_S + i * FA2_BN;
            float m_ref = 0.f, l = 0.f;          // reference maximum of the exponentials (scaled, log2 units), normaliser
            bool ok = true;
            for (int t = 0; t < T && ok; ++t) {
                if (!fa2_wait(&ctl->s_full[i], t & 1, ctl, p.status, 7)) { ok = false; break; }
                ptx::tc_fence_after();
                const int valid = min(FA2_BN, p.M - (kt0 + t) * FA2_BN);  // keys of this tile that exist (< 128 only in the last)
                // ---- the row's 128 scores, read once and kept in registers from the maximum to the exponentials
                uint32_t v[FA2_BN];
#pragma unroll
                for (int c0 = 0; c0 < FA2_BN; c0 += 32) ptx::tmem_ld_32x32(s_addr + c0, *reinterpret_cast<uint32_t(*)[32]>(&v[c0]));
                ptx::tmem_ld_wait();
                if (valid < FA2_BN) {
#pragma unroll
                    for (int g = 0; g < FA2_BN; ++g)
                        if (g >= valid) v[g] = 0xff800000u;  // a key that does not exist: -inf, weight 0
                }
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;  // four chains of three-input maxima
#pragma unroll
                for (int g = 0; g < FA2_BN; g += 8) {
                    mx0 = fa2_max3(mx0, __uint_as_float(v[g]), __uint_as_float(v[g + 1]));
                    mx1 = fa2_max3(mx1, __uint_as_float(v[g + 2]), __uint_as_float(v[g + 3]));
                    mx2 = fa2_max3(mx2, __uint_as_float(v[g + 4]), __uint_as_float(v[g + 5]));
                    mx3 = fa2_max3(mx3, __uint_as_float(v[g + 6]), __uint_as_float(v[g + 7]));
                }
                const float m_t = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
                // ---- does the reference move?  (never at the first tile: o is overwritten there, not accumulated)
                float f = 1.0f;
                if (t == 0) {
                    m_ref = m_t;
                } else if (m_t > m_ref + FA2_RESCALE_LOG2) {
                    f = fa2_exp2(m_ref - m_t);
                    m_ref = m_t;
                    l *= f;
                }
                ctl->factor[i][r] = f;
                const unsigned any = __ballot_sync(0xffffffffu, f != 1.0f);
                if (lane == 0) {
                    ctl->need[i][q] = any != 0u;
                    ptx::mbar_arrive(&ctl->corr_req[i]);  // the keeper of these rows can start while the exponentials run
                }
                // ---- P_t = 2^(S scale - m_ref) as bf16, two keys per 32-bit word (the lower key in the lower half), packed
                // ---- in place (word g/2 <= g: nothing still needed is overwritten), row sum in fp32 on four chains; P goes
                // ---- over columns 0-63 of the score buffer
                float ls0 = 0.f, ls1 = 0.f, ls2 = 0.f, ls3 = 0.f;
#pragma unroll
                for (int g = 0; g < FA2_BN; g += 8) {
                    float e[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) e[u] = fa2_exp2(fmaf(__uint_as_float(v[g + u]), p.scale_log2, -m_ref));
                    ls0 += e[0] + e[1]; ls1 += e[2] + e[3]; ls2 += e[4] + e[5]; ls3 += e[6] + e[7];
#pragma unroll
                    for (int u = 0; u < 8; u += 2) {
                        __nv_bfloat162 hh = __floats2bfloat162_rn(e[u], e[u + 1]);
                        v[(g + u) >> 1] = *reinterpret_cast<uint32_t*>(&hh);
                    }
                }
                const float lsum = (ls0 + ls1) + (ls2 + ls3);
                fa2_tmem_st_32x32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                fa2_tmem_st_32x32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                l += lsum;
                fa2_tmem_st_wait();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctl->p_ready[i]);
            }
            if (part < 0) {
                ctl->row_l[i][r] = l;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctl->l_done[i]);
            } else if (ok && fa2_wait(&ctl->pv_done[i], (T - 1) & 1, ctl, p.status, 13)) {
                // ---- a part of a sliced unit: its (m, l, o) for these 32 rows go to scratch; the last part to arrive folds
                // ---- all parts in part order.  (The row threads do this, not the keepers: they are idle by now, both query
                // ---- tiles proceed at once, and they have the registers to keep a whole round of loads in flight.)
                ptx::tc_fence_after();
                const uint32_t o_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + COL_O + i * D;
                // slot of part k; within it piece j (four columns) of lane t sits at float (j * 32 + t) * 4, so that a warp
                // writes and reads 512 contiguous bytes at a time
                constexpr int SLOT = fa2_tail_slot_floats(D);
                const int tu = unit - p.full_units, w = i * 4 + q;
                float* slots = p.tail_ws + (static_cast<size_t>(tu) * p.tail_parts * 8 + w) * SLOT;
                float* mine = slots + static_cast<size_t>(part) * 8 * SLOT;
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t v[32];
                    ptx::tmem_ld_32x32(o_addr + c0, v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int g = 0; g < 32; g += 4)
                        *reinterpret_cast<float4*>(mine + (((c0 + g) >> 2) * 32 + lane) * 4) =
                            make_float4(__uint_as_float(v[g]), __uint_as_float(v[g + 1]), __uint_as_float(v[g + 2]), __uint_as_float(v[g + 3]));
                }
                mine[32 * D + lane] = m_ref;
                mine[32 * D + 32 + lane] = l;
                __threadfence();
                __syncwarp();
                int arrived = 0;
                if (lane == 0) arrived = atomicAdd(&p.tail_counters[tu * 8 + w], 1);
                arrived = __shfl_sync(0xffffffffu, arrived, 0);
                if (arrived == p.tail_parts - 1) {
                    if (lane == 0) p.tail_counters[tu * 8 + w] = 0;  // every part has arrived: zero again for the next launch
                    __threadfence();
                    float a[FA2_TAIL_MAX_PARTS], m = -INFINITY, lsum = 0.f;
#pragma unroll
                    for (int k = 0; k < FA2_TAIL_MAX_PARTS; ++k) {
                        a[k] = -INFINITY;
                        if (k < p.tail_parts) a[k] = __ldcg(slots + static_cast<size_t>(k) * 8 * SLOT + 32 * D + lane);
                        m = fmaxf(m, a[k]);
                    }
#pragma unroll
                    for (int k = 0; k < FA2_TAIL_MAX_PARTS; ++k) {
                        a[k] = fa2_exp2(a[k] - m);  // 0 for a part that does not exist
                        if (k < p.tail_parts)
                            lsum = __fadd_rn(lsum, __fmul_rn(__ldcg(slots + static_cast<size_t>(k) * 8 * SLOT + 32 * D + 32 + lane), a[k]));
                    }
                    const float inv = 1.0f / lsum;
                    const int row = n0 + i * FA2_BM + r;
                    float* dst = p.O + (static_cast<long long>(b) * p.N + row) * D;
#pragma unroll
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        float4 x[FA2_TAIL_MAX_PARTS][8];  // all loads of 32 columns in flight at once
#pragma unroll
                        for (int k = 0; k < FA2_TAIL_MAX_PARTS; ++k)
                            if (k < p.tail_parts) {
#pragma unroll
                                for (int g = 0; g < 8; ++g)
                                    x[k][g] = __ldcg(reinterpret_cast<const float4*>(slots + static_cast<size_t>(k) * 8 * SLOT + (((c0 >> 2) + g) * 32 + lane) * 4));
                            }
                        if (row < p.N) {
#pragma unroll
                            for (int g = 0; g < 8; ++g) {
                                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                                for (int k = 0; k < FA2_TAIL_MAX_PARTS; ++k)
                                    if (k < p.tail_parts) {
                                        acc.x = __fadd_rn(acc.x, __fmul_rn(x[k][g].x, a[k]));
                                        acc.y = __fadd_rn(acc.y, __fmul_rn(x[k][g].y, a[k]));
                                        acc.z = __fadd_rn(acc.z, __fmul_rn(x[k][g].z, a[k]));
                                        acc.w = __fadd_rn(acc.w, __fmul_rn(x[k][g].w, a[k]));
                                    }
                                *reinterpret_cast<float4*>(dst + c0 + g * 4) = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
                            }
                        }
                    }
                }
            }
        }
        ptx::tc_fence_before();
    } else {
        fa2_regs_dec<FA2_REGS_KEEPER>();
        // ------------------------------------------------------------ output keepers: one thread per row, both query tiles
        const int q = warp & 3;
        const int r = q * 32 + lane;
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + COL_O;
        bool ok = true;
        for (int t = 0; t < T && ok; ++t) {
            for (int i = 0; i < ntq; ++i) {
                if (!fa2_wait(&ctl->corr_req[i], t & 1, ctl, p.status, 6)) { ok = false; break; }
                if (ctl->need[i][q]) {  // uniform over the warp
                    // the product of the previous key tile must have landed before the row is touched
                    if (!fa2_wait(&ctl->pv_done[i], (t - 1) & 1, ctl, p.status, 10)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const float f = ctl->factor[i][r];
#pragma unroll
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t v[32];
                        ptx::tmem_ld_32x32(lane_addr + i * D + c0, v);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int g = 0; g < 32; ++g) v[g] = __float_as_uint(__uint_as_float(v[g]) * f);
                        fa2_tmem_st_32x32(lane_addr + i * D + c0, v);
                    }
                    fa2_tmem_st_wait();
                    ptx::tc_fence_before();
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&ctl->o_ready[i]);
            }
        }
        // ---- O = o / l (the parts of a sliced unit are folded by their row threads instead)
        for (int i = 0; i < ntq && ok && part < 0; ++i) {
            if (!fa2_wait(&ctl->pv_done[i], (T - 1) & 1, ctl, p.status, 11)) { ok = false; break; }
            if (!fa2_wait(&ctl->l_done[i], 0, ctl, p.status, 12)) { ok = false; break; }
            ptx::tc_fence_after();
            const int row = n0 + i * FA2_BM + r;
            float* dst = p.O + (static_cast<long long>(b) * p.N + row) * D;
            const float inv = 1.0f / ctl->row_l[i][r];
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(lane_addr + i * D + c0, v);
                ptx::tmem_ld_wait();
                if (row < p.N) {
#pragma unroll
                    for (int g = 0; g < 32; g += 4)
                        *reinterpret_cast<float4*>(dst + c0 + g) = make_float4(__uint_as_float(v[g]) * inv, __uint_as_float(v[g + 1]) * inv,
                                                                               __uint_as_float(v[g + 2]) * inv, __uint_as_float(v[g + 3]) * inv);
                }
            }
        }
        ptx::tc_fence_before();
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 13) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc<1>(tmem_base, TMEM_COLS);
    }
}

}  // namespace cyc
