// fp32 recurrence on tensor cores (used when the caller does not ask for the strict
// per-element k order): every operand x is split into two TF32 parts,
//     hi = x with its 13 low significand bits dropped  (what a kind::tf32 MMA reads from an fp32 word),
//     lo = tf32(x - hi)                                  (round to nearest),
// and each k-step accumulates  A_lo*B_hi + A_hi*B_lo + A_hi*B_hi  into the same fp32
// TMEM accumulator (three tcgen05.mma kind::tf32 per k-step).  The dropped terms
// (A_lo*B_lo < 2^-20 and the rounding of lo < 2^-22, relative to |A_ik||B_kj|) stay far
// inside the 1e-5 * sum_k |A_ik||B_kj| acceptance bound.
//
// Same two-SM organisation as umma_pair_kernel.cuh (256 x 256 tile of C per CTA pair,
// B half per CTA, double-buffered TMEM, TMA-store export) with one more role: two sets of four
// "split" warps per CTA compute the lo part of each landed fp32 stage into a second
// buffer before the MMA thread may read it (the landed tile itself serves as the hi
// part).  The split is element-wise, so it is indifferent to the swizzled tile layout.
//
// Barriers: full[s] (per CTA: its own 32 KB of copies), ready[l] (leader: the split warps of
// the stage's turn in each CTA; the peer's arrive across the pair with a CTA-scope release,
// which is enough because every split thread has already made its writes visible to the async
// proxy and the tiles are read by the tensor cores only), empty[s] and lo_empty[l] (both, by
// the leader's multicast commits), acc_full[a] (both), acc_empty[a] (leader, 8).
#pragma once
#include "umma_pair_kernel.cuh"

namespace cyc {

#ifndef CYC_X3_SPLIT_SETS
#define CYC_X3_SPLIT_SETS 1
#endif
constexpr int X3_SPLIT_WARPS = 8;                         // split warps per CTA
constexpr int X3_SPLIT_SETS = CYC_X3_SPLIT_SETS;          // sets of split warps, taking stages in turn
constexpr int X3_SET_WARPS = X3_SPLIT_WARPS / X3_SPLIT_SETS;
constexpr int X3_THREADS = 192 + X3_SPLIT_WARPS * 32;     // TMA, MMA, 4 epilogue warps, then the split warps
#ifndef CYC_X3_BK
#define CYC_X3_BK 32
#endif
// A stage holds BK = 32 (or 16) values of k: A (128 rows) + B half (128 columns), BK * 4 bytes of k each.  Two rings share
// 192 KB: the landed fp32 tiles (read by the MMAs as the hi parts) and the lo parts the split warps derive from them.  A
// landed tile is held from the copy's issue to the end of its MMAs, a lo tile only from the split to the end of the MMAs,
// so the first ring is the deeper one (four and two stages of 32 KB; three and three were 49-52 microseconds on the
// 65536 x 256 x 256 problem).  Six and six stages of 16 KB (BK = 16, 64-byte swizzle) measured 61-62: what counts is the
// bytes in flight, not the number of stages.
constexpr int X3_BK = CYC_X3_BK;
constexpr int X3_STAGE_HI = 2 * 128 * X3_BK * 4;
#ifndef CYC_X3_RAW_STAGES
#define CYC_X3_RAW_STAGES (128 / CYC_X3_BK)
#endif
#ifndef CYC_X3_LO_STAGES
#define CYC_X3_LO_STAGES (64 / CYC_X3_BK)
#endif
constexpr int X3_RAW_STAGES = CYC_X3_RAW_STAGES, X3_LO_STAGES = CYC_X3_LO_STAGES;
static_assert(X3_RAW_STAGES <= 8 && X3_LO_STAGES <= 8 && X3_LO_STAGES <= X3_RAW_STAGES, "ring sizes");
constexpr int X3_PREFETCH = 256 / X3_BK;  // k-blocks of A requested from L2 ahead of the ring
constexpr int X3_SMEM_BYTES = (X3_RAW_STAGES + X3_LO_STAGES) * X3_STAGE_HI + PAIR_STAGING_BYTES_4 + 1024 + 1024;

struct X3Ctl {
    uint64_t full[8];      // landed-tile ring: copies done
    uint64_t empty[8];     // landed-tile ring: MMAs done
    uint64_t ready[8];     // lo ring: split done
    uint64_t lo_empty[8];  // lo ring: MMAs done
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    volatile int abort;
};

__device__ __forceinline__ bool x3_wait(uint64_t* bar, uint32_t parity, X3Ctl* ctl, int* status, int where) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (ctl->abort) return false;
        if (clock64() - t0 > UMMA_WAIT_CYCLES) {
            ctl->abort = 1;
            atomicExch(status, 0x200 | where);
            return false;
        }
    }
    return true;
}

// fp32 bit pattern -> nearest TF32 (10 explicit significand bits; ties away from zero), low 13 bits cleared.
// Integer arithmetic on the encoding: adding half a TF32 ulp carries into the exponent exactly as rounding does.
__device__ __forceinline__ uint32_t tf32_round(uint32_t bits) { return (bits + 0x1000u) & 0xFFFFE000u; }

template <bool B_MN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(X3_THREADS, 1)
umma_pair_tf32x3_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                        const __grid_constant__ CUtensorMap tmC, const PairParams p) {
    constexpr int BK = X3_BK;  // fp32 elements of k per stage: one 128-byte (or 64-byte) swizzle row
    constexpr int UK = 8;    // k extent of one kind::tf32 MMA
    constexpr int CH = 32;   // B stored [K][N]: columns per 128-byte row
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC = umma_instr_desc(1, 2, B_MN, 256, PAIR_BN);
    constexpr int STAGES = X3_RAW_STAGES, LSTAGES = X3_LO_STAGES;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* smem_lo = smem + STAGES * X3_STAGE_HI;
    uint8_t* staging = smem_lo + LSTAGES * X3_STAGE_HI;
    X3Ctl* ctl = reinterpret_cast<X3Ctl*>(staging + PAIR_STAGING_BYTES_4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const long long pair = blockIdx.x >> 1;
    const long long num_pairs = gridDim.x >> 1;
    const int num_kb = (p.K + BK - 1) / BK;

    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&ctl->full[s], 1);
            ptx::mbar_init(&ctl->empty[s], 1);
        }
        for (int l = 0; l < LSTAGES; ++l) {
            ptx::mbar_init(&ctl->ready[l], 2 * X3_SET_WARPS);  // the split warps of the stage's turn, both CTAs
            ptx::mbar_init(&ctl->lo_empty[l], 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&ctl->acc_full[a], 1);
            ptx::mbar_init(&ctl->acc_empty[a], 8);
        }
        ctl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
        ptx::prefetch_tensormap(&tmC);
    }
    if (warp == 1) {
        ptx::tmem_alloc<2>(&ctl->tmem_base, TMEM_COLS);
        ptx::tmem_relinquish<2>();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_arrive();
    ptx::cluster_wait();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs, own barrier)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            ptx::grid_dependency_wait();  // the set-up above may overlap the previous kernel; nothing it wrote is read before it ends
            // A is streamed from HBM exactly once, and the ring is only three stages deep: a second cursor runs
            // X3_PREFETCH k-blocks ahead and asks L2 for the A tiles, so the copies into the ring hit L2
            int pf_item = 0, pf_kb = 0;
            PairWork pw;
            bool pf_more = pair_work_item(p, num_kb, pair, num_pairs, 0, pw);
            auto prefetch_next = [&]() {
                if (!pf_more) return;
                int b, tm, tn;
                umma_tile_coord(pw.tile, p.tiles_m, p.tiles_n, b, tm, tn);
                ptx::tma_prefetch_l2_3d(&tmA, (pw.kb0 + pf_kb) * BK, tm * 256 + static_cast<int>(rank) * PAIR_HALF, b);
                if (++pf_kb == pw.nkb) { pf_kb = 0; pf_more = pair_work_item(p, num_kb, pair, num_pairs, ++pf_item, pw); }
            };
            for (int i = 0; i < X3_PREFETCH; ++i) prefetch_next();
            PairWork w;
            for (int item = 0; ok && pair_work_item(p, num_kb, pair, num_pairs, item, w); ++item) {
                int b, tm, tn;
                umma_tile_coord(w.tile, p.tiles_m, p.tiles_n, b, tm, tn);
                const int m0 = tm * 256 + static_cast<int>(rank) * PAIR_HALF;
                const int n0 = tn * PAIR_BN + static_cast<int>(rank) * PAIR_HALF;
                for (int kb = w.kb0; kb < w.kb0 + w.nkb; ++kb) {
                    prefetch_next();
                    if (!x3_wait(&ctl->empty[stage], phase ^ 1, ctl, p.status, 1)) { ok = false; break; }
                    uint8_t* sa = smem + stage * X3_STAGE_HI;
                    uint8_t* sb = sa + 128 * BK * 4;
                    ptx::mbar_arrive_expect_tx(&ctl->full[stage], X3_STAGE_HI);
                    ptx::tma_load_3d(sa, &tmA, &ctl->full[stage], kb * BK, m0, b);
                    if constexpr (!B_MN) {
                        ptx::tma_load_3d(sb, &tmB, &ctl->full[stage], kb * BK, n0, b);
                    } else {
#pragma unroll
                        for (int c = 0; c < PAIR_HALF / CH; ++c)
                            ptx::tma_load_3d(sb + c * (BK * 128), &tmB, &ctl->full[stage], n0 + c * CH, kb * BK, b);
                    }
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
                const int back = issued < STAGES ? static_cast<int>(issued) : STAGES;
                int s = stage;
                uint32_t ph = phase;
                for (int n = 0; n < back; ++n) {
                    if (--s < 0) { s = STAGES - 1; ph ^= 1; }
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(&ctl->full[s], ph) && clock64() - t0 < UMMA_WAIT_CYCLES) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (rank == 0) {  // the whole warp walks the loop converged, one elected lane issues
            const uint32_t leader = ptx::elect_one();
            int stage = 0, lstage = 0;
            uint32_t lphase = 0;
            int local = 0;
            bool ok = true;
            PairWork w;
            for (; ok && pair_work_item(p, num_kb, pair, num_pairs, local, w); ++local) {
                const int ab = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1;
                if (!x3_wait(&ctl->acc_empty[ab], acc_phase ^ 1, ctl, p.status, 2)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ab * PAIR_BN);
                for (int kb = 0; kb < w.nkb; ++kb) {  // the first k-block of a slice starts from zero
                    if (!x3_wait(&ctl->ready[lstage], lphase, ctl, p.status, 3)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t sa = ptx::smem_u32(smem + stage * X3_STAGE_HI);
                    const uint32_t sb = sa + 128 * BK * 4;
                    const uint32_t la = ptx::smem_u32(smem_lo + lstage * X3_STAGE_HI);
                    const uint32_t lb = la + 128 * BK * 4;
#pragma unroll
                    for (int k = 0; k < BK / UK; ++k) {
                        // K-major rows of BK * 4 bytes (128- or 64-byte swizzle), groups of 8 rows one after another
                        constexpr uint32_t KSBO = 8 * BK * 4, KSW = BK == 32 ? 2 : 4;
                        const uint64_t a_hi = umma_smem_desc(sa + k * 32, 16, KSBO, KSW);
                        const uint64_t a_lo = umma_smem_desc(la + k * 32, 16, KSBO, KSW);
                        uint64_t b_hi, b_lo;
                        if constexpr (!B_MN) {
                            b_hi = umma_smem_desc(sb + k * 32, 16, KSBO, KSW);
                            b_lo = umma_smem_desc(lb + k * 32, 16, KSBO, KSW);
                        } else {
                            // B stored [K][N]: 128-byte rows of 32 columns, 32-byte chunks permuted over groups of
                            // 4 k-rows (512 B apart); the next 32 columns are BK*128 B further on
                            b_hi = umma_smem_desc(sb + k * (UK * 128), BK * 128, 512, 1);
                            b_lo = umma_smem_desc(lb + k * (UK * 128), BK * 128, 512, 1);
                        }
                        ptx::umma_elect<KIND_TF32, 2>(d_tmem, a_lo, b_hi, IDESC, (kb | k) != 0 ? 1u : 0u, leader);
                        ptx::umma_elect<KIND_TF32, 2>(d_tmem, a_hi, b_lo, IDESC, 1u, leader);
                        ptx::umma_elect<KIND_TF32, 2>(d_tmem, a_hi, b_hi, IDESC, 1u, leader);
                    }
                    ptx::umma_commit_pair_elect(&ctl->empty[stage], 3, leader);
                    ptx::umma_commit_pair_elect(&ctl->lo_empty[lstage], 3, leader);
                    if (++stage == STAGES) stage = 0;
                    if (++lstage == LSTAGES) { lstage = 0; lphase ^= 1; }
                }
                if (ok) ptx::umma_commit_pair_elect(&ctl->acc_full[ab], 3, leader);
            }
        }
        __syncwarp();
    } else if (warp >= 6) {
        // ------------------------------------------------------------ split warps: x -> (hi, lo)
        // the sets of four warps take stages in turn, so the fixed latencies of one stage's split
        // (wait, store drain, proxy fence) overlap with the other set's work
        const int set = (warp - 6) / X3_SET_WARPS;
        constexpr int NT = 32 * X3_SET_WARPS;
        const int tid = (threadIdx.x - 6 * 32) % NT;  // index within the set
        int stage = 0, lstage = 0;
        uint32_t phase = 0, lphase = 0;
        uint32_t turn = 0;
        bool ok = true;
        PairWork w;
        auto advance = [&]() {
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
            if (++lstage == LSTAGES) { lstage = 0; lphase ^= 1; }
        };
        for (int item = 0; ok && pair_work_item(p, num_kb, pair, num_pairs, item, w); ++item) {
            for (int kb = 0; kb < w.nkb; ++kb, ++turn) {
                // Every set observes every use of every stage, its own or not: a parity wait tells phase k from phase
                // k + 1 only, and copies may land out of order, so a set that skipped the other set's turn could otherwise
                // take the previous use of a stage for the one it is waiting for.
                if (!x3_wait(&ctl->full[stage], phase, ctl, p.status, 5)) { ok = false; break; }
                if (!x3_wait(&ctl->lo_empty[lstage], lphase ^ 1, ctl, p.status, 6)) { ok = false; break; }
                if (turn % X3_SPLIT_SETS != static_cast<uint32_t>(set)) {
                    advance();
                    continue;
                }
                const uint8_t* base = smem + stage * X3_STAGE_HI;
                uint8_t* lo_base = smem_lo + lstage * X3_STAGE_HI;
#pragma unroll 1
                for (int it0 = 0; it0 < X3_STAGE_HI / (NT * 16); it0 += 4) {
                    uint4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) v[u] = *reinterpret_cast<const uint4*>(base + (tid + NT * (it0 + u)) * 16);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t x[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                        uint32_t lo[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            // hi = x with the 13 low significand bits dropped: exactly what the tensor core reads
                            // from the untouched fp32 tile.  inf/NaN stay in the hi part only.
                            const uint32_t hi = x[e] & 0xFFFFE000u;
                            const float r = __uint_as_float(x[e]) - __uint_as_float(hi);  // exact, below 2^-10 |x|
                            lo[e] = ((x[e] & 0x7F800000u) == 0x7F800000u) ? 0u : tf32_round(__float_as_uint(r));
                        }
                        const int off = (tid + NT * (it0 + u)) * 16;
                        *reinterpret_cast<uint4*>(lo_base + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    }
                }
                ptx::fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) ptx::mbar_arrive(&ctl->ready[lstage]);
                    else ptx::mbar_arrive_remote(&ctl->ready[lstage], 0);
                }
                advance();
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: C_ij <- [i,k_end]_C (both CTAs)
        const int q = warp & 3;
        uint8_t* my_stage = staging + q * 8192;
        const uint32_t lane_taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        int local = 0, sbuf = 0;
        bool ok = true;
        PairWork w;
        for (; ok && pair_work_item(p, num_kb, pair, num_pairs, local, w); ++local) {
            const int ab = local & 1;
            const uint32_t acc_phase = (local >> 1) & 1;
            int b, tm, tn;
            umma_tile_coord(w.tile, p.tiles_m, p.tiles_n, b, tm, tn);
            if (!x3_wait(&ctl->acc_full[ab], acc_phase, ctl, p.status, 4)) { ok = false; break; }
            ptx::tc_fence_after();
            const int row0 = tm * 256 + static_cast<int>(rank) * PAIR_HALF + q * 32;
            const int row = row0 + lane;
            float* crow = static_cast<float*>(p.C) + static_cast<long long>(b) * p.sC + static_cast<long long>(row) * p.N;
            const int nchunks = min(PAIR_BN / 32, (p.N - tn * PAIR_BN + 31) / 32);
            auto export_piece = [&](const uint32_t (&v)[32], int c0) {
                const int col = tn * PAIR_BN + c0;
                if (p.tma_store) {
                    uint8_t* buf = my_stage + sbuf * 4096;
                    if (lane == 0) ptx::tma_store_wait_read<1>();
                    __syncwarp();
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        *reinterpret_cast<uint4*>(buf + lane * 128 + ((g ^ (lane & 7)) << 4)) = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_3d(&tmC, buf, col, row0, b);
                        ptx::tma_store_commit();
                    }
                    sbuf ^= 1;
                } else if (row < p.M) {
#pragma unroll
                    for (int g = 0; g < 32; ++g)
                        if (col + g < p.N) reinterpret_cast<uint32_t*>(crow)[col + g] = v[g];
                }
            };
            // the tensor-memory read of the next piece is in flight while this one is staged and stored
            uint32_t va[32], vb[32];
            ptx::tmem_ld_32x32(lane_taddr + static_cast<uint32_t>(ab * PAIR_BN), va);
#pragma unroll 1
            for (int c = 0; c < nchunks; c += 2) {
                ptx::tmem_ld_wait();
                if (c + 1 < nchunks) ptx::tmem_ld_32x32(lane_taddr + static_cast<uint32_t>(ab * PAIR_BN + (c + 1) * 32), vb);
                export_piece(va, c * 32);
                if (c + 1 < nchunks) {
                    ptx::tmem_ld_wait();
                    if (c + 2 < nchunks) ptx::tmem_ld_32x32(lane_taddr + static_cast<uint32_t>(ab * PAIR_BN + (c + 2) * 32), va);
                    export_piece(vb, (c + 1) * 32);
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_remote(&ctl->acc_empty[ab], 0);
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();
        __syncwarp();
    }

    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_arrive();
    ptx::cluster_wait();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc<2>(tmem_base, TMEM_COLS);
    }
}

}  // namespace cyc
