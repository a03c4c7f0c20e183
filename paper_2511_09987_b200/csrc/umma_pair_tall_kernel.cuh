// Two-SM tensor-core kernel with TALL tiles: a pair of CTAs owns a 512 x 256 block of C.
// Same organisation as umma_pair_kernel.cuh, but each CTA holds the weights of TWO blocks of
// 128 rows (rows r*128.. of the upper and of the lower 256-row half of the tile), so one
// B half-tile in shared memory now feeds 512 rows of cells: 96 KB enter the pair per
// k-block for 512 x 256 outputs instead of 64 KB for 256 x 256 -- a quarter less traffic
// from L2 into the SMs per multiply-accumulate, which is what bounds the 256 x 256 kernel.
// The price: the two fp32/int32 accumulators (2 x 256 TMEM columns per CTA) now belong to the
// same tile, so the export of a tile no longer overlaps the k loop of the next one.  Eight
// epilogue warps (four per accumulator) keep that exposed time short, and the kernel is
// only selected when the k loop is long enough to amortise it.
//
// Barriers: full[s] (leader: 1 arrival + the bytes of both CTAs' copies), empty[s] (both, by
// the leader's multicast commit), acc_full (both), acc_empty (leader, 16 warp arrivals).
#pragma once
#include "umma_pair_kernel.cuh"

namespace cyc {

constexpr int TALL_THREADS = 320;                 // TMA, MMA, 2 x 4 epilogue warps
constexpr int TALL_STAGE_A = 128 * 128;           // one block of 128 rows x 128 bytes of k
constexpr int TALL_STAGE_BYTES = 3 * 128 * 128;   // two row blocks of A + the B half
constexpr int TALL_STAGES = 4;
constexpr int TALL_STAGING_BYTES = 8 * 4096;      // one 32 x 32 box per epilogue warp
constexpr int TALL_SMEM_BYTES = TALL_STAGES * TALL_STAGE_BYTES + TALL_STAGING_BYTES + 1024 + 1024;

template <int KIND, bool B_MN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TALL_THREADS, 1)
umma_pair_tall_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                      const __grid_constant__ CUtensorMap tmC, const PairParams p) {
    using Tr = UmmaTraits<KIND>;
    using Out = typename Tr::Out;
    constexpr int BK = 128 / Tr::ELEM_BYTES;
    constexpr int UK = 32 / Tr::ELEM_BYTES;
    constexpr int CH = 128 / Tr::ELEM_BYTES;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC = umma_instr_desc(Tr::CFMT, Tr::FMT, B_MN, 256, PAIR_BN);
    constexpr int STAGES = TALL_STAGES;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* staging = smem + STAGES * TALL_STAGE_BYTES;
    UmmaCtl* ctl = reinterpret_cast<UmmaCtl*>(staging + TALL_STAGING_BYTES);

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
        ptx::mbar_init(&ctl->acc_full[0], 1);
        ptx::mbar_init(&ctl->acc_empty[0], 16);
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
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            const uint32_t full0 = ptx::mapa_u32(ptx::smem_u32(&ctl->full[0]), 0);  // the leader's full[] barriers
            ptx::grid_dependency_wait();  // the set-up above may overlap the previous kernel; nothing it wrote is read before it ends
            for (long long t = pair; t < p.num_tiles && ok; t += num_pairs) {
                int b, tm, tn;
                umma_tile_coord(t, p.tiles_m, p.tiles_n, b, tm, tn);
                const int m0 = tm * 512 + static_cast<int>(rank) * PAIR_HALF;  // upper row block; the lower one is 256 rows on
                const int n0 = tn * PAIR_BN + static_cast<int>(rank) * PAIR_HALF;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!umma_wait(&ctl->empty[stage], phase ^ 1, ctl, p.status, 1)) { ok = false; break; }
                    uint8_t* sa = smem + stage * TALL_STAGE_BYTES;
                    uint8_t* sb = sa + 2 * TALL_STAGE_A;
                    const uint32_t bar = full0 + static_cast<uint32_t>(stage * sizeof(uint64_t));
                    if (rank == 0) ptx::mbar_arrive_expect_tx(&ctl->full[stage], 2 * TALL_STAGE_BYTES);
                    ptx::tma_load_3d_pair(sa, &tmA, bar, kb * BK, m0, b);
                    ptx::tma_load_3d_pair(sa + TALL_STAGE_A, &tmA, bar, kb * BK, m0 + 256, b);
                    if constexpr (!B_MN) {
                        ptx::tma_load_3d_pair(sb, &tmB, bar, kb * BK, n0, b);
                    } else {
#pragma unroll
                        for (int c = 0; c < PAIR_HALF / CH; ++c)
                            ptx::tma_load_3d_pair(sb + c * (BK * 128), &tmB, bar, n0 + c * CH, kb * BK, b);
                    }
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok && rank == 0) {
                // leave no copy in flight: wait (bounded) for the loads already issued
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
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            bool ok = true;
            for (long long t = pair; t < p.num_tiles && ok; t += num_pairs, ++local) {
                // both accumulators belong to the previous tile until its export has drained them
                if (!umma_wait(&ctl->acc_empty[0], (local & 1) ^ 1, ctl, p.status, 2)) { ok = false; break; }
                ptx::tc_fence_after();
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!umma_wait(&ctl->full[stage], phase, ctl, p.status, 3)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t sa = ptx::smem_u32(smem + stage * TALL_STAGE_BYTES);
                    const uint32_t sb = sa + 2 * TALL_STAGE_A;
#pragma unroll
                    for (int k = 0; k < BK / UK; ++k) {
                        const uint64_t a0 = umma_smem_desc(sa + k * 32, 16, 1024);
                        const uint64_t a1 = umma_smem_desc(sa + TALL_STAGE_A + k * 32, 16, 1024);
                        uint64_t bdesc;
                        if constexpr (!B_MN) bdesc = umma_smem_desc(sb + k * 32, 16, 1024);
                        else bdesc = umma_smem_desc(sb + k * (UK * 128), BK * 128, 1024);
                        const uint32_t acc = (kb | k) != 0 ? 1u : 0u;
                        ptx::umma_elect<KIND, 2>(tmem_base, a0, bdesc, IDESC, acc, leader);            // rows   0..255 of the tile
                        ptx::umma_elect<KIND, 2>(tmem_base + PAIR_BN, a1, bdesc, IDESC, acc, leader);  // rows 256..511 of the tile
                    }
                    ptx::umma_commit_pair_elect(&ctl->empty[stage], 3, leader);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) ptx::umma_commit_pair_elect(&ctl->acc_full[0], 3, leader);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue: C_ij <- [i,k_end]_C
        const int q = warp & 3;          // TMEM lane quarter
        const int rb = (warp - 2) >> 2;  // which accumulator / row block this warp drains
        uint8_t* buf = staging + (warp - 2) * 4096;
        int local = 0;
        bool ok = true;
        for (long long t = pair; t < p.num_tiles && ok; t += num_pairs, ++local) {
            int b, tm, tn;
            umma_tile_coord(t, p.tiles_m, p.tiles_n, b, tm, tn);
            if (!umma_wait(&ctl->acc_full[0], local & 1, ctl, p.status, 4)) { ok = false; break; }
            ptx::tc_fence_after();
            const int row0 = tm * 512 + rb * 256 + static_cast<int>(rank) * PAIR_HALF + q * 32;
            const int row = row0 + lane;
            Out* crow = static_cast<Out*>(p.C) + static_cast<long long>(b) * p.sC + static_cast<long long>(row) * p.N;
#pragma unroll 1
            for (int c0 = 0; c0 < PAIR_BN; c0 += 32) {
                const int col = tn * PAIR_BN + c0;
                if (col >= p.N) break;  // uniform over the warp
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(rb * PAIR_BN + c0), v);
                if (p.tma_store) {
                    if (lane == 0) ptx::tma_store_wait_read<0>();  // the previous store has read the staging buffer
                    __syncwarp();
                    ptx::tmem_ld_wait();
                    // 32 rows x 128 B, 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7)
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        *reinterpret_cast<uint4*>(buf + lane * 128 + ((g ^ (lane & 7)) << 4)) = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_3d(&tmC, buf, col, row0, b);
                        ptx::tma_store_commit();
                    }
                } else {
                    ptx::tmem_ld_wait();
                    if (row < p.M) {
#pragma unroll
                        for (int g = 0; g < 32; ++g)
                            if (col + g < p.N) reinterpret_cast<uint32_t*>(crow)[col + g] = v[g];
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_remote(&ctl->acc_empty[0], 0);
        }
        if (lane == 0) ptx::tma_store_wait_all<0>();
        __syncwarp();
    }

    // neither CTA may leave (or free TMEM) while its peer can still reach its shared memory or barriers
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
