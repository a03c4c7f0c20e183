// Two-SM tensor-core kernel: a pair of CTAs (one thread-block cluster of 2) owns a
// 256 x 256 block of C.  Each CTA holds the weights of 128 rows i (its half of the
// cells) and HALF of the injected B tile (128 of the 256 time steps j); one
// tcgen05.mma.cta_group::2, issued by the leader CTA, multiplies the 256 rows by all
// 256 columns, reading the peer's half of B from the peer's shared memory.  B is thus
// fetched from L2 once per pair instead of once per CTA -- the on-chip counterpart
// of forwarding B from cell (i,k) to cell (i+1,k) instead of reloading it -- and no
// multicast copy is involved.  Each CTA's TMEM keeps the partial sums of its own 128
// rows (two 256-column accumulators, so the export of one tile overlaps the k loop
// of the next).  The export goes TMEM -> registers -> swizzled shared memory -> TMA
// store, which writes full 128-byte lines and clips at the edges of C.
//
// Barriers (per CTA unless noted):
//   full[s]      leader only: 1 arrival (its producer, with the byte count of BOTH
//                CTAs' copies) + the bytes of both CTAs' TMA loads
//   empty[s]     both: arrival by the leader's tcgen05.commit (multicast to the pair)
//   acc_full[a]  both: arrival by the leader's commit after the last k-block
//   acc_empty[a] leader only: 8 arrivals = 4 epilogue warps of each CTA
#pragma once
#include "umma_kernel.cuh"

namespace cyc {

struct PairParams {
    void* C;
    int M, N, K;
    long long sC;
    int tiles_m, tiles_n;  // 256 x 256 tiles
    long long num_tiles;
    int tma_store;  // 1: export through the C tensor map; 0: direct stores (unaligned C)
    int* status;
    // split-K: the k loop of every tile is cut into `split_k` slices of `kb_per_slice` k-blocks; the tile list
    // then runs over (batch * split_k) entries and entry e = b * split_k + s writes the partial sums of slice s
    // to plane e of the output (a workspace that a second kernel adds up).  split_k = 1: the plain recurrence.
    int split_k = 1;
    int kb_per_slice = 0;
};

// k-block range [kb0, kb0 + nkb) of tile-list entry `e`, and the operand batch index it reads from
__device__ __forceinline__ void pair_k_range(const PairParams& p, int num_kb, int e, int& b, int& kb0, int& nkb) {
    if (p.split_k <= 1) { b = e; kb0 = 0; nkb = num_kb; return; }
    b = e / p.split_k;
    const int s = e - b * p.split_k;
    kb0 = s * p.kb_per_slice;
    nkb = min(p.kb_per_slice, num_kb - kb0);
}

constexpr int PAIR_BN = 256;        // columns of C per pair tile
constexpr int PAIR_HALF = 128;      // B columns (and A rows) held by one CTA
constexpr int PAIR_STAGE_A = 128 * 128;
constexpr int PAIR_STAGE_B = 128 * 128;
constexpr int PAIR_STAGE_BYTES = PAIR_STAGE_A + PAIR_STAGE_B;
constexpr int PAIR_STAGING_BYTES = 4 * 2 * 4096;  // 4 epilogue warps x 2 buffers x (32 rows x 128 B)

template <int STAGES>
constexpr int pair_smem_bytes() { return STAGES * PAIR_STAGE_BYTES + PAIR_STAGING_BYTES + 1024 + 1024; }

template <int KIND, bool B_MN, int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(UMMA_THREADS, 1)
umma_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmC, const PairParams p) {
    using Tr = UmmaTraits<KIND>;
    using Out = typename Tr::Out;
    constexpr int BK = 128 / Tr::ELEM_BYTES;
    constexpr int UK = 32 / Tr::ELEM_BYTES;
    constexpr int CH = 128 / Tr::ELEM_BYTES;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC = umma_instr_desc(Tr::CFMT, Tr::FMT, B_MN, 256, PAIR_BN);
    static_assert(STAGES <= 8, "control block holds 8 stage barriers");

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* staging = smem + STAGES * PAIR_STAGE_BYTES;
    UmmaCtl* ctl = reinterpret_cast<UmmaCtl*>(staging + PAIR_STAGING_BYTES);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();  // 0 = leader (issues the MMAs), 1 = peer
    const long long pair = blockIdx.x >> 1;
    const long long num_pairs = gridDim.x >> 1;
    const int num_kb = (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&ctl->full[s], 1);
            ptx::mbar_init(&ctl->empty[s], 1);
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
    ptx::cluster_arrive();  // the peer's barriers exist before anything is signalled across the pair
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
            for (long long t = pair; t < p.num_tiles && ok; t += num_pairs) {
                int e, tm, tn, b, kb0, nkb;
                umma_tile_coord(t, p.tiles_m, p.tiles_n, e, tm, tn);
                pair_k_range(p, num_kb, e, b, kb0, nkb);
                const int m0 = tm * 256 + static_cast<int>(rank) * PAIR_HALF;      // this CTA's 128 rows of cells
                const int n0 = tn * PAIR_BN + static_cast<int>(rank) * PAIR_HALF;  // this CTA's half of the B tile
                for (int kb = kb0; kb < kb0 + nkb; ++kb) {
                    if (!umma_wait(&ctl->empty[stage], phase ^ 1, ctl, p.status, 1)) { ok = false; break; }
                    uint8_t* sa = smem + stage * PAIR_STAGE_BYTES;
                    uint8_t* sb = sa + PAIR_STAGE_A;
                    const uint32_t bar = full0 + static_cast<uint32_t>(stage * sizeof(uint64_t));
                    if (rank == 0) ptx::mbar_arrive_expect_tx(&ctl->full[stage], 2 * PAIR_STAGE_BYTES);
                    ptx::tma_load_3d_pair(sa, &tmA, bar, kb * BK, m0, b);
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
        if (lane == 0 && rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            bool ok = true;
            for (long long t = pair; t < p.num_tiles && ok; t += num_pairs, ++local) {
                const int ab = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1;
                if (!umma_wait(&ctl->acc_empty[ab], acc_phase ^ 1, ctl, p.status, 2)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ab * PAIR_BN);
                int e, tm, tn, b, kb0, nkb;
                umma_tile_coord(t, p.tiles_m, p.tiles_n, e, tm, tn);
                pair_k_range(p, num_kb, e, b, kb0, nkb);
                for (int kb = 0; kb < nkb; ++kb) {  // the first k-block of the slice starts from zero
                    if (!umma_wait(&ctl->full[stage], phase, ctl, p.status, 3)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t sa = ptx::smem_u32(smem + stage * PAIR_STAGE_BYTES);
                    const uint32_t sb = sa + PAIR_STAGE_A;
#pragma unroll
                    for (int k = 0; k < BK / UK; ++k) {
                        const uint64_t adesc = umma_smem_desc(sa + k * 32, 16, 1024);
                        uint64_t bdesc;
                        if constexpr (!B_MN) bdesc = umma_smem_desc(sb + k * 32, 16, 1024);
                        else bdesc = umma_smem_desc(sb + k * (UK * 128), BK * 128, 1024);
                        ptx::umma<KIND, 2>(d_tmem, adesc, bdesc, IDESC, (kb | k) != 0 ? 1u : 0u);
                    }
                    ptx::umma_commit_pair(&ctl->empty[stage], 3);  // both CTAs may refill this stage
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) ptx::umma_commit_pair(&ctl->acc_full[ab], 3);  // [i,k_end]_C complete in both CTAs
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue: C_ij <- [i,k_end]_C (both CTAs)
        const int q = warp & 3;
        uint8_t* my_stage = staging + q * 8192;
        int local = 0, sbuf = 0;
        bool ok = true;
        for (long long t = pair; t < p.num_tiles && ok; t += num_pairs, ++local) {
            const int ab = local & 1;
            const uint32_t acc_phase = (local >> 1) & 1;
            int b, tm, tn;
            umma_tile_coord(t, p.tiles_m, p.tiles_n, b, tm, tn);
            if (!umma_wait(&ctl->acc_full[ab], acc_phase, ctl, p.status, 4)) { ok = false; break; }
            ptx::tc_fence_after();
            const int row0 = tm * 256 + static_cast<int>(rank) * PAIR_HALF + q * 32;
            const int row = row0 + lane;
            Out* crow = static_cast<Out*>(p.C) + static_cast<long long>(b) * p.sC + static_cast<long long>(row) * p.N;
#pragma unroll 1
            for (int c0 = 0; c0 < PAIR_BN; c0 += 32) {
                const int col = tn * PAIR_BN + c0;
                if (col >= p.N) break;  // uniform over the warp
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(ab * PAIR_BN + c0), v);
                if (p.tma_store) {
                    uint8_t* buf = my_stage + sbuf * 4096;
                    if (lane == 0) ptx::tma_store_wait_read<1>();  // the store that last used this buffer has read it
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
                    sbuf ^= 1;
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
            if (lane == 0) ptx::mbar_arrive_cluster(&ctl->acc_empty[ab], 0);
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
