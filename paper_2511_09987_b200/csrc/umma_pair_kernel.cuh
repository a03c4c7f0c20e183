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
    // Sliced tail (umma_pair_kernel only; never under the fixed-k-order flag): when the tile count is not a multiple
    // of the number of CTA pairs, the last `tail_tiles` tiles of the list would occupy only some pairs for one more
    // whole k loop.  Instead each of them is cut into `tail_S` k-slices of `tail_kb` k-blocks, the tail_tiles * tail_S
    // slices go to different pairs as their FIRST work item, and for every 32-row strip of such a tile the warp that
    // finishes its slice last adds the other slices' partial sums (parked in `tail_ws`) in increasing k and exports
    // C.  Nobody waits for anybody: `tail_counters` (one per strip, zero between launches) tells a warp whether it
    // is the last.
    int tail_S = 0;
    int tail_tiles = 0;
    int tail_kb = 0;
    void* tail_ws = nullptr;
    int* tail_counters = nullptr;
};

// one item of a pair's work list: a tile (or one k-slice of a tail tile) with its k-block range
struct PairWork {
    long long tile;  // index into the tile list (for split_k: the (problem, slice) entry)
    int kb0, nkb;
    int slice;       // k-slice of a tail tile, or -1
    int tail_index;  // which tail tile
};

// i-th work item of pair `pair` (of `num_pairs`); false when the pair's list is exhausted
__device__ __forceinline__ bool pair_work_item(const PairParams& p, int num_kb, long long pair, long long num_pairs, int i, PairWork& w) {
    long long full_tiles = p.num_tiles;
    if (p.tail_S > 1) {
        full_tiles = p.num_tiles - p.tail_tiles;
        const long long units = static_cast<long long>(p.tail_tiles) * p.tail_S;
        if (pair < units) {
            if (i == 0) {
                w.tail_index = static_cast<int>(pair / p.tail_S);
                w.slice = static_cast<int>(pair - static_cast<long long>(w.tail_index) * p.tail_S);
                w.tile = full_tiles + w.tail_index;
                w.kb0 = w.slice * p.tail_kb;
                w.nkb = min(p.tail_kb, num_kb - w.kb0);
                return true;
            }
            --i;
        }
    }
    w.tile = pair + static_cast<long long>(i) * num_pairs;
    w.slice = -1;
    w.tail_index = 0;
    w.kb0 = 0;
    w.nkb = num_kb;
    return w.tile < full_tiles;
}

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
#ifndef CYC_PAIR_EPI_WARPS
#define CYC_PAIR_EPI_WARPS 4
#endif
// Epilogue warps per CTA: four (one per tensor-memory lane quarter, 256 columns each) or eight (two per quarter, 128
// columns each; the ring then has five stages instead of six, so that 64 KB of export staging fit).  Measured: eight
// warps change nothing on the batched 256^3 problems (94.9 against 95.0-95.4 us: the export is not what bounds them) and
// cost 4 % on int8 4096^3 (the sixth stage matters there), so four it is.
constexpr int PAIR_EPI_WARPS = CYC_PAIR_EPI_WARPS;
constexpr int PAIR_EPI_COLS = PAIR_BN * 4 / PAIR_EPI_WARPS;     // columns of a tile one epilogue warp exports
constexpr int PAIR_THREADS = 64 + 32 * PAIR_EPI_WARPS;          // producer, MMA issuer, epilogue warps
constexpr int PAIR_STAGES = PAIR_EPI_WARPS == 8 ? 5 : 6;
constexpr int PAIR_STAGING_BYTES = PAIR_EPI_WARPS * 2 * 4096;   // per epilogue warp 2 buffers of 32 rows x 128 B
constexpr int PAIR_STAGING_BYTES_4 = 4 * 2 * 4096;              // the kernels with four epilogue warps
constexpr int PAIR_STRIPS = 2 * PAIR_EPI_WARPS;                 // strips of a tile: one per epilogue warp of the pair
constexpr int PAIR_STRIP_BYTES = 32 * PAIR_EPI_COLS * 4;        // partial sums of one strip (32 rows x the warp's columns)
constexpr int PAIR_TILE_BYTES = PAIR_STRIPS * PAIR_STRIP_BYTES; // = 256 KB

// k-slice of a tail tile, seen from the epilogue warp that owns strip `strip` of the tile (32 rows x `nchunks` pieces of 32
// columns starting at column `col0`): park
// the strip's partial sums (16-byte piece g of a lane's 32 values at (g * 32 + lane) * 16, so that one store instruction
// writes 512 contiguous bytes), give the accumulator at `acc_taddr` back, and find out whether the other slices of the
// strip are already there.  If so, C_ij = the slices' sums added in increasing k (the slice at hand is read back like
// the others; the read of the next piece is in flight while this one is added), handed piece by piece to
// `export_piece(values, first column within the tile)`.  (`ptx::mbar_arrive_remote` gives the accumulator back.)
template <typename Out, typename ExportFn>
__device__ __forceinline__ void pair_tail_strip(const PairParams& p, const PairWork& w, int strip, uint32_t acc_taddr, int col0, int nchunks, int lane,
                                                uint64_t* acc_empty, ExportFn&& export_piece) {
    uint8_t* tile_ws = static_cast<uint8_t*>(p.tail_ws) + static_cast<size_t>(w.tail_index) * p.tail_S * PAIR_TILE_BYTES;
    uint8_t* mine = tile_ws + static_cast<size_t>(w.slice) * PAIR_TILE_BYTES + strip * PAIR_STRIP_BYTES;
#pragma unroll 1
    for (int c = 0; c < nchunks; ++c) {
        uint32_t v[32];
        ptx::tmem_ld_32x32(acc_taddr + static_cast<uint32_t>(col0 + c * 32), v);
        ptx::tmem_ld_wait();
        uint4* dst = reinterpret_cast<uint4*>(mine + c * 4096);
#pragma unroll
        for (int g = 0; g < 8; ++g) dst[g * 32 + lane] = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
    }
    ptx::tc_fence_before();
    __threadfence();  // this lane's partial sums are out before the warp is counted
    __syncwarp();
    int arrived = 0;
    if (lane == 0) {
        ptx::mbar_arrive_remote(acc_empty, 0);
        arrived = atomicAdd(&p.tail_counters[w.tail_index * PAIR_STRIPS + strip], 1);
    }
    arrived = __shfl_sync(0xffffffffu, arrived, 0);
    if (arrived != p.tail_S - 1) return;  // a later warp finishes this strip
    __threadfence();
    if (lane == 0) p.tail_counters[w.tail_index * PAIR_STRIPS + strip] = 0;  // zero again for the next launch
    const uint8_t* strip_ws = tile_ws + strip * PAIR_STRIP_BYTES;
    const int pieces = nchunks * p.tail_S;
    auto fetch = [&](int i, uint32_t (&o)[32]) {
        const int c = i / p.tail_S, sl = i - c * p.tail_S;
        const uint4* src = reinterpret_cast<const uint4*>(strip_ws + static_cast<size_t>(sl) * PAIR_TILE_BYTES + c * 4096);
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const uint4 x = __ldcg(src + g * 32 + lane);  // written by another SM: read through L2
            o[4 * g] = x.x; o[4 * g + 1] = x.y; o[4 * g + 2] = x.z; o[4 * g + 3] = x.w;
        }
    };
    if (pieces == 0) return;  // this warp's columns lie outside C
    uint32_t cur[32], nxt[32], sum[32] = {};
    fetch(0, cur);
#pragma unroll 1
    for (int i = 0; i < pieces; ++i) {
        if (i + 1 < pieces) fetch(i + 1, nxt);
        const int c = i / p.tail_S, sl = i - c * p.tail_S;
#pragma unroll
        for (int g = 0; g < 32; ++g) {
            Out x, y;
            memcpy(&x, &cur[g], 4);
            memcpy(&y, &sum[g], 4);
            y = sl == 0 ? x : y + x;
            memcpy(&sum[g], &y, 4);
        }
        if (sl == p.tail_S - 1) export_piece(sum, col0 + c * 32);
#pragma unroll
        for (int g = 0; g < 32; ++g) cur[g] = nxt[g];
    }
}

template <int STAGES>
constexpr int pair_smem_bytes() { return STAGES * PAIR_STAGE_BYTES + PAIR_STAGING_BYTES + 1024 + 1024; }

template <int KIND, bool B_MN, int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PAIR_THREADS, 1)
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

    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&ctl->full[s], 1);
            ptx::mbar_init(&ctl->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&ctl->acc_full[a], 1);
            ptx::mbar_init(&ctl->acc_empty[a], 2 * PAIR_EPI_WARPS);
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
            ptx::grid_dependency_wait();  // the set-up above may overlap the previous kernel; operands may not be read before it ends
            PairWork w;
            for (int item = 0; ok && pair_work_item(p, num_kb, pair, num_pairs, item, w); ++item) {
                int e, tm, tn, b, kb0, nkb;
                umma_tile_coord(w.tile, p.tiles_m, p.tiles_n, e, tm, tn);
                pair_k_range(p, num_kb, e, b, kb0, nkb);
                if (w.slice >= 0) { kb0 = w.kb0; nkb = w.nkb; }
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
        // ------------------------------------------------------------ MMA issuer (leader CTA only): the whole warp walks
        // ------------------------------------------------------------ the loop converged, one elected lane issues
        if (rank == 0) {
            const uint32_t leader = ptx::elect_one();
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            bool ok = true;
            PairWork w;
            for (; ok && pair_work_item(p, num_kb, pair, num_pairs, local, w); ++local) {
                const int ab = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1;
                if (!umma_wait(&ctl->acc_empty[ab], acc_phase ^ 1, ctl, p.status, 2)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ab * PAIR_BN);
                int e, tm, tn, b, kb0, nkb;
                umma_tile_coord(w.tile, p.tiles_m, p.tiles_n, e, tm, tn);
                pair_k_range(p, num_kb, e, b, kb0, nkb);
                if (w.slice >= 0) nkb = w.nkb;
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
                        ptx::umma_elect<KIND, 2>(d_tmem, adesc, bdesc, IDESC, (kb | k) != 0 ? 1u : 0u, leader);
                    }
                    ptx::umma_commit_pair_elect(&ctl->empty[stage], 3, leader);  // both CTAs may refill this stage
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) ptx::umma_commit_pair_elect(&ctl->acc_full[ab], 3, leader);  // [i,k_end]_C complete in both CTAs
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue: C_ij <- [i,k_end]_C (both CTAs)
        const int q = warp & 3;                                  // tensor-memory lane quarter this warp may read
        const int ew = warp - 2;                                 // epilogue warp 0 .. PAIR_EPI_WARPS - 1
        const int col_first = (ew >> 2) * PAIR_EPI_COLS;         // its columns of the tile: [col_first, col_first + PAIR_EPI_COLS)
        uint8_t* my_stage = staging + ew * 8192;
        const uint32_t lane_taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        int local = 0, sbuf = 0;
        bool ok = true;
        PairWork w;
        for (; ok && pair_work_item(p, num_kb, pair, num_pairs, local, w); ++local) {
            const int ab = local & 1;
            const uint32_t acc_phase = (local >> 1) & 1;
            int b, tm, tn;
            umma_tile_coord(w.tile, p.tiles_m, p.tiles_n, b, tm, tn);
            if (!umma_wait(&ctl->acc_full[ab], acc_phase, ctl, p.status, 4)) { ok = false; break; }
            ptx::tc_fence_after();
            const int row0 = tm * 256 + static_cast<int>(rank) * PAIR_HALF + q * 32;
            const int row = row0 + lane;
            Out* crow = static_cast<Out*>(p.C) + static_cast<long long>(b) * p.sC + static_cast<long long>(row) * p.N;
            // 32-column pieces of this warp's columns that lie inside C
            const int nchunks = max(0, min(PAIR_EPI_COLS / 32, (p.N - tn * PAIR_BN - col_first + 31) / 32));
            // one 32 x 32 piece of C (this lane's row, 32 consecutive columns starting at c0) leaves the SM
            auto export_piece = [&](const uint32_t (&v)[32], int c0) {
                const int col = tn * PAIR_BN + c0;
                if (p.tma_store) {
                    uint8_t* buf = my_stage + sbuf * 4096;
                    if (lane == 0) ptx::tma_store_wait_read<1>();  // the store that last used this buffer has read it
                    __syncwarp();
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
                } else if (row < p.M) {
#pragma unroll
                    for (int g = 0; g < 32; ++g)
                        if (col + g < p.N) reinterpret_cast<uint32_t*>(crow)[col + g] = v[g];
                }
            };
            if (w.slice < 0) {
                // whole tile: the tensor-memory read of the next piece is in flight while this one is staged and stored
                uint32_t va[32], vb[32];
                const uint32_t acc = lane_taddr + static_cast<uint32_t>(ab * PAIR_BN + col_first);
                if (nchunks > 0) ptx::tmem_ld_32x32(acc, va);
#pragma unroll 1
                for (int c = 0; c < nchunks; c += 2) {
                    ptx::tmem_ld_wait();
                    if (c + 1 < nchunks) ptx::tmem_ld_32x32(acc + static_cast<uint32_t>((c + 1) * 32), vb);
                    export_piece(va, col_first + c * 32);
                    if (c + 1 < nchunks) {
                        ptx::tmem_ld_wait();
                        if (c + 2 < nchunks) ptx::tmem_ld_32x32(acc + static_cast<uint32_t>((c + 2) * 32), va);
                        export_piece(vb, col_first + (c + 1) * 32);
                    }
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_remote(&ctl->acc_empty[ab], 0);
                continue;
            }
            // k-slice of a tail tile
            pair_tail_strip<Out>(p, w, static_cast<int>(rank) * PAIR_EPI_WARPS + ew, lane_taddr + static_cast<uint32_t>(ab * PAIR_BN), col_first, nchunks,
                                 lane, &ctl->acc_empty[ab], export_piece);
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
