// Tensor-core kernel for the bf16 and int8 recurrences (and TF32 building block).
//
// Mapping of the weight-stationary array onto one SM: a CTA owns a BM x BN block
// of C, i.e. the cells of BM rows i for all k, over BN time steps j.
//   * the stationary weights [i,k]_W = A_ik and the injected column values
//     B_kj arrive as TMA tiles in a multi-stage shared-memory ring (mbarrier
//     full/empty pairs) -- the ring replaces the north->south forwarding of B:
//     one B tile in shared memory is read by all BM rows of the MMA;
//   * the running partial sum [i,k]_C lives in tensor memory (TMEM) for the whole
//     k loop -- the west->east forward never touches memory; k-blocks are issued
//     in increasing order by one thread, the first with accumulate disabled
//     (the zero entering at the west boundary);
//   * at k_end the epilogue warps read the accumulator with tcgen05.ld and write
//     C_ij, while the MMA warp already works on the next tile in the second
//     TMEM buffer.
// Roles: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM), warps 2..5 =
// epilogue.  Persistent CTAs walk the tile list (batch, m-tile, n-tile).
// Every wait is bounded; a wait that runs out raises a status word and all roles
// leave their loops.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "ptx.cuh"

namespace cyc {

constexpr int UMMA_THREADS = 192;
constexpr int UMMA_BM = 128;
constexpr long long UMMA_WAIT_CYCLES = 1ll << 31;  // about a second

enum UmmaKind { KIND_BF16 = 0, KIND_I8 = 1, KIND_TF32 = 2 };

struct UmmaParams {
    void* C;
    int M, N, K;
    long long sC;  // batch stride of C, elements
    int tiles_m, tiles_n;
    long long num_tiles;
    int* status;  // device status word
};

template <int KIND>
struct UmmaTraits;
template <>
struct UmmaTraits<KIND_BF16> {
    static constexpr int ELEM_BYTES = 2, FMT = 1, CFMT = 1;
    using Out = float;
};
template <>
struct UmmaTraits<KIND_I8> {
    static constexpr int ELEM_BYTES = 1, FMT = 1, CFMT = 2;
    using Out = int32_t;
};
template <>
struct UmmaTraits<KIND_TF32> {
    static constexpr int ELEM_BYTES = 4, FMT = 2, CFMT = 1;
    using Out = float;
};

// 64-bit shared-memory matrix descriptor, 128-byte swizzle.
//   bits [0,14) start address >> 4 ; [16,30) leading-dimension byte offset >> 4 ;
//   [32,46) stride-dimension byte offset >> 4 ; [46,48) = 1 ; [61,64) swizzle: 2 = 128 B rows
//   with 16-byte chunks permuted over 8 rows, 1 = 128 B rows with 32-byte chunks permuted over 4
//   rows (the only MN-major layout for 32-bit operands)
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle = 2) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= static_cast<uint64_t>(swizzle) << 61;
    return d;
}

// 32-bit instruction descriptor: [4,6) D format, [7,10) A format, [10,13) B format,
// bit 15 A major (0 = K), bit 16 B major (1 = MN), [17,23) N >> 3, [24,29) M >> 4.
__host__ __device__ constexpr uint32_t umma_instr_desc(int cfmt, int fmt, bool b_mn_major, int m, int n) {
    return (static_cast<uint32_t>(cfmt) << 4) | (static_cast<uint32_t>(fmt) << 7) | (static_cast<uint32_t>(fmt) << 10) |
           (static_cast<uint32_t>(b_mn_major ? 1 : 0) << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(m >> 4) << 24);
}

template <int KIND, bool B_MN, int BN, int STAGES>
struct UmmaSmem {
    using Tr = UmmaTraits<KIND>;
    static constexpr int BK = 128 / Tr::ELEM_BYTES;          // one 128-byte swizzle row of k
    static constexpr int A_BYTES = UMMA_BM * 128;            // BM rows x 128 B
    static constexpr int B_BYTES = BN * 128;                 // K-major: BN rows x 128 B ; MN-major: (BN/CH) boxes of BK rows x 128 B
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int BAR_BYTES = 1024;
    static constexpr int TOTAL = STAGES * STAGE_BYTES + BAR_BYTES + 1024;  // + alignment slack
};

struct UmmaCtl {  // lives in the barrier page of shared memory
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    volatile int abort;
};

__device__ __forceinline__ bool umma_wait(uint64_t* bar, uint32_t parity, UmmaCtl* ctl, int* status, int where) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (ctl->abort) return false;
        if (clock64() - t0 > UMMA_WAIT_CYCLES) {
            ctl->abort = 1;
            atomicExch(status, 0x100 | where);
            return false;
        }
    }
    return true;
}

// tile index -> (batch, m-tile, n-tile).  Inside a batch entry tiles are walked in
// bands of 16 m-tiles, n-tile by n-tile, so that CTAs running together share A and B panels in L2.
__device__ __forceinline__ void umma_tile_coord(long long t, int tiles_m, int tiles_n, int& b, int& tm, int& tn) {
    const long long per_batch = static_cast<long long>(tiles_m) * tiles_n;
    b = static_cast<int>(t / per_batch);
    int r = static_cast<int>(t - b * per_batch);
    constexpr int BAND = 16;
    const int band_tiles = BAND * tiles_n;
    const int band = r / band_tiles;
    const int in_band = r - band * band_tiles;
    const int rows_in_band = min(BAND, tiles_m - band * BAND);
    tm = band * BAND + in_band % rows_in_band;
    tn = in_band / rows_in_band;
}

template <int KIND, bool B_MN, int BN, int STAGES>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
umma_recurrence_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const UmmaParams p) {
    using Tr = UmmaTraits<KIND>;
    using Sm = UmmaSmem<KIND, B_MN, BN, STAGES>;
    using Out = typename Tr::Out;
    constexpr int BK = Sm::BK;
    constexpr int UK = 32 / Tr::ELEM_BYTES;  // k extent of one MMA: 32 bytes
    constexpr int CH = 128 / Tr::ELEM_BYTES; // MN-major B: n extent of one 128-byte swizzle row
    constexpr uint32_t TMEM_COLS = 2 * BN;   // two accumulators (512 columns at BN = 256)
    static_assert(TMEM_COLS == 128 || TMEM_COLS == 256 || TMEM_COLS == 512, "TMEM allocation must be a power of two");
    static_assert(STAGES <= 8, "control block holds 8 stage barriers");
    constexpr uint32_t IDESC = umma_instr_desc(Tr::CFMT, Tr::FMT, B_MN, UMMA_BM, BN);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    UmmaCtl* ctl = reinterpret_cast<UmmaCtl*>(smem + STAGES * Sm::STAGE_BYTES);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_kb = (p.K + BK - 1) / BK;

    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&ctl->full[s], 1);
            ptx::mbar_init(&ctl->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&ctl->acc_full[a], 1);
            ptx::mbar_init(&ctl->acc_empty[a], 4);
        }
        ctl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
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
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            ptx::grid_dependency_wait();  // the set-up above may overlap the previous kernel; nothing it wrote is read before it ends
            for (long long t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x) {
                int b, tm, tn;
                umma_tile_coord(t, p.tiles_m, p.tiles_n, b, tm, tn);
                const int m0 = tm * UMMA_BM, n0 = tn * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!umma_wait(&ctl->empty[stage], phase ^ 1, ctl, p.status, 1)) { ok = false; break; }
                    uint8_t* sa = smem + stage * Sm::STAGE_BYTES;
                    uint8_t* sb = sa + Sm::A_BYTES;
                    ptx::mbar_arrive_expect_tx(&ctl->full[stage], Sm::STAGE_BYTES);
                    // weights A_ik of rows m0.., k-slab kb  (tensor map dims: k, i, batch)
                    ptx::tma_load_3d(sa, &tmA, &ctl->full[stage], kb * BK, m0, b);
                    if constexpr (!B_MN) {
                        // B stored [N][K]: one box of BN rows j x 128 bytes of k  (dims: k, j, batch)
                        ptx::tma_load_3d(sb, &tmB, &ctl->full[stage], kb * BK, n0, b);
                    } else {
                        // B stored [K][N]: boxes of BK rows k x 128 bytes of j  (dims: j, k, batch)
#pragma unroll
                        for (int c = 0; c < BN / CH; ++c)
                            ptx::tma_load_3d(sb + c * (BK * 128), &tmB, &ctl->full[stage], n0 + c * CH, kb * BK, b);
                    }
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {
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
        // ------------------------------------------------------------ MMA issuer: the whole warp walks the loop
        // ------------------------------------------------------------ converged, one elected lane issues
        {
            const uint32_t leader = ptx::elect_one();
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            bool ok = true;
            for (long long t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x, ++local) {
                const int ab = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1;
                if (!umma_wait(&ctl->acc_empty[ab], acc_phase ^ 1, ctl, p.status, 2)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ab * BN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!umma_wait(&ctl->full[stage], phase, ctl, p.status, 3)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t sa = ptx::smem_u32(smem + stage * Sm::STAGE_BYTES);
                    const uint32_t sb = sa + Sm::A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / UK; ++k) {
                        // A, K-major: rows 128 B apart, 8-row groups 1024 B apart; k advances 32 B inside the swizzle row
                        const uint64_t adesc = umma_smem_desc(sa + k * 32, 16, 1024);
                        uint64_t bdesc;
                        if constexpr (!B_MN) bdesc = umma_smem_desc(sb + k * 32, 16, 1024);
                        // B, MN-major: 128-byte rows of j, 8 k-rows per 1024 B group (stride dim), next j chunk BK*128 B on (leading dim)
                        else bdesc = umma_smem_desc(sb + k * (UK * 128), BK * 128, 1024);
                        ptx::umma_elect<KIND, 1>(d_tmem, adesc, bdesc, IDESC, (kb | k) != 0 ? 1u : 0u, leader);
                    }
                    ptx::umma_commit_elect(&ctl->empty[stage], leader);  // stage reusable once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) ptx::umma_commit_elect(&ctl->acc_full[ab], leader);  // [i,k_end]_C complete for this tile
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue: C_ij <- [i,k_end]_C
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        int local = 0;
        bool ok = true;
        const bool vec_ok = (p.N % 4 == 0) && ((reinterpret_cast<uintptr_t>(p.C) & 15) == 0) && (p.sC % 4 == 0);
        for (long long t = blockIdx.x; t < p.num_tiles && ok; t += gridDim.x, ++local) {
            const int ab = local & 1;
            const uint32_t acc_phase = (local >> 1) & 1;
            int b, tm, tn;
            umma_tile_coord(t, p.tiles_m, p.tiles_n, b, tm, tn);
            if (!umma_wait(&ctl->acc_full[ab], acc_phase, ctl, p.status, 4)) { ok = false; break; }
            ptx::tc_fence_after();
            const int row = tm * UMMA_BM + q * 32 + lane;
            Out* crow = static_cast<Out*>(p.C) + static_cast<long long>(b) * p.sC + static_cast<long long>(row) * p.N;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + static_cast<uint32_t>(ab * BN + c0), v);
                ptx::tmem_ld_wait();
                const int col = tn * BN + c0;
                if (row < p.M && col < p.N) {
                    if (vec_ok && col + 32 <= p.N) {
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            *reinterpret_cast<uint4*>(crow + col + 4 * g) = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                    } else {
#pragma unroll
                        for (int g = 0; g < 32; ++g)
                            if (col + g < p.N) reinterpret_cast<uint32_t*>(crow)[col + g] = v[g];
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->acc_empty[ab]);
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc<1>(tmem_base, TMEM_COLS);
    }
}

}  // namespace cyc
