// Weight-stationary form of the fp32 recurrence on tensor cores, for a small B (K <= 256, N <= 256) under a long A:
// the shape the paper's weight-stationary program is written for -- the weights stay in the array, the other operand
// streams past them (Section "Space-time Mappings of Dataflow Recurrences").
//
// The product is evaluated transposed, C^T = B^T A^T, so that the STATIONARY operand is the one a tcgen05 MMA can take
// from tensor memory: per CTA pair, B^T (n x k) is split once into hi + lo TF32 parts; hi goes to tensor memory
// (lane = n, 128 lanes per CTA, column = k), lo to shared memory (K-major, 128-byte swizzle).  A then streams through a
// shared-memory ring in tiles of 128 rows (64 per CTA, 32 values of k a stage) and is split as in
// umma_pair_tf32x3_kernel.cuh (the landed tile is the hi part as it stands, split warps write the lo part), and each
// k-step accumulates
//      B^T_hi * A_lo + B^T_lo * A_hi + B^T_hi * A_hi
// into a 128-column accumulator (lane = n, column = row of A): two of the three MMAs read their first operand from
// tensor memory, and nothing of B crosses shared memory again after the prologue.  Against the tile-by-tile kernel this
// takes a third of the shared-memory traffic per row of A away (B is neither copied nor split per tile, and its hi part
// is never read from shared memory), which is what bounds that kernel on this shape.
// Export: a lane holds C[row][n] for 32 consecutive rows of A, so the 32 lanes of a warp hold 32 consecutive n of each
// row: the warp lays 16 rows x 128 bytes into a staging buffer of its own (conflict-free) and hands them to a TMA store,
// two such buffers in turn.  (Plain stores from registers, 128 bytes per instruction, were measured at 67 clocks per
// instruction and made the export the longest path of the kernel.)
//
// B stored [N][K] is B^T as it stands: its tiles land by TMA directly where the lo parts belong, in the layout the MMA
// reads; B stored [K][N] passes through two buffers borrowed from the still idle ring and is transposed by the threads.
//
// Roles per CTA (320 threads): warp 0 TMA producer, warp 1 MMA issuer (leader CTA), warps 2-9 first split B^T (thread =
// row n = TMEM lane); then warps 2-5 export and warps 6-9 split the A stages.  Every wait is bounded.
#pragma once
#include "umma_kernel.cuh"

namespace cyc {

constexpr int WS_THREADS = 320;
constexpr int WS_BK = 32;                         // fp32 values of k per stage: one 128-byte swizzle row
constexpr int WS_ROWS = 128;                      // rows of A per tile (64 per CTA)
constexpr int WS_HALF = WS_ROWS / 2;
constexpr int WS_KMAX = 256, WS_NMAX = 256;
constexpr int WS_STAGE_RAW = WS_HALF * WS_BK * 4;  // 8 KB: this CTA's 64 rows x 128 B
constexpr int WS_STAGE_BYTES = 2 * WS_STAGE_RAW;   // followed by their lo parts
constexpr int WS_STAGES = 5;
constexpr int WS_WLO_BYTES = (WS_KMAX / WS_BK) * 128 * 128;  // 8 slabs of 128 rows (n) x 128 B: 128 KB
constexpr int WS_TEMP_BYTES = 4 * 64 * 128;                  // a quarter of B^T's k range as landed: 4 boxes of 64 k x 32 n
static_assert(2 * WS_TEMP_BYTES <= WS_STAGES * WS_STAGE_BYTES, "the prologue borrows the ring for two such buffers");
constexpr int WS_STAGING_BYTES = 4 * 2 * 16 * 128;           // per export warp two buffers of 16 rows x 128 B
constexpr int WS_SMEM_BYTES = WS_WLO_BYTES + WS_STAGES * WS_STAGE_BYTES + WS_STAGING_BYTES + 1024 + 1024;

struct WsParams {
    float* C;         // [M][N]
    int M, N, K;
    long long tiles;  // ceil(M / 128)
    int* status;
};

struct WsCtl {
    uint64_t full[8];      // stage: copy landed (per CTA)
    uint64_t ready[8];     // stage: lo parts written, both CTAs (leader)
    uint64_t empty[8];     // stage: MMAs done (both, by the leader's multicast commit)
    uint64_t acc_full[2];  // accumulator complete (both)
    uint64_t acc_empty[2]; // accumulator read out, both CTAs (leader)
    uint64_t w_full[2];    // a quarter of B^T landed in one of two buffers borrowed from the ring (per CTA)
    uint64_t w_free[2];    // ... and consumed (per CTA, 8 warps)
    uint64_t w_ready;      // B^T split and in place, both CTAs (leader, 16 warps)
    uint32_t tmem_base;
    volatile int abort;
};

__device__ __forceinline__ bool ws_wait(uint64_t* bar, uint32_t parity, WsCtl* ctl, int* status, int where) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (ctl->abort) return false;
        if (clock64() - t0 > UMMA_WAIT_CYCLES) {
            ctl->abort = 1;
            atomicExch(status, 0x400 | where);
            return false;
        }
    }
    return true;
}

// fp32 bit pattern -> nearest TF32, low 13 bits cleared (integer arithmetic on the encoding)
__device__ __forceinline__ uint32_t ws_tf32_round(uint32_t bits) { return (bits + 0x1000u) & 0xFFFFE000u; }
// lo part of x: tf32(x - hi), hi = x with its 13 low significand bits dropped; inf / NaN stay in the hi part only
__device__ __forceinline__ uint32_t ws_lo(uint32_t x) {
    const uint32_t hi = x & 0xFFFFE000u;
    const float r = __uint_as_float(x) - __uint_as_float(hi);
    return ((x & 0x7F800000u) == 0x7F800000u) ? 0u : ws_tf32_round(__float_as_uint(r));
}

// D[tmem] (+)= A[tmem] * B[smem], TF32, CTA pair, issued by the elected lane of a converged warp
__device__ __forceinline__ void ws_umma_tmem_a(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate, uint32_t leader) {
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "setp.ne.b32 q, %5, 0;\n"
        "@q tcgen05.mma.cta_group::2.kind::tf32 [%0], [%1], %2, %3, p;\n"
        "}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(leader)
        : "memory");
}
__device__ __forceinline__ void ws_tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
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
__device__ __forceinline__ void ws_tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// tmA: A as [M][K] fp32, box 32 k x 64 rows, 128-byte swizzle.  tmC: C as [M][N] fp32, box 32 n x 16 rows, no swizzle.
// tmW: B stored [K][N] (B_NK = false): box 32 n x 64 k, no swizzle; B stored [N][K] (B_NK = true: B^T as it is in memory):
// box 32 k x 128 n, 128-byte swizzle -- the tiles then land in the layout the MMA reads, and the lo parts replace them
// in place.
template <bool B_NK>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(WS_THREADS, 1)
umma_ws_tf32x3_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                      const __grid_constant__ CUtensorMap tmC, const WsParams p) {
    constexpr int UK = 8;                       // k extent of one kind::tf32 MMA
    constexpr uint32_t TMEM_COLS = 512;         // B^T_hi (256 columns of k) | accumulator 0 | accumulator 1 (128 each)
    constexpr uint32_t COL_ACC = 256;
    constexpr uint32_t IDESC = umma_instr_desc(1, 2, false, 256, WS_ROWS);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* w_lo = smem;                        // B^T_lo: slab j (k in [32 j, 32 j + 32)) at j * 16 KB, row n at n * 128
    uint8_t* ring = smem + WS_WLO_BYTES;
    uint8_t* staging = ring + WS_STAGES * WS_STAGE_BYTES;
    WsCtl* ctl = reinterpret_cast<WsCtl*>(staging + WS_STAGING_BYTES);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const long long pair = blockIdx.x >> 1;
    const long long num_pairs = gridDim.x >> 1;
    const int num_kb = (p.K + WS_BK - 1) / WS_BK;

    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < WS_STAGES; ++s) {
            ptx::mbar_init(&ctl->full[s], 1);
            ptx::mbar_init(&ctl->ready[s], 8);   // four split warps in each CTA
            ptx::mbar_init(&ctl->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(&ctl->acc_full[a], 1);
            ptx::mbar_init(&ctl->acc_empty[a], 8);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&ctl->w_full[b], 1);
            ptx::mbar_init(&ctl->w_free[b], 8);
        }
        ptx::mbar_init(&ctl->w_ready, 16);
        ctl->abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmW);
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

    // B^T into place (warps 2-9, thread = row n of this CTA's half = TMEM lane): of every landed quarter (64 values of k) the
    // warps 2-5 take the first 32, the warps 6-9 the second; hi parts to tensor memory, lo parts to shared memory in the
    // K-major swizzled layout the MMA reads.
    auto place_weights = [&](int part) -> bool {
        const int q = warp & 3;                  // TMEM lane quarter this warp may access
        const int n_loc = q * 32 + lane;
        const uint32_t lane_taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        if constexpr (B_NK) {
            // all eight slabs landed in place (row n at n * 128, 16-byte chunks permuted by n % 8): hi parts out, lo parts over them
            if (!ws_wait(&ctl->w_full[0], 0, ctl, p.status, 8)) return false;
            for (int j = part; j < WS_KMAX / WS_BK; j += 2) {
                uint8_t* row = w_lo + j * (128 * 128) + n_loc * 128;
                uint32_t hi[32];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint4* ptr = reinterpret_cast<uint4*>(row + ((c ^ (n_loc & 7)) << 4));
                    const uint4 x = *ptr;
                    hi[4 * c] = x.x & 0xFFFFE000u; hi[4 * c + 1] = x.y & 0xFFFFE000u;
                    hi[4 * c + 2] = x.z & 0xFFFFE000u; hi[4 * c + 3] = x.w & 0xFFFFE000u;
                    *ptr = make_uint4(ws_lo(x.x), ws_lo(x.y), ws_lo(x.z), ws_lo(x.w));
                }
                ws_tmem_st_32x32(lane_taddr + static_cast<uint32_t>(j * WS_BK), hi);
            }
            ws_tmem_st_wait();
        }
        for (int qi = 0; qi < (B_NK ? 0 : 4); ++qi) {
            const int b = qi & 1;
            if (!ws_wait(&ctl->w_full[b], (qi >> 1) & 1, ctl, p.status, 8)) return false;
            // landed: box c = n_loc / 32 holds 64 rows k (128 B each) of 32 columns n
            const uint8_t* src = ring + b * WS_TEMP_BYTES + (n_loc >> 5) * (64 * 128) + (n_loc & 31) * 4 + part * 32 * 128;
            const int k0 = qi * 64 + part * 32;
            uint8_t* slab = w_lo + (k0 / WS_BK) * (128 * 128) + n_loc * 128;
            uint32_t hi[32];
#pragma unroll
            for (int c = 0; c < 8; ++c) {    // 16-byte chunk c of the row: four values of k
                uint32_t lo4[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t x = *reinterpret_cast<const uint32_t*>(src + (4 * c + e) * 128);
                    hi[4 * c + e] = x & 0xFFFFE000u;
                    lo4[e] = ws_lo(x);
                }
                *reinterpret_cast<uint4*>(slab + ((c ^ (n_loc & 7)) << 4)) = make_uint4(lo4[0], lo4[1], lo4[2], lo4[3]);
            }
            ws_tmem_st_32x32(lane_taddr + static_cast<uint32_t>(k0), hi);
            ws_tmem_st_wait();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->w_free[b]);   // the borrowed buffer may be overwritten
        }
        ptx::fence_proxy_async_smem();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            if (rank == 0) ptx::mbar_arrive(&ctl->w_ready);
            else ptx::mbar_arrive_remote(&ctl->w_ready, 0);
        }
        return true;
    };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs, own barriers)
        if (lane == 0) {
            bool ok = true;
            ptx::grid_dependency_wait();  // the set-up above may overlap the previous kernel; nothing it wrote is read before it ends
            // B^T, this CTA's 128 columns n, in four quarters of k through two buffers in the (still idle) ring
            int wq = 0;   // quarters requested
            if constexpr (B_NK) {   // B^T as stored: straight into its place, the ring stays free
                wq = 1;
                ptx::mbar_arrive_expect_tx(&ctl->w_full[0], WS_WLO_BYTES);
#pragma unroll
                for (int j = 0; j < WS_KMAX / WS_BK; ++j)
                    ptx::tma_load_3d(w_lo + j * (128 * 128), &tmW, &ctl->w_full[0], j * WS_BK, static_cast<int>(rank) * 128, 0);
            }
            for (int qi = 0; qi < (B_NK ? 0 : 4) && ok; ++qi) {
                const int b = qi & 1;
                if (qi >= 2 && !ws_wait(&ctl->w_free[b], 0, ctl, p.status, 1)) { ok = false; break; }
                ++wq;
                ptx::mbar_arrive_expect_tx(&ctl->w_full[b], WS_TEMP_BYTES);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    ptx::tma_load_3d(ring + b * WS_TEMP_BYTES + c * (64 * 128), &tmW, &ctl->w_full[b], static_cast<int>(rank) * 128 + c * 32, qi * 64, 0);
            }
            for (int b = 0; b < (B_NK ? 0 : 2) && ok; ++b)   // the ring is the ring again
                if (!ws_wait(&ctl->w_free[b], 1, ctl, p.status, 2)) ok = false;
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            for (long long tile = pair; ok && tile < p.tiles; tile += num_pairs) {
                const int row0 = static_cast<int>(tile) * WS_ROWS + static_cast<int>(rank) * WS_HALF;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!ws_wait(&ctl->empty[stage], phase ^ 1, ctl, p.status, 3)) { ok = false; break; }
                    ptx::mbar_arrive_expect_tx(&ctl->full[stage], WS_STAGE_RAW);
                    ptx::tma_load_3d(ring + stage * WS_STAGE_BYTES, &tmA, &ctl->full[stage], kb * WS_BK, row0, 0);
                    ++issued;
                    if (++stage == WS_STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok) {  // leave no copy in flight: wait (bounded) for what was issued
                const long long t0 = clock64();
                for (int b = 0; b < 2; ++b) {
                    const int uses = (wq + 1 - b) / 2;   // copies into buffer b
                    while (uses > 0 && !ptx::mbar_try_wait(&ctl->w_full[b], (uses - 1) & 1) && clock64() - t0 < UMMA_WAIT_CYCLES) {}
                }
                const int back = issued < WS_STAGES ? static_cast<int>(issued) : WS_STAGES;
                int s = stage;
                uint32_t ph = phase;
                for (int n = 0; n < back; ++n) {
                    if (--s < 0) { s = WS_STAGES - 1; ph ^= 1; }
                    const long long t1 = clock64();
                    while (!ptx::mbar_try_wait(&ctl->full[s], ph) && clock64() - t1 < UMMA_WAIT_CYCLES) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (rank == 0) {  // the whole warp walks the loop converged, one elected lane issues
            const uint32_t leader = ptx::elect_one();
            bool ok = ws_wait(&ctl->w_ready, 0, ctl, p.status, 4);
            ptx::tc_fence_after();
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            // An MMA of this shape runs for 64 clocks: every instruction between two of them counts.  Descriptors are
            // built once; a stage, a slab or a k-step only adds its byte offset (in 16-byte units) to the address field,
            // which cannot carry out of its 14 bits below 256 KB.
            const uint64_t ring_desc = umma_smem_desc(ptx::smem_u32(ring), 16, 1024);
            const uint64_t wlo_desc = umma_smem_desc(ptx::smem_u32(w_lo), 16, 1024);
            for (long long tile = pair; ok && tile < p.tiles; tile += num_pairs, ++local) {
                const int ab = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1;
                if (!ws_wait(&ctl->acc_empty[ab], acc_phase ^ 1, ctl, p.status, 5)) { ok = false; break; }
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + COL_ACC + static_cast<uint32_t>(ab * WS_ROWS);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!ws_wait(&ctl->ready[stage], phase, ctl, p.status, 6)) { ok = false; break; }
                    ptx::tc_fence_after();
                    // K-major rows of 128 bytes under the 128-byte swizzle, groups of 8 rows 1024 bytes apart
                    const uint64_t a_stage = ring_desc + static_cast<uint64_t>((stage * WS_STAGE_BYTES) >> 4);
                    const uint64_t w_slab = wlo_desc + static_cast<uint64_t>((kb * (128 * 128)) >> 4);
#pragma unroll
                    for (int k = 0; k < WS_BK / UK; ++k) {
                        const uint64_t a_hi = a_stage + static_cast<uint64_t>((k * 32) >> 4);
                        const uint64_t a_lo = a_hi + static_cast<uint64_t>(WS_STAGE_RAW >> 4);
                        const uint64_t w_lo_d = w_slab + static_cast<uint64_t>((k * 32) >> 4);
                        const uint32_t w_hi_t = tmem_base + static_cast<uint32_t>(kb * WS_BK + k * UK);
                        ws_umma_tmem_a(d_tmem, w_hi_t, a_lo, IDESC, (kb | k) != 0 ? 1u : 0u, leader);
                        ptx::umma_elect<KIND_TF32, 2>(d_tmem, w_lo_d, a_hi, IDESC, 1u, leader);
                        ws_umma_tmem_a(d_tmem, w_hi_t, a_hi, IDESC, 1u, leader);
                    }
                    ptx::umma_commit_pair_elect(&ctl->empty[stage], 3, leader);
                    if (++stage == WS_STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) ptx::umma_commit_pair_elect(&ctl->acc_full[ab], 3, leader);
            }
        }
        __syncwarp();
    } else if (warp >= 6) {
        // ------------------------------------------------------------ split warps: their share of B^T, then the lo parts of
        // ------------------------------------------------------------ the landed A stages
        const int tid = threadIdx.x - 6 * 32;   // 0 .. 127
        int stage = 0;
        uint32_t phase = 0;
        bool ok = place_weights(1);
        for (long long tile = pair; ok && tile < p.tiles; tile += num_pairs) {
            for (int kb = 0; kb < num_kb; ++kb) {
                if (!ws_wait(&ctl->full[stage], phase, ctl, p.status, 7)) { ok = false; break; }
                uint8_t* base = ring + stage * WS_STAGE_BYTES;
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) v[u] = *reinterpret_cast<const uint4*>(base + (tid + 128 * u) * 16);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    *reinterpret_cast<uint4*>(base + WS_STAGE_RAW + (tid + 128 * u) * 16) = make_uint4(ws_lo(v[u].x), ws_lo(v[u].y), ws_lo(v[u].z), ws_lo(v[u].w));
                ptx::fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) ptx::mbar_arrive(&ctl->ready[stage]);
                    else ptx::mbar_arrive_remote(&ctl->ready[stage], 0);
                }
                if (++stage == WS_STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------ warps 2-5: their share of B^T, then the export
        const int q = warp & 3;                  // TMEM lane quarter this warp may access
        const int n_loc = q * 32 + lane;         // row of B^T in this CTA = TMEM lane
        const uint32_t lane_taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        bool ok = place_weights(0);
        // ---- export: C[row][n] <- accumulator (lane = n, column = row of the tile)
        const int n0 = static_cast<int>(rank) * 128 + q * 32;   // this warp's 32 columns of C
        uint8_t* my_stage = staging + (warp - 2) * (2 * 16 * 128);
        int sbuf = 0, local = 0;
        auto export_rows = [&](const uint32_t (&v)[32], int row) {   // 32 rows starting at `row`, as two stores of 16
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint8_t* buf = my_stage + sbuf * (16 * 128);
                if (lane == 0) ptx::tma_store_wait_read<1>();   // the store before the last has read this buffer
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 16; ++j) *reinterpret_cast<uint32_t*>(buf + j * 128 + lane * 4) = v[half * 16 + j];
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && n0 < p.N && row + half * 16 < p.M) {   // the store clips at the edges of C
                    ptx::tma_store_3d(&tmC, buf, n0, row + half * 16, 0);
                    ptx::tma_store_commit();
                }
                sbuf ^= 1;
            }
        };
        for (long long tile = pair; ok && tile < p.tiles; tile += num_pairs, ++local) {
            const int ab = local & 1;
            const uint32_t acc_phase = (local >> 1) & 1;
            if (!ws_wait(&ctl->acc_full[ab], acc_phase, ctl, p.status, 9)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint32_t acc = lane_taddr + COL_ACC + static_cast<uint32_t>(ab * WS_ROWS);
            const int row0 = static_cast<int>(tile) * WS_ROWS;
            uint32_t va[32], vb[32];
            ptx::tmem_ld_32x32(acc, va);
#pragma unroll 1
            for (int c = 0; c < WS_ROWS / 32; c += 2) {   // the tensor-memory read of the next piece is in flight meanwhile
                ptx::tmem_ld_wait();
                ptx::tmem_ld_32x32(acc + (c + 1) * 32, vb);
                export_rows(va, row0 + c * 32);
                ptx::tmem_ld_wait();
                if (c + 2 < WS_ROWS / 32) ptx::tmem_ld_32x32(acc + (c + 2) * 32, va);
                export_rows(vb, row0 + (c + 1) * 32);
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
