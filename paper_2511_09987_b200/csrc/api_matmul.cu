// The matrix-multiply recurrence: kernel selection, tensor-map construction, launches, and the entry points
// cyc_recurrence_matmul, _batched, _host, _splitk_static, cyc_kernel_for and cyc_schedule_for.  See include/cyc.h.
#include <cstdlib>

#include "api_internal.h"
#include "simt_kernel.cuh"
#include "umma_kernel.cuh"
#include "umma_pair_kernel.cuh"
#include "umma_pair_tall_kernel.cuh"
#include "splitk_reduce_kernel.cuh"
#include "umma_pair_tf32x3_kernel.cuh"
#include "umma_ws_tf32x3_kernel.cuh"

namespace cyc {

// Fixed workspace of cyc_recurrence_matmul_splitk_static: lives in every device that loads the library, from load
// to exit.  In host code this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) unsigned char g_static_workspace[CYC_STATIC_WORKSPACE_BYTES];

// host-side validation; no CUDA call
int validate(const Problem& q) {
    if (q.dtype != CYC_F32 && q.dtype != CYC_BF16_F32 && q.dtype != CYC_I8_I32) return CYC_ERR_INVALID_ARG;
    if (q.flags & ~(CYC_FLAG_FIXED_K_ORDER | CYC_FLAG_B_COL_MAJOR)) return CYC_ERR_INVALID_ARG;
    if (q.batch <= 0 || q.M <= 0 || q.N <= 0 || q.K <= 0) return CYC_ERR_INVALID_ARG;
    if (!q.A || !q.B || !q.C) return CYC_ERR_INVALID_ARG;
    if (q.sA < q.M * q.K || q.sB < q.K * q.N || q.sC < q.M * q.N) return CYC_ERR_INVALID_ARG;
    const int eb = elem_bytes(q.dtype);
    if ((reinterpret_cast<uintptr_t>(q.A) % eb) || (reinterpret_cast<uintptr_t>(q.B) % eb) || (reinterpret_cast<uintptr_t>(q.C) % 4))
        return CYC_ERR_INVALID_ARG;
    // C must not overlap A or B
    const uintptr_t c0 = reinterpret_cast<uintptr_t>(q.C), c1 = c0 + static_cast<uintptr_t>((q.batch - 1) * q.sC + q.M * q.N) * 4;
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(q.A), a1 = a0 + static_cast<uintptr_t>((q.batch - 1) * q.sA + q.M * q.K) * eb;
    const uintptr_t b0 = reinterpret_cast<uintptr_t>(q.B), b1 = b0 + static_cast<uintptr_t>((q.batch - 1) * q.sB + q.K * q.N) * eb;
    if ((c0 < a1 && a0 < c1) || (c0 < b1 && b0 < c1)) return CYC_ERR_INVALID_ARG;
    if (q.M > 0x7fffffffll || q.N > 0x7fffffffll || q.K > 0x7fffffffll || q.batch > 0x7fffffffll) return CYC_ERR_UNSUPPORTED;
    if (q.dtype == CYC_I8_I32 && q.K > 131071) return CYC_ERR_UNSUPPORTED;  // int32 partial sums stay exact: K * 2^14 < 2^31
    return CYC_OK;
}

enum Family { FAM_SIMT = 0, FAM_UMMA = 1, FAM_UMMA_3XTF32 = 2, FAM_UMMA_PAIR = 3, FAM_UMMA_TALL = 4, FAM_UMMA_SPLITK = 5, FAM_UMMA_3XTF32_WS = 6 };

// the tensor-core kernels move tiles with TMA: 16-byte aligned bases and pitches
static bool tma_ok(const Problem& q) {
    const int eb = elem_bytes(q.dtype);
    const bool colmajor = (q.flags & CYC_FLAG_B_COL_MAJOR) != 0;
    if (reinterpret_cast<uintptr_t>(q.A) % 16 || reinterpret_cast<uintptr_t>(q.B) % 16) return false;
    if ((lda_of(q) * eb) % 16) return false;            // A pitch
    (void)colmajor;
    if ((ldb_of(q) * eb) % 16) return false;            // B pitch ([N][K] or [K][N] storage)
    if (q.batch > 1 && ((q.sA * eb) % 16 || (q.sB * eb) % 16)) return false;
    return true;
}

// Split-K plan for problems with too few 256 x 256 tiles to occupy the CTA pairs but a long k loop:
// S slices of kb_per_slice k-blocks (at least 8 each), so that tiles * S approaches the number of pairs.
// Not used under CYC_FLAG_FIXED_K_ORDER (the flag promises one owner per C_ij).
struct SplitPlan {
    int S = 1, kb_per_slice = 0;
};
static SplitPlan plan_split_k(const Problem& q) {
    SplitPlan sp;
    if (q.flags & CYC_FLAG_FIXED_K_ORDER) return sp;
    const int bk = 128 / elem_bytes(q.dtype);
    const long long nkb = (q.K + bk - 1) / bk;
    const long long tiles = q.batch * ((q.M + 255) / 256) * ((q.N + 255) / 256);
    if (tiles * 2 > kCtaPairs || nkb < 16) return sp;
    long long S = kCtaPairs / tiles;
    if (S > nkb / 8) S = nkb / 8;
    if (S < 2) return sp;
    sp.kb_per_slice = static_cast<int>((nkb + S - 1) / S);
    sp.S = static_cast<int>((nkb + sp.kb_per_slice - 1) / sp.kb_per_slice);  // no empty slice
    if (sp.S < 2) sp = SplitPlan();
    return sp;
}

static Family choose(const Problem& q) {
    if (q.dtype == CYC_F32) {
        // strict per-element k order or unaligned problems: the general kernel
        if ((q.flags & CYC_FLAG_FIXED_K_ORDER) || !tma_ok(q)) return FAM_SIMT;
        // a small B under a long A: B stays in tensor memory and A streams past it (weight-stationary form); worth its
        // prologue from two 128-row tiles per CTA pair on.  It always does the work of 256 columns, and is still the
        // faster one for any narrower B (65536 x 64 x 256: 34 us against 119 us on the general kernel, whose tiles are 128
        // columns wide whatever N is).
        if (q.batch == 1 && q.N <= WS_NMAX && q.K <= WS_KMAX && q.M >= 2 * WS_ROWS * kCtaPairs &&
            reinterpret_cast<uintptr_t>(q.C) % 16 == 0)
            return FAM_UMMA_3XTF32_WS;
        if (q.M <= 128 || q.N <= 128) return FAM_SIMT;   // too few rows or columns for a CTA pair
        return FAM_UMMA_3XTF32;
    }
    if (!tma_ok(q)) return FAM_SIMT;
    const int bk = 128 / elem_bytes(q.dtype);
    const long long nkb = (q.K + bk - 1) / bk;
    const long long tall_tiles = q.batch * ((q.M + 511) / 512) * ((q.N + 255) / 256);
    // 512 x 256 tiles need a long k loop (their export is not overlapped; measured break-even near 64 k-blocks,
    // a clear gain from 128) and enough tiles to occupy every CTA pair
    if (q.M > 256 && q.N > 128 && nkb >= 96 && tall_tiles >= kCtaPairs) return FAM_UMMA_TALL;
    if (q.M > 128 && q.N > 128)  // enough rows and columns for a CTA pair
        return plan_split_k(q).S > 1 ? FAM_UMMA_SPLITK : FAM_UMMA_PAIR;
    return FAM_UMMA;
}
// ------------------------------------------------------------------ SIMT launch
template <typename TIn, typename TAcc>
static int launch_simt(const Problem& q, cudaStream_t st) {
    SimtParams p;
    p.A = q.A; p.B = q.B; p.C = q.C;
    p.M = static_cast<int>(q.M); p.N = static_cast<int>(q.N); p.K = static_cast<int>(q.K);
    p.sA = q.sA; p.sB = q.sB; p.sC = q.sC;
    p.lda = lda_of(q);
    const bool colmajor = (q.flags & CYC_FLAG_B_COL_MAJOR) != 0;
    p.b_sk = colmajor ? 1 : ldb_of(q);
    p.b_sj = colmajor ? ldb_of(q) : 1;
    p.tiles_m = static_cast<int>((q.M + SIMT_BM - 1) / SIMT_BM);
    p.tiles_n = static_cast<int>((q.N + SIMT_BN - 1) / SIMT_BN);
    const long long blocks = q.batch * p.tiles_m * p.tiles_n;
    if (blocks > 0x7fffffffll) return CYC_ERR_UNSUPPORTED;
    if (blocks < 74) {  // too few large tiles to occupy even half the SMs: smaller tiles, shorter per-thread chains
        p.tiles_m = static_cast<int>((q.M + SIMT_S_BM - 1) / SIMT_S_BM);
        p.tiles_n = static_cast<int>((q.N + SIMT_S_BN - 1) / SIMT_S_BN);
        const long long small_blocks = q.batch * p.tiles_m * p.tiles_n;
        simt_recurrence_small_kernel<TIn, TAcc><<<static_cast<unsigned>(small_blocks), SIMT_THREADS, 0, st>>>(p);
        CYC_CUDA(cudaGetLastError());
        g_launches.fetch_add(1);
        return CYC_OK;
    }
    bool vec = false;
    if constexpr (sizeof(TIn) == 4) {
        vec = !colmajor && q.ldb == 0 && q.K % 4 == 0 && lda_of(q) % 4 == 0 && q.N % 4 == 0 && q.sA % 4 == 0 && q.sB % 4 == 0 && q.sC % 4 == 0 &&
              reinterpret_cast<uintptr_t>(q.A) % 16 == 0 && reinterpret_cast<uintptr_t>(q.B) % 16 == 0 &&
              reinterpret_cast<uintptr_t>(q.C) % 16 == 0;
    }
    if constexpr (sizeof(TIn) == 4) {
        if (vec) simt_recurrence_kernel<TIn, TAcc, true><<<static_cast<unsigned>(blocks), SIMT_THREADS, 0, st>>>(p);
        else simt_recurrence_kernel<TIn, TAcc, false><<<static_cast<unsigned>(blocks), SIMT_THREADS, 0, st>>>(p);
    } else {
        simt_recurrence_kernel<TIn, TAcc, false><<<static_cast<unsigned>(blocks), SIMT_THREADS, 0, st>>>(p);
    }
    CYC_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return CYC_OK;
}
// result map: C[batch][M][N] of 32-bit words, boxes of 32 rows x 32 columns (128 bytes)
static int make_c_map(CUtensorMap* m, int dtype, void* C, long long M, long long N, long long batch, long long sC) {
    const CUtensorMapDataType dt = dtype == CYC_I8_I32 ? CU_TENSOR_MAP_DATA_TYPE_INT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    return make_map_raw(m, dt, 4, C, N, M, batch, N, sC, 32, 32);
}

// ------------------------------------------------------------------ tensor-core launch
template <int KIND, bool B_MN, int BN, int STAGES>
static int launch_umma_cfg(const Problem& q, cudaStream_t st, int sms) {
    using Sm = UmmaSmem<KIND, B_MN, BN, STAGES>;
    constexpr int BK = Sm::BK;
    constexpr int CH = 128 / UmmaTraits<KIND>::ELEM_BYTES;
    CUtensorMap tmA, tmB;
    int rc = make_map(&tmA, q.dtype, q.A, q.K, q.M, q.batch, lda_of(q), q.sA, BK, UMMA_BM);
    if (rc) return rc;
    if (B_MN) rc = make_map(&tmB, q.dtype, q.B, q.N, q.K, q.batch, ldb_of(q), q.sB, CH, BK);
    else rc = make_map(&tmB, q.dtype, q.B, q.K, q.N, q.batch, ldb_of(q), q.sB, BK, BN);
    if (rc) return rc;

    UmmaParams p;
    p.C = q.C;
    p.M = static_cast<int>(q.M); p.N = static_cast<int>(q.N); p.K = static_cast<int>(q.K);
    p.sC = q.sC;
    p.tiles_m = static_cast<int>((q.M + UMMA_BM - 1) / UMMA_BM);
    p.tiles_n = static_cast<int>((q.N + BN - 1) / BN);
    p.num_tiles = q.batch * p.tiles_m * p.tiles_n;
    if (int rc_ = status_word(&p.status)) return rc_;

    auto kern = umma_recurrence_kernel<KIND, B_MN, BN, STAGES>;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), Sm::TOTAL)) return rc_;
    const long long grid = p.num_tiles < sms ? p.num_tiles : sms;
    CYC_CUDA(launch_pdl(kern, static_cast<unsigned>(grid), UMMA_THREADS, Sm::TOTAL, st, tmA, tmB, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}

// ------------------------------------------------------------------ sliced tail of the two-SM kernel
// When the tile count leaves a remainder of at most half the CTA pairs, the remainder tiles are cut into k-slices
// that all pairs work on first (see PairParams).  Not under CYC_FLAG_FIXED_K_ORDER: the flag promises one owner per
// C_ij.  S slices (at most 4) of a minimum length each; S * remainder <= pairs.
struct TailPlan {
    int S = 0, tiles = 0, kb = 0;
};
static TailPlan plan_tail(const Problem& q, long long num_tiles, long long pairs) {
    TailPlan tp;
    if ((q.flags & CYC_FLAG_FIXED_K_ORDER) || num_tiles <= pairs) return tp;
    const int bk = 128 / elem_bytes(q.dtype);
    const long long nkb = (q.K + bk - 1) / bk;
    const long long rem = num_tiles % pairs;
    // bf16 and int8 only: measured on the fp32 (3xTF32) kernel, whose tiles are short, the parked slices cost more than
    // the idle pairs (64 against 50 microseconds on the 65536 x 256 x 256 problem)
    const long long min_kb = 8;  // a slice must amortise its own export
    if (q.dtype == CYC_F32 || rem == 0 || rem * 2 > pairs || nkb < 2 * min_kb) return tp;
    long long S = std::min<long long>({pairs / rem, nkb / min_kb, 4});
    if (S < 2) return tp;
    tp.kb = static_cast<int>((nkb + S - 1) / S);
    tp.S = static_cast<int>((nkb + tp.kb - 1) / tp.kb);  // no empty slice
    tp.tiles = static_cast<int>(rem);
    if (tp.S < 2) tp = TailPlan();
    return tp;
}

// Scratch of the sliced tail: partial-sum slots for up to one slice per CTA pair and one counter per 32-row strip,
// kept per (device, stream) by kept_scratch_for.
constexpr size_t kTailDataBytes = static_cast<size_t>(kCtaPairs) * PAIR_TILE_BYTES;
constexpr size_t kTailCounterBytes = static_cast<size_t>(kCtaPairs) * PAIR_STRIPS * sizeof(int);

// ------------------------------------------------------------------ two-SM tensor-core launch
// `ws` != nullptr: split-K -- the kernel writes plan.S planes of partial sums per problem into ws
template <int KIND, bool B_MN>
static int launch_pair_cfg(const Problem& q, cudaStream_t st, int sms, void* ws = nullptr, SplitPlan plan = SplitPlan()) {
    constexpr int STAGES = PAIR_STAGES;
    constexpr int BK = 128 / UmmaTraits<KIND>::ELEM_BYTES;
    constexpr int CH = 128 / UmmaTraits<KIND>::ELEM_BYTES;
    constexpr int SMEM = pair_smem_bytes<STAGES>();
    CUtensorMap tmA, tmB, tmC;
    int rc = make_map(&tmA, q.dtype, q.A, q.K, q.M, q.batch, lda_of(q), q.sA, BK, PAIR_HALF);
    if (rc) return rc;
    if (B_MN) rc = make_map(&tmB, q.dtype, q.B, q.N, q.K, q.batch, ldb_of(q), q.sB, CH, BK);
    else rc = make_map(&tmB, q.dtype, q.B, q.K, q.N, q.batch, ldb_of(q), q.sB, BK, PAIR_HALF);
    if (rc) return rc;
    PairParams p;
    void* out = ws ? ws : q.C;
    const long long out_planes = ws ? q.batch * plan.S : q.batch;
    const long long out_stride = ws ? q.M * q.N : q.sC;
    p.tma_store = (reinterpret_cast<uintptr_t>(out) % 16 == 0 && q.N % 4 == 0 && (out_planes == 1 || out_stride % 4 == 0)) ? 1 : 0;
    if (p.tma_store) {
        rc = make_c_map(&tmC, q.dtype, out, q.M, q.N, out_planes, out_stride);
        if (rc) return rc;
    } else {
        tmC = tmA;  // never used
    }
    p.C = out;
    p.M = static_cast<int>(q.M); p.N = static_cast<int>(q.N); p.K = static_cast<int>(q.K);
    p.sC = out_stride;
    p.tiles_m = static_cast<int>((q.M + 255) / 256);
    p.tiles_n = static_cast<int>((q.N + PAIR_BN - 1) / PAIR_BN);
    p.num_tiles = out_planes * p.tiles_m * p.tiles_n;
    if (ws) {
        p.split_k = plan.S;
        p.kb_per_slice = plan.kb_per_slice;
    }
    if (int rc_ = status_word(&p.status)) return rc_;
    auto kern = umma_pair_kernel<KIND, B_MN, STAGES>;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), SMEM)) return rc_;
    const long long max_pairs = sms / 2;
    const long long pairs = p.num_tiles < max_pairs ? p.num_tiles : max_pairs;
    if (!ws && pairs <= kCtaPairs) {
        const TailPlan tp = plan_tail(q, p.num_tiles, pairs);
        if (tp.S > 1) {
            uint8_t* data = nullptr;
            int* counters = nullptr;
            if (int rc_ = kept_scratch_for(st, SCRATCH_MATMUL_TAIL, kTailDataBytes, kTailCounterBytes, &data, &counters)) return rc_;
            if (data) {
                p.tail_S = tp.S; p.tail_tiles = tp.tiles; p.tail_kb = tp.kb;
                p.tail_ws = data; p.tail_counters = counters;
            }
        }
    }
    CYC_CUDA(launch_pdl(kern, static_cast<unsigned>(2 * pairs), PAIR_THREADS, SMEM, st, tmA, tmB, tmC, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}
// ------------------------------------------------------------------ split-K
// partial sums of plan.S k-slices into the workspace (CTA-pair kernel), then their sum in slice order into C.
// `ws` = nullptr: the workspace comes from the library's pool for the duration of the two kernels.
template <int KIND>
static int launch_splitk(const Problem& q, cudaStream_t st, int sms, void* ws, const SplitPlan& plan) {
    using Out = typename UmmaTraits<KIND>::Out;
    const long long plane = q.M * q.N;
    const size_t bytes = static_cast<size_t>(q.batch) * plan.S * plane * sizeof(Out);
    const bool pooled = ws == nullptr;
    if (pooled) {
        cudaMemPool_t pool;
        int rc = workspace_pool(&pool);
        if (rc) return rc;
        CYC_CUDA(cudaMallocFromPoolAsync(&ws, bytes, pool, st));
    }
    const bool b_mn = (q.flags & CYC_FLAG_B_COL_MAJOR) == 0;
    int rc = b_mn ? launch_pair_cfg<KIND, true>(q, st, sms, ws, plan) : launch_pair_cfg<KIND, false>(q, st, sms, ws, plan);
    if (rc == CYC_OK) {
        const int vec4 = (plane % 4 == 0 && q.sC % 4 == 0 && reinterpret_cast<uintptr_t>(q.C) % 16 == 0 &&
                          reinterpret_cast<uintptr_t>(ws) % 16 == 0) ? 1 : 0;
        const long long work = (vec4 ? plane / 4 : plane) * q.batch;
        long long blocks = (work + 127) / 128;  // short kernel: spread the work over as many SMs as possible
        if (blocks > 16ll * sms) blocks = 16ll * sms;
        cudaError_t e = launch_pdl(splitk_reduce_kernel<Out>, static_cast<unsigned>(blocks), 128, 0, st, static_cast<const Out*>(ws),
                                   static_cast<Out*>(q.C), plane, q.sC, plan.S, q.batch, vec4);
        if (e != cudaSuccess) rc = cuda_fail(e, "splitk_reduce_kernel launch");
        else g_launches.fetch_add(1);
    }
    if (pooled) {
        cudaError_t e = cudaFreeAsync(ws, st);
        if (e != cudaSuccess && rc == CYC_OK) rc = cuda_fail(e, "cudaFreeAsync");
    }
    return rc;
}

// 512 x 256 tiles: selected when the k loop is long enough to amortise the unoverlapped export
template <int KIND, bool B_MN>
static int launch_pair_tall_cfg(const Problem& q, cudaStream_t st, int sms) {
    constexpr int BK = 128 / UmmaTraits<KIND>::ELEM_BYTES;
    constexpr int CH = 128 / UmmaTraits<KIND>::ELEM_BYTES;
    CUtensorMap tmA, tmB, tmC;
    int rc = make_map(&tmA, q.dtype, q.A, q.K, q.M, q.batch, lda_of(q), q.sA, BK, PAIR_HALF);
    if (rc) return rc;
    if (B_MN) rc = make_map(&tmB, q.dtype, q.B, q.N, q.K, q.batch, ldb_of(q), q.sB, CH, BK);
    else rc = make_map(&tmB, q.dtype, q.B, q.K, q.N, q.batch, ldb_of(q), q.sB, BK, PAIR_HALF);
    if (rc) return rc;
    PairParams p;
    p.tma_store = (reinterpret_cast<uintptr_t>(q.C) % 16 == 0 && q.N % 4 == 0 && (q.batch == 1 || q.sC % 4 == 0)) ? 1 : 0;
    if (p.tma_store) {
        rc = make_c_map(&tmC, q.dtype, q.C, q.M, q.N, q.batch, q.sC);
        if (rc) return rc;
    } else {
        tmC = tmA;  // never used
    }
    p.C = q.C;
    p.M = static_cast<int>(q.M); p.N = static_cast<int>(q.N); p.K = static_cast<int>(q.K);
    p.sC = q.sC;
    p.tiles_m = static_cast<int>((q.M + 511) / 512);
    p.tiles_n = static_cast<int>((q.N + PAIR_BN - 1) / PAIR_BN);
    p.num_tiles = q.batch * p.tiles_m * p.tiles_n;
    if (int rc_ = status_word(&p.status)) return rc_;
    auto kern = umma_pair_tall_kernel<KIND, B_MN>;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), TALL_SMEM_BYTES)) return rc_;
    const long long max_pairs = sms / 2;
    const long long pairs = p.num_tiles < max_pairs ? p.num_tiles : max_pairs;
    CYC_CUDA(launch_pdl(kern, static_cast<unsigned>(2 * pairs), TALL_THREADS, TALL_SMEM_BYTES, st, tmA, tmB, tmC, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}

template <bool B_MN>
static int launch_tf32x3_cfg(const Problem& q, cudaStream_t st, int sms) {
    CUtensorMap tmA, tmB, tmC;
    // K-major tiles: rows of X3_BK fp32 (128 or 64 bytes) under the swizzle of that width
    const CUtensorMapSwizzle ksw = X3_BK == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    int rc = make_map(&tmA, q.dtype, q.A, q.K, q.M, q.batch, lda_of(q), q.sA, X3_BK, PAIR_HALF, ksw);
    if (rc) return rc;
    // fp32 B stored [K][N] feeds the MMA column-contiguous: 32-byte-chunk swizzle (see umma_smem_desc)
    if (B_MN) rc = make_map(&tmB, q.dtype, q.B, q.N, q.K, q.batch, ldb_of(q), q.sB, 32, X3_BK, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B);
    else rc = make_map(&tmB, q.dtype, q.B, q.K, q.N, q.batch, ldb_of(q), q.sB, X3_BK, PAIR_HALF, ksw);
    if (rc) return rc;
    PairParams p;
    p.tma_store = (reinterpret_cast<uintptr_t>(q.C) % 16 == 0 && q.N % 4 == 0 && (q.batch == 1 || q.sC % 4 == 0)) ? 1 : 0;
    if (p.tma_store) {
        rc = make_c_map(&tmC, q.dtype, q.C, q.M, q.N, q.batch, q.sC);
        if (rc) return rc;
    } else {
        tmC = tmA;  // never used
    }
    p.C = q.C;
    p.M = static_cast<int>(q.M); p.N = static_cast<int>(q.N); p.K = static_cast<int>(q.K);
    p.sC = q.sC;
    p.tiles_m = static_cast<int>((q.M + 255) / 256);
    p.tiles_n = static_cast<int>((q.N + PAIR_BN - 1) / PAIR_BN);
    p.num_tiles = q.batch * p.tiles_m * p.tiles_n;
    if (int rc_ = status_word(&p.status)) return rc_;
    auto kern = umma_pair_tf32x3_kernel<B_MN>;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), X3_SMEM_BYTES)) return rc_;
    const long long max_pairs = sms / 2;
    const long long pairs = p.num_tiles < max_pairs ? p.num_tiles : max_pairs;
    CYC_CUDA(launch_pdl(kern, static_cast<unsigned>(2 * pairs), X3_THREADS, X3_SMEM_BYTES, st, tmA, tmB, tmC, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}

// weight-stationary form: B^T resident in tensor memory (hi) and shared memory (lo), A streamed in 128-row tiles
template <bool B_NK>
static int launch_tf32x3_ws(const Problem& q, cudaStream_t st, int sms) {
    CUtensorMap tmA, tmW, tmC;
    int rc = make_map(&tmA, q.dtype, q.A, q.K, q.M, 1, lda_of(q), q.M * q.K, WS_BK, WS_HALF, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    if (B_NK) rc = make_map(&tmW, q.dtype, q.B, q.K, q.N, 1, ldb_of(q), q.K * q.N, WS_BK, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    else rc = make_map(&tmW, q.dtype, q.B, q.N, q.K, 1, ldb_of(q), q.K * q.N, 32, 64, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc) return rc;
    rc = make_map(&tmC, q.dtype, q.C, q.N, q.M, 1, q.N, q.M * q.N, 32, 16, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc) return rc;
    WsParams p;
    p.C = static_cast<float*>(q.C);
    p.M = static_cast<int>(q.M); p.N = static_cast<int>(q.N); p.K = static_cast<int>(q.K);
    p.tiles = (q.M + WS_ROWS - 1) / WS_ROWS;
    if (int rc_ = status_word(&p.status)) return rc_;
    auto kern = umma_ws_tf32x3_kernel<B_NK>;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), WS_SMEM_BYTES)) return rc_;
    const long long max_pairs = sms / 2;
    const long long pairs = p.tiles < max_pairs ? p.tiles : max_pairs;
    CYC_CUDA(launch_pdl(kern, static_cast<unsigned>(2 * pairs), WS_THREADS, WS_SMEM_BYTES, st, tmA, tmW, tmC, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}

static int launch_tf32x3(const Problem& q, cudaStream_t st) {
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    if (di.cc_major != 10) {
        snprintf(g_err, sizeof g_err, "tensor-core kernels need an sm_100 device");
        return CYC_ERR_UNSUPPORTED;
    }
    if (choose(q) == FAM_UMMA_3XTF32_WS)
        return (q.flags & CYC_FLAG_B_COL_MAJOR) ? launch_tf32x3_ws<true>(q, st, di.sms) : launch_tf32x3_ws<false>(q, st, di.sms);
    return (q.flags & CYC_FLAG_B_COL_MAJOR) ? launch_tf32x3_cfg<false>(q, st, di.sms) : launch_tf32x3_cfg<true>(q, st, di.sms);
}

template <int KIND>
static int launch_umma(const Problem& q, cudaStream_t st) {
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    if (di.cc_major != 10) {
        snprintf(g_err, sizeof g_err, "tensor-core kernels need an sm_100 device");
        return CYC_ERR_UNSUPPORTED;
    }
    const bool b_mn = (q.flags & CYC_FLAG_B_COL_MAJOR) == 0;
    const Family fam = choose(q);
    if (fam == FAM_UMMA_TALL)
        return b_mn ? launch_pair_tall_cfg<KIND, true>(q, st, di.sms) : launch_pair_tall_cfg<KIND, false>(q, st, di.sms);
    if (fam == FAM_UMMA_SPLITK) return launch_splitk<KIND>(q, st, di.sms, nullptr, plan_split_k(q));
    if (fam == FAM_UMMA_PAIR)
        return b_mn ? launch_pair_cfg<KIND, true>(q, st, di.sms) : launch_pair_cfg<KIND, false>(q, st, di.sms);
    const bool wide = q.N > 128;
    if (b_mn) return wide ? launch_umma_cfg<KIND, true, 256, 4>(q, st, di.sms) : launch_umma_cfg<KIND, true, 128, 6>(q, st, di.sms);
    return wide ? launch_umma_cfg<KIND, false, 256, 4>(q, st, di.sms) : launch_umma_cfg<KIND, false, 128, 6>(q, st, di.sms);
}

// kernel selection and launch for a validated problem (also used for the sub-problems the library builds itself)
static const char* family_name(Family f) {
    switch (f) {
        case FAM_UMMA: return "tcgen05";
        case FAM_UMMA_PAIR: return "tcgen05_pair";
        case FAM_UMMA_TALL: return "tcgen05_pair_tall";
        case FAM_UMMA_SPLITK: return "tcgen05_pair_splitk";
        case FAM_UMMA_3XTF32: return "tcgen05_3xtf32";
        case FAM_UMMA_3XTF32_WS: return "tcgen05_3xtf32_ws";
        default: return "simt";
    }
}

int route(const Problem& q, cudaStream_t st) {
    if (log_enabled())
        fprintf(stderr, "cyc: batch=%lld M=%lld N=%lld K=%lld dtype=%d flags=0x%x lda=%lld ldb=%lld -> %s\n", q.batch, q.M, q.N, q.K, q.dtype, q.flags,
                lda_of(q), ldb_of(q), family_name(choose(q)));
    switch (choose(q)) {
        case FAM_UMMA:
        case FAM_UMMA_PAIR:
        case FAM_UMMA_TALL:
        case FAM_UMMA_SPLITK:
            return q.dtype == CYC_BF16_F32 ? launch_umma<KIND_BF16>(q, st) : launch_umma<KIND_I8>(q, st);
        case FAM_UMMA_3XTF32:
        case FAM_UMMA_3XTF32_WS:
            return launch_tf32x3(q, st);
        default:
            if (q.dtype == CYC_F32) return launch_simt<float, float>(q, st);
            if (q.dtype == CYC_BF16_F32) return launch_simt<__nv_bfloat16, float>(q, st);
            return launch_simt<int8_t, int>(q, st);
    }
}

int dispatch(const Problem& q, cudaStream_t st) {
    int rc = validate(q);
    if (rc) return rc;
    return route(q, st);
}
}  // namespace cyc

using namespace cyc;

extern "C" int cyc_recurrence_matmul(int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B, void* C,
                                     void* stream, unsigned flags) {
    Problem q{1, M, N, K, dtype, A, B, C, M * K, K * N, M * N, flags};
    if (M <= 0 || N <= 0 || K <= 0) return CYC_ERR_INVALID_ARG;
    return dispatch(q, static_cast<cudaStream_t>(stream));
}

extern "C" int cyc_recurrence_matmul_batched(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A,
                                             int64_t strideA, const void* B, int64_t strideB, void* C, int64_t strideC,
                                             void* stream, unsigned flags) {
    if (batch <= 0 || M <= 0 || N <= 0 || K <= 0 || strideA < 0 || strideB < 0 || strideC < 0) return CYC_ERR_INVALID_ARG;
    Problem q{batch, M, N, K, dtype, A, B, C, strideA ? strideA : M * K, strideB ? strideB : K * N, strideC ? strideC : M * N, flags};
    return dispatch(q, static_cast<cudaStream_t>(stream));
}

// Host-buffer evaluation.  Device buffers come from the library's pool; for large problems the rows of A and C (or the
// problems of a batch) are cut into chunks so that the upload of chunk i+1, the kernel of chunk i and the download of
// chunk i-1 overlap (two helper streams, ordered against the caller's stream by events).  The helper streams and
// events are created once per device and kept; a mutex serialises host-buffer calls on one device (they would share
// the PCIe link anyway).
constexpr int kHostChunksMax = 16;
struct HostPipe {
    bool ready = false;
    cudaStream_t up = nullptr, down = nullptr;
    cudaEvent_t ev_start = nullptr, ev_down = nullptr, ev_up[kHostChunksMax] = {}, ev_done[kHostChunksMax] = {};
    std::mutex mu;
};
static int host_pipe(HostPipe** out) {
    static std::mutex mu;
    static HostPipe pipes[64];
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CYC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(mu);
    HostPipe& hp = pipes[dev];
    if (!hp.ready) {
        CYC_CUDA(cudaStreamCreateWithFlags(&hp.up, cudaStreamNonBlocking));
        CYC_CUDA(cudaStreamCreateWithFlags(&hp.down, cudaStreamNonBlocking));
        CYC_CUDA(cudaEventCreateWithFlags(&hp.ev_start, cudaEventDisableTiming));
        CYC_CUDA(cudaEventCreateWithFlags(&hp.ev_down, cudaEventDisableTiming));
        for (int c = 0; c < kHostChunksMax; ++c) {
            CYC_CUDA(cudaEventCreateWithFlags(&hp.ev_up[c], cudaEventDisableTiming));
            CYC_CUDA(cudaEventCreateWithFlags(&hp.ev_done[c], cudaEventDisableTiming));
        }
        hp.ready = true;
    }
    *out = &hp;
    return CYC_OK;
}

extern "C" int cyc_recurrence_matmul_host(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A_host,
                                          const void* B_host, void* C_host, void* stream, unsigned flags) {
    if (batch <= 0 || M <= 0 || N <= 0 || K <= 0 || !A_host || !B_host || !C_host) return CYC_ERR_INVALID_ARG;
    if (dtype != CYC_F32 && dtype != CYC_BF16_F32 && dtype != CYC_I8_I32) return CYC_ERR_INVALID_ARG;
    if (flags & ~(CYC_FLAG_FIXED_K_ORDER | CYC_FLAG_B_COL_MAJOR)) return CYC_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t eb = static_cast<size_t>(elem_bytes(dtype));
    const size_t na = static_cast<size_t>(batch) * M * K * eb, nb = static_cast<size_t>(batch) * K * N * eb,
                 nc = static_cast<size_t>(batch) * M * N * 4;
    // one allocation, three 256-byte aligned regions
    const size_t oa = 0, ob = (na + 255) & ~static_cast<size_t>(255), oc = ob + ((nb + 255) & ~static_cast<size_t>(255));
    cudaMemPool_t pool;
    int rc = workspace_pool(&pool);
    if (rc) return rc;
    HostPipe* hp = nullptr;
    rc = host_pipe(&hp);
    if (rc) return rc;
    std::lock_guard<std::mutex> pipe_lock(hp->mu);
    uint8_t* d = nullptr;
    CYC_CUDA(cudaMallocFromPoolAsync(reinterpret_cast<void**>(&d), oc + nc, pool, st));
    const uint8_t* hA = static_cast<const uint8_t*>(A_host);
    const uint8_t* hB = static_cast<const uint8_t*>(B_host);
    uint8_t* hC = static_cast<uint8_t*>(C_host);
    cudaError_t e = cudaSuccess;

    // chunks: rows of one problem (multiples of 512), or whole problems of a batch; about 8 MB of traffic each, so
    // that the first kernel starts early and the last download is short
    const bool by_rows = batch == 1;
    const long long units = by_rows ? M : batch;
    long long nch = static_cast<long long>((na + nc) / (8u << 20));
    nch = std::max<long long>(1, std::min<long long>(nch, kHostChunksMax));
    long long per = (units + nch - 1) / nch;
    if (by_rows) per = (per + 511) / 512 * 512;
    if (per < 1) per = 1;
    nch = (units + per - 1) / per;

    if (nch <= 1) {
        if ((e = cudaMemcpyAsync(d + oa, hA, na, cudaMemcpyHostToDevice, st)) != cudaSuccess ||
            (e = cudaMemcpyAsync(d + ob, hB, nb, cudaMemcpyHostToDevice, st)) != cudaSuccess)
            rc = cuda_fail(e, "cudaMemcpyAsync(host to device)");
        if (!rc) {
            Problem q{batch, M, N, K, dtype, d + oa, d + ob, d + oc, M * K, K * N, M * N, flags};
            rc = dispatch(q, st);
        }
        if (!rc && (e = cudaMemcpyAsync(hC, d + oc, nc, cudaMemcpyDeviceToHost, st)) != cudaSuccess)
            rc = cuda_fail(e, "cudaMemcpyAsync(device to host)");
    } else {
        auto ok = [&](cudaError_t err, const char* what) {
            if (err != cudaSuccess && !rc) rc = cuda_fail(err, what);
            return rc == CYC_OK;
        };
        // the helper streams start after whatever the caller's stream holds (the allocation included)
        ok(cudaEventRecord(hp->ev_start, st), "cudaEventRecord");
        ok(cudaStreamWaitEvent(hp->up, hp->ev_start, 0), "cudaStreamWaitEvent");
        ok(cudaStreamWaitEvent(hp->down, hp->ev_start, 0), "cudaStreamWaitEvent");
        if (by_rows && !rc) ok(cudaMemcpyAsync(d + ob, hB, nb, cudaMemcpyHostToDevice, hp->up), "cudaMemcpyAsync(B)");
        for (long long c = 0; c < nch && !rc; ++c) {
            const long long u0 = c * per, un = (u0 + per <= units ? per : units - u0);
            // byte offsets of this chunk in A, B, C
            const size_t a_off = static_cast<size_t>(u0) * (by_rows ? K : M * K) * eb, a_len = static_cast<size_t>(un) * (by_rows ? K : M * K) * eb;
            const size_t c_off = static_cast<size_t>(u0) * (by_rows ? N : M * N) * 4, c_len = static_cast<size_t>(un) * (by_rows ? N : M * N) * 4;
            const size_t b_off = by_rows ? 0 : static_cast<size_t>(u0) * K * N * eb, b_len = by_rows ? 0 : static_cast<size_t>(un) * K * N * eb;
            ok(cudaMemcpyAsync(d + oa + a_off, hA + a_off, a_len, cudaMemcpyHostToDevice, hp->up), "cudaMemcpyAsync(A chunk)");
            if (b_len) ok(cudaMemcpyAsync(d + ob + b_off, hB + b_off, b_len, cudaMemcpyHostToDevice, hp->up), "cudaMemcpyAsync(B chunk)");
            ok(cudaEventRecord(hp->ev_up[c], hp->up), "cudaEventRecord");
            ok(cudaStreamWaitEvent(st, hp->ev_up[c], 0), "cudaStreamWaitEvent");
            if (!rc) {
                Problem q{by_rows ? 1 : un, by_rows ? un : M, N, K, dtype, d + oa + a_off, d + ob + b_off, d + oc + c_off, (by_rows ? un : M) * K, K * N,
                          (by_rows ? un : M) * N, flags};
                rc = dispatch(q, st);
            }
            ok(cudaEventRecord(hp->ev_done[c], st), "cudaEventRecord");
            ok(cudaStreamWaitEvent(hp->down, hp->ev_done[c], 0), "cudaStreamWaitEvent");
            ok(cudaMemcpyAsync(hC + c_off, d + oc + c_off, c_len, cudaMemcpyDeviceToHost, hp->down), "cudaMemcpyAsync(C chunk)");
        }
        // the caller's stream continues (and the buffer is freed) only after the last download
        if (cudaEventRecord(hp->ev_down, hp->down) == cudaSuccess) cudaStreamWaitEvent(st, hp->ev_down, 0);
        else cudaStreamSynchronize(hp->down);
        if (rc) { cudaStreamSynchronize(hp->up); cudaStreamSynchronize(hp->down); }
    }
    cudaFreeAsync(d, st);
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess && !rc) rc = cuda_fail(e, "cudaStreamSynchronize");
    return rc;
}

// Device address of the fixed workspace on the current device, looked up once per device.
static int static_workspace_address(void** out) {
    static std::mutex mu;
    static void* addr[64] = {};
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CYC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        CYC_CUDA(cudaGetSymbolAddress(&p, g_static_workspace));  // the current device's copy of the array
        addr[dev] = p;
    }
    *out = addr[dev];
    return CYC_OK;
}

extern "C" int cyc_recurrence_matmul_splitk_static(int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B,
                                                   void* C, void* stream, unsigned flags) {
    if (M <= 0 || N <= 0 || K <= 0) return CYC_ERR_INVALID_ARG;
    if (flags & CYC_FLAG_FIXED_K_ORDER) return CYC_ERR_INVALID_ARG;  // the flag asks for one owner per C_ij; this schedule has several
    Problem q{1, M, N, K, dtype, A, B, C, M * K, K * N, M * N, flags};
    int rc = validate(q);
    if (rc) return rc;
    if (dtype == CYC_F32 || !tma_ok(q) || M <= 128 || N <= 128) {
        snprintf(g_err, sizeof g_err, "split-K needs bf16 or int8 operands, 16-byte aligned bases and pitches, M > 128 and N > 128");
        return CYC_ERR_UNSUPPORTED;
    }
    // as many k-slices as there are idle CTA pairs, at least 8 k-blocks each, and no more than fit the fixed array
    const int bk = 128 / elem_bytes(dtype);
    const long long nkb = (K + bk - 1) / bk;
    const long long tiles = ((M + 255) / 256) * ((N + 255) / 256);
    const long long plane_bytes = M * N * 4;
    long long S = kCtaPairs / tiles;
    if (S > nkb / 8) S = nkb / 8;
    if (S > static_cast<long long>(CYC_STATIC_WORKSPACE_BYTES) / plane_bytes) S = static_cast<long long>(CYC_STATIC_WORKSPACE_BYTES) / plane_bytes;
    if (S < 2) {
        snprintf(g_err, sizeof g_err,
                 "no split-K plan fits: need >= 2 slices of >= 8 k-blocks, at most %lld CTA pairs' worth of tiles, and "
                 "2*M*N*4 bytes <= the fixed workspace of %lld bytes",
                 static_cast<long long>(kCtaPairs), static_cast<long long>(CYC_STATIC_WORKSPACE_BYTES));
        return CYC_ERR_UNSUPPORTED;
    }
    SplitPlan plan;
    plan.kb_per_slice = static_cast<int>((nkb + S - 1) / S);
    plan.S = static_cast<int>((nkb + plan.kb_per_slice - 1) / plan.kb_per_slice);
    DeviceInfo di;
    rc = device_info(&di);
    if (rc) return rc;
    if (di.cc_major != 10) {
        snprintf(g_err, sizeof g_err, "tensor-core kernels need an sm_100 device");
        return CYC_ERR_UNSUPPORTED;
    }
    void* ws = nullptr;
    rc = static_workspace_address(&ws);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return dtype == CYC_BF16_F32 ? launch_splitk<KIND_BF16>(q, st, di.sms, ws, plan) : launch_splitk<KIND_I8>(q, st, di.sms, ws, plan);
}
extern "C" const char* cyc_kernel_for(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B,
                                      const void* C, unsigned flags) {
    if (batch <= 0 || M <= 0 || N <= 0 || K <= 0) return nullptr;
    Problem q{batch, M, N, K, dtype, A, B, const_cast<void*>(C), M * K, K * N, M * N, flags};
    if (validate(q) != CYC_OK) return nullptr;
    return family_name(choose(q));
}

extern "C" const char* cyc_schedule_for(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B,
                                        const void* C, unsigned flags) {
    if (batch <= 0 || M <= 0 || N <= 0 || K <= 0) return nullptr;
    Problem q{batch, M, N, K, dtype, A, B, const_cast<void*>(C), M * K, K * N, M * N, flags};
    if (validate(q) != CYC_OK) return nullptr;
    const Family fam = choose(q);
    if (fam == FAM_UMMA_SPLITK) return "k_sliced";
    if (fam == FAM_UMMA_PAIR) {
        const long long tiles = q.batch * ((q.M + 255) / 256) * ((q.N + 255) / 256);
        if (plan_tail(q, tiles, kCtaPairs).S > 1) return "output_stationary+k_sliced_tail";
    }
    return "output_stationary";
}
