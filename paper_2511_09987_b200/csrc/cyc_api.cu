// C ABI of the library: argument validation, kernel selection, tensor-map
// construction and launches.  See include/cyc.h for the contract.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <set>
#include <utility>
#include <vector>
#include <type_traits>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/cyc.h"
#include "simt_kernel.cuh"
#include "umma_kernel.cuh"
#include "umma_pair_kernel.cuh"
#include "umma_pair_tall_kernel.cuh"
#include "splitk_reduce_kernel.cuh"
#include "umma_pair_tf32x3_kernel.cuh"
#include "trsm_diag_kernel.cuh"
#include "fa2_kernel.cuh"
#include "scan_kernel.cuh"
#include "chol_diag_kernel.cuh"

namespace cyc {

// raised by a kernel whose bounded wait ran out; one word per device (module scope)
__device__ int g_device_status = 0;

// Fixed workspace of cyc_recurrence_matmul_splitk_static: lives in every device that loads the library, from load
// to exit.  In host code this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) unsigned char g_static_workspace[CYC_STATIC_WORKSPACE_BYTES];

// Self-test of the bounded-wait path: one CTA waits on an mbarrier that nothing ever arrives on, with a
// caller-chosen clock budget, and reports through the same status word and abort flag as the real kernels.
__global__ void bounded_wait_selftest_kernel(long long budget_cycles, int* status) {
    __shared__ uint64_t bar;
    __shared__ volatile int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(&bar, 0)) {
            if (clock64() - t0 > budget_cycles) {
                abort_flag = 1;
                atomicExch(status, 0x7f0);
                break;
            }
        }
    } else {
        // the other role polls the abort flag the way the kernels' roles do, with its own (larger) budget
        const long long t0 = clock64();
        while (!abort_flag && clock64() - t0 < 64 * budget_cycles) {}
    }
    __syncthreads();
}

static std::atomic<long long> g_launches{0};
static thread_local char g_err[512] = "";

static int cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_err, sizeof g_err, "%s: %s", what, cudaGetErrorString(e));
    return CYC_ERR_CUDA;
}
#define CYC_CUDA(call)                                    \
    do {                                                  \
        cudaError_t e_ = (call);                          \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

// Launch with programmatic stream serialisation: the kernel may be scheduled while the kernel before it on the stream
// is still running; each kernel launched this way executes griddepcontrol.wait before it touches global memory.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

static int elem_bytes(int dtype) { return dtype == CYC_F32 ? 4 : (dtype == CYC_BF16_F32 ? 2 : 1); }

struct Problem {
    long long batch, M, N, K;
    int dtype;
    const void *A, *B;
    void* C;
    long long sA, sB, sC;
    unsigned flags;
    long long lda = 0;  // row pitch of A in elements; 0 = dense (K).  Only internal callers set it (sub-blocks of L).
    long long ldb = 0;  // pitch of B in elements (between rows k, or between columns j when stored [N][K]); 0 = dense
};
static long long lda_of(const Problem& q) { return q.lda ? q.lda : q.K; }
static long long ldb_of(const Problem& q) { return q.ldb ? q.ldb : ((q.flags & CYC_FLAG_B_COL_MAJOR) ? q.K : q.N); }

// host-side validation; no CUDA call
static int validate(const Problem& q) {
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

enum Family { FAM_SIMT = 0, FAM_UMMA = 1, FAM_UMMA_3XTF32 = 2, FAM_UMMA_PAIR = 3, FAM_UMMA_TALL = 4, FAM_UMMA_SPLITK = 5 };
constexpr long long kCtaPairs = 74;  // CTA pairs resident on a B200 (148 SMs); used by the tile-shape rule

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
        // strict per-element k order, small or unaligned problems: the general kernel
        if ((q.flags & CYC_FLAG_FIXED_K_ORDER) || !tma_ok(q) || q.M <= 128 || q.N <= 128) return FAM_SIMT;
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

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static int get_encoder(EncodeTiledFn* out) {
    static std::mutex mu;
    static EncodeTiledFn fn = nullptr;
    std::lock_guard<std::mutex> lk(mu);
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qr;
        CYC_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qr));
        if (qr != cudaDriverEntryPointSuccess || !sym) {
            snprintf(g_err, sizeof g_err, "cuTensorMapEncodeTiled not available from the driver");
            return CYC_ERR_CUDA;
        }
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    *out = fn;
    return CYC_OK;
}

// rank-3 map over a [d2][d1][d0] array (d0 contiguous), box [1][box1][box0], 128-byte swizzle
static int make_map_raw(CUtensorMap* m, CUtensorMapDataType dt, int eb, const void* base, long long d0, long long d1, long long d2,
                        long long pitch1_elems, long long pitch2_elems, int box0, int box1,
                        CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    EncodeTiledFn enc;
    int rc = get_encoder(&enc);
    if (rc) return rc;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d0), static_cast<cuuint64_t>(d1), static_cast<cuuint64_t>(d2)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(pitch1_elems) * eb, static_cast<cuuint64_t>(pitch2_elems) * eb};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(box0), static_cast<cuuint32_t>(box1), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_err, sizeof g_err, "cuTensorMapEncodeTiled failed with CUresult %d", static_cast<int>(r));
        return CYC_ERR_CUDA;
    }
    return CYC_OK;
}

// operand map (A or B) in the problem's input type
static int make_map(CUtensorMap* m, int dtype, const void* base, long long d0, long long d1, long long d2, long long pitch1_elems,
                    long long pitch2_elems, int box0, int box1, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    const CUtensorMapDataType dt = dtype == CYC_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                    : (dtype == CYC_BF16_F32 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8);
    return make_map_raw(m, dt, elem_bytes(dtype), base, d0, d1, d2, pitch1_elems, pitch2_elems, box0, box1, swizzle);
}

// result map: C[batch][M][N] of 32-bit words, boxes of 32 rows x 32 columns (128 bytes)
static int make_c_map(CUtensorMap* m, int dtype, void* C, long long M, long long N, long long batch, long long sC) {
    const CUtensorMapDataType dt = dtype == CYC_I8_I32 ? CU_TENSOR_MAP_DATA_TYPE_INT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    return make_map_raw(m, dt, 4, C, N, M, batch, N, sC, 32, 32);
}

struct DeviceInfo {
    int sms = 0, cc_major = 0;
    bool known = false;
};
static int device_info(DeviceInfo* out) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(mu);
    if (dev < 0 || dev >= 64) return CYC_ERR_UNSUPPORTED;
    if (!cache[dev].known) {
        CYC_CUDA(cudaDeviceGetAttribute(&cache[dev].sms, cudaDevAttrMultiProcessorCount, dev));
        CYC_CUDA(cudaDeviceGetAttribute(&cache[dev].cc_major, cudaDevAttrComputeCapabilityMajor, dev));
        cache[dev].known = true;
    }
    *out = cache[dev];
    return CYC_OK;
}

// Once per device: the address of the status word, and the opt-in to more than 48 KB of dynamic shared memory for a
// kernel.  Both are remembered so that the per-call path makes neither runtime call again.
static int status_word(int** out) {
    static std::mutex mu;
    static int* addr[64] = {};
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CYC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(mu);
    if (!addr[dev]) CYC_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&addr[dev]), g_device_status));
    *out = addr[dev];
    return CYC_OK;
}

static int ensure_dynamic_smem(const void* kernel, int bytes) {
    static std::mutex mu;
    static std::set<std::pair<const void*, int>> done;
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(mu);
    if (done.count({kernel, dev})) return CYC_OK;
    CYC_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    done.insert({kernel, dev});
    return CYC_OK;
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

// Scratch of the sliced tail: partial-sum slots for up to one slice per CTA pair and one counter per 32-row strip.
// The counters must be zero when a launch starts and the kernel leaves them zero, so the memory is kept for the
// life of the process -- one scratch per (device, stream), because launches on one stream are ordered and launches on
// different streams are not.  At most kTailScratchMax are created per device; beyond that a launch simply runs the
// plain schedule.  A device-side timeout may leave counters non-zero: cyc_last_device_status marks every scratch
// dirty and the next use clears it on its stream.
struct TailScratch {
    int dev = -1;
    cudaStream_t stream = nullptr;
    uint8_t* ws = nullptr;
    int* counters = nullptr;
    bool dirty = false;
};
constexpr int kTailScratchMax = 8;
constexpr size_t kTailCounterBytes = static_cast<size_t>(kCtaPairs) * 8 * sizeof(int);
static std::mutex g_tail_mu;
static TailScratch g_tail_scratch[64];
static int g_tail_scratch_count = 0;

static void tail_scratch_mark_dirty() {
    std::lock_guard<std::mutex> lk(g_tail_mu);
    for (int i = 0; i < g_tail_scratch_count; ++i) g_tail_scratch[i].dirty = true;
}

// returns CYC_OK with *out = nullptr when no scratch can be had (the caller then runs the plain schedule)
static int tail_scratch_for(cudaStream_t st, TailScratch** out) {
    *out = nullptr;
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); return CYC_OK; }
    std::lock_guard<std::mutex> lk(g_tail_mu);
    TailScratch* found = nullptr;
    int on_dev = 0;
    for (int i = 0; i < g_tail_scratch_count; ++i) {
        if (g_tail_scratch[i].dev != dev) continue;
        ++on_dev;
        if (g_tail_scratch[i].stream == st) found = &g_tail_scratch[i];
    }
    if (!found) {
        // creating one allocates and clears memory: not while the stream is being captured into a graph
        if (cap != cudaStreamCaptureStatusNone || on_dev >= kTailScratchMax || g_tail_scratch_count >= 64) return CYC_OK;
        void* mem = nullptr;
        const size_t bytes = static_cast<size_t>(kCtaPairs) * PAIR_TILE_BYTES + kTailCounterBytes;
        if (cudaMalloc(&mem, bytes) != cudaSuccess) { cudaGetLastError(); return CYC_OK; }
        if (cudaMemset(static_cast<uint8_t*>(mem) + static_cast<size_t>(kCtaPairs) * PAIR_TILE_BYTES, 0, kTailCounterBytes) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(mem);
            return CYC_OK;
        }
        found = &g_tail_scratch[g_tail_scratch_count++];
        found->dev = dev;
        found->stream = st;
        found->ws = static_cast<uint8_t*>(mem);
        found->counters = reinterpret_cast<int*>(found->ws + static_cast<size_t>(kCtaPairs) * PAIR_TILE_BYTES);
        found->dirty = false;
    }
    if (found->dirty) {
        if (cap != cudaStreamCaptureStatusNone) return CYC_OK;
        CYC_CUDA(cudaMemsetAsync(found->counters, 0, kTailCounterBytes, st));
        found->dirty = false;
    }
    *out = found;
    return CYC_OK;
}

// ------------------------------------------------------------------ two-SM tensor-core launch
// `ws` != nullptr: split-K -- the kernel writes plan.S planes of partial sums per problem into ws
template <int KIND, bool B_MN>
static int launch_pair_cfg(const Problem& q, cudaStream_t st, int sms, void* ws = nullptr, SplitPlan plan = SplitPlan()) {
    constexpr int STAGES = 6;
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
            TailScratch* sc = nullptr;
            if (int rc_ = tail_scratch_for(st, &sc)) return rc_;
            if (sc) {
                p.tail_S = tp.S; p.tail_tiles = tp.tiles; p.tail_kb = tp.kb;
                p.tail_ws = sc->ws; p.tail_counters = sc->counters;
            }
        }
    }
    CYC_CUDA(launch_pdl(kern, static_cast<unsigned>(2 * pairs), UMMA_THREADS, SMEM, st, tmA, tmB, tmC, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}

// ------------------------------------------------------------------ split-K
// Workspace for the partial sums: stream-ordered allocations from a pool the library owns (one per device),
// so that repeated calls reuse the same memory without a synchronising cudaMalloc.
static int workspace_pool(cudaMemPool_t* out, bool create = true) {
    static std::mutex mu;
    static cudaMemPool_t pools[64] = {};
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CYC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(mu);
    if (!pools[dev] && create) {
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        CYC_CUDA(cudaMemPoolCreate(&pools[dev], &props));
        unsigned long long keep = ~0ull;  // keep freed blocks for the next call instead of returning them to the driver
        CYC_CUDA(cudaMemPoolSetAttribute(pools[dev], cudaMemPoolAttrReleaseThreshold, &keep));
    }
    *out = pools[dev];
    return CYC_OK;
}

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

static int launch_tf32x3(const Problem& q, cudaStream_t st) {
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    if (di.cc_major != 10) {
        snprintf(g_err, sizeof g_err, "tensor-core kernels need an sm_100 device");
        return CYC_ERR_UNSUPPORTED;
    }
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
static int route(const Problem& q, cudaStream_t st) {
    switch (choose(q)) {
        case FAM_UMMA:
        case FAM_UMMA_PAIR:
        case FAM_UMMA_TALL:
        case FAM_UMMA_SPLITK:
            return q.dtype == CYC_BF16_F32 ? launch_umma<KIND_BF16>(q, st) : launch_umma<KIND_I8>(q, st);
        case FAM_UMMA_3XTF32:
            return launch_tf32x3(q, st);
        default:
            if (q.dtype == CYC_F32) return launch_simt<float, float>(q, st);
            if (q.dtype == CYC_BF16_F32) return launch_simt<__nv_bfloat16, float>(q, st);
            return launch_simt<int8_t, int>(q, st);
    }
}

static int dispatch(const Problem& q, cudaStream_t st) {
    int rc = validate(q);
    if (rc) return rc;
    return route(q, st);
}

// ------------------------------------------------------------------ block lower-triangular solve
// X_i = TRSM(L_ii, B_i - sum_{j<i} GEMM(L_ij, X_j)).  The block rows are split recursively: solve the upper part,
// form the partial sums of the lower part's rows over the solved block columns with one recurrence-matmul launch
// (triangular space; written to the plane of this recursion level), solve the lower part.  A diagonal tile subtracts
// the planes of every level that covered its rows (its end-of-row accumulator) and solves (diagonal space).
struct TrsmPlan {
    long long n, m, T;
    const float* L;
    const float* B;
    float* X;
    float* W;
    long long plane;
    unsigned flags;
    cudaStream_t st;
};

static int trsm_diag(const TrsmPlan& t, long long b, unsigned mask) {
    TrsmDiagParams p;
    p.L = t.L;
    p.B = t.B + b * t.T * t.m; p.X = t.X + b * t.T * t.m; p.W = t.W ? t.W + b * t.T * t.m : nullptr;  // first row of the tile
    p.plane = t.plane;
    p.b_r = p.x_r = p.w_r = t.m;
    p.b_c = p.x_c = p.w_c = 1;
    p.n = static_cast<int>(t.n); p.m = static_cast<int>(t.m);
    p.r0 = static_cast<int>(b * t.T);
    p.rows = static_cast<int>(t.n - b * t.T < t.T ? t.n - b * t.T : t.T);
    p.mask = mask;
    const long long blocks = (t.m + TRSM_CW - 1) / TRSM_CW;
    CYC_CUDA(launch_pdl(trsm_diag_kernel, static_cast<unsigned>(blocks), TRSM_THREADS, TRSM_SMEM_BYTES, t.st, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}

static int trsm_range(const TrsmPlan& t, long long b0, long long b1, unsigned mask, int level) {
    if (b1 - b0 == 1) return trsm_diag(t, b0, mask);
    const long long mid = b0 + (b1 - b0 + 1) / 2;
    int rc = trsm_range(t, b0, mid, mask, level + 1);
    if (rc) return rc;
    const long long r0 = mid * t.T, r1 = b1 * t.T < t.n ? b1 * t.T : t.n, k0 = b0 * t.T, k1 = mid * t.T;
    Problem q{1, r1 - r0, t.m, k1 - k0, CYC_F32, t.L + r0 * t.n + k0, t.X + k0 * t.m, t.W + level * t.plane + r0 * t.m,
              (r1 - r0) * t.n, (k1 - k0) * t.m, (r1 - r0) * t.m, t.flags & CYC_FLAG_FIXED_K_ORDER, t.n};
    rc = route(q, t.st);
    if (rc) return rc;
    return trsm_range(t, mid, b1, mask | (1u << level), level + 1);
}

// ------------------------------------------------------------------ FlashAttention-2 recurrence
template <int D>
static int launch_fa2(long long batch, long long N, long long M, const void* Q, const void* K, const void* V, float* O, cudaStream_t st) {
    CUtensorMap tmQ, tmK, tmV;
    int rc = make_map(&tmQ, CYC_BF16_F32, Q, D, N, batch, D, N * D, 64, FA2_BM);
    if (rc) return rc;
    rc = make_map(&tmK, CYC_BF16_F32, K, D, M, batch, D, M * D, 64, FA2_BN);
    if (rc) return rc;
    rc = make_map(&tmV, CYC_BF16_F32, V, D, M, batch, D, M * D, 64, FA2_BN);
    if (rc) return rc;
    Fa2Params p;
    p.O = O;
    p.N = static_cast<int>(N); p.M = static_cast<int>(M);
    p.tiles_q = static_cast<int>((N + FA2_ROWS - 1) / FA2_ROWS);
    p.scale_log2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(D)));
    if (int rc_ = status_word(&p.status)) return rc_;
    auto kern = fa2_kernel<D>;
    {
        // the kernel redistributes the registers it was launched with among its warps and counts on 128 per thread
        static std::atomic<int> checked{0};
        if (!checked.load()) {
            cudaFuncAttributes fa;
            CYC_CUDA(cudaFuncGetAttributes(&fa, kern));
            if (fa.numRegs < FA2_REGS_LAUNCH) {
                snprintf(g_err, sizeof g_err, "flash attention kernel compiled to %d registers per thread, %d expected", fa.numRegs, FA2_REGS_LAUNCH);
                return CYC_ERR_CUDA;
            }
            checked.store(1);
        }
    }
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), Fa2Smem<D>::TOTAL)) return rc_;
    CYC_CUDA(launch_pdl(kern, static_cast<unsigned>(batch * p.tiles_q), FA2_THREADS, Fa2Smem<D>::TOTAL, st, tmQ, tmK, tmV, p));
    g_launches.fetch_add(1);
    return CYC_OK;
}

}  // namespace cyc

// ====================================================================== C ABI
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

extern "C" int cyc_pool_reserved_bytes(int64_t* out) {
    if (!out) return CYC_ERR_INVALID_ARG;
    *out = 0;
    cudaMemPool_t pool = nullptr;
    int rc = workspace_pool(&pool, /*create=*/false);
    if (rc) return rc;
    if (pool) {
        unsigned long long bytes = 0;
        CYC_CUDA(cudaMemPoolGetAttribute(pool, cudaMemPoolAttrReservedMemCurrent, &bytes));
        *out = static_cast<int64_t>(bytes);
    }
    return CYC_OK;
}

extern "C" int cyc_block_trsm(int64_t n, int64_t m, int64_t tile, int dtype, const void* L, const void* B, void* X,
                              void* stream, unsigned flags) {
    if (n <= 0 || m <= 0 || tile < 0 || tile > TRSM_T_MAX || !L || !B || !X) return CYC_ERR_INVALID_ARG;
    if (dtype != CYC_F32 && dtype != CYC_BF16_F32 && dtype != CYC_I8_I32) return CYC_ERR_INVALID_ARG;
    if (flags & ~CYC_FLAG_FIXED_K_ORDER) return CYC_ERR_INVALID_ARG;
    const uintptr_t l0 = reinterpret_cast<uintptr_t>(L), b0 = reinterpret_cast<uintptr_t>(B), x0 = reinterpret_cast<uintptr_t>(X);
    if ((l0 | b0 | x0) % 4) return CYC_ERR_INVALID_ARG;
    if (n > 0x7fffffffll || m > 0x7fffffffll) return CYC_ERR_UNSUPPORTED;
    if (dtype != CYC_F32) return CYC_ERR_UNSUPPORTED;  // the solve is defined for fp32 only
    const uintptr_t lbytes = static_cast<uintptr_t>(n) * n * 4, xbytes = static_cast<uintptr_t>(n) * m * 4;
    if (x0 < l0 + lbytes && l0 < x0 + xbytes) return CYC_ERR_INVALID_ARG;                // X over L
    if (x0 != b0 && x0 < b0 + xbytes && b0 < x0 + xbytes) return CYC_ERR_INVALID_ARG;    // X over B, other than in place
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    TrsmPlan t;
    t.n = n; t.m = m; t.T = tile ? tile : TRSM_T_MAX;
    t.L = static_cast<const float*>(L); t.B = static_cast<const float*>(B); t.X = static_cast<float*>(X);
    t.W = nullptr; t.plane = n * m; t.flags = flags; t.st = st;
    const long long nb = (n + t.T - 1) / t.T;
    int levels = 0;
    while ((1ll << levels) < nb) ++levels;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(trsm_diag_kernel), TRSM_SMEM_BYTES)) return rc_;
    if (levels) {
        cudaMemPool_t pool;
        int rc = workspace_pool(&pool);
        if (rc) return rc;
        void* ws = nullptr;
        CYC_CUDA(cudaMallocFromPoolAsync(&ws, static_cast<size_t>(levels) * t.plane * sizeof(float), pool, st));
        t.W = static_cast<float*>(ws);
    }
    int rc = trsm_range(t, 0, nb, 0u, 0);
    if (t.W) {
        cudaError_t e = cudaFreeAsync(t.W, st);
        if (e != cudaSuccess && rc == CYC_OK) rc = cuda_fail(e, "cudaFreeAsync");
    }
    return rc;
}

extern "C" int cyc_flash_attention(int64_t batch, int64_t N, int64_t M, int64_t d, int dtype, const void* Q, const void* K,
                                   const void* V, void* O, void* stream, unsigned flags) {
    if (batch <= 0 || N <= 0 || M <= 0 || d <= 0 || !Q || !K || !V || !O || flags != 0) return CYC_ERR_INVALID_ARG;
    if (dtype != CYC_F32 && dtype != CYC_BF16_F32 && dtype != CYC_I8_I32) return CYC_ERR_INVALID_ARG;
    const uintptr_t q0 = reinterpret_cast<uintptr_t>(Q), k0 = reinterpret_cast<uintptr_t>(K), v0 = reinterpret_cast<uintptr_t>(V),
                    o0 = reinterpret_cast<uintptr_t>(O);
    if ((q0 | k0 | v0) % 2 || o0 % 4) return CYC_ERR_INVALID_ARG;
    const uintptr_t obytes = static_cast<uintptr_t>(batch) * N * d * 4, qbytes = static_cast<uintptr_t>(batch) * N * d * 2,
                    kbytes = static_cast<uintptr_t>(batch) * M * d * 2;
    if ((o0 < q0 + qbytes && q0 < o0 + obytes) || (o0 < k0 + kbytes && k0 < o0 + obytes) || (o0 < v0 + kbytes && v0 < o0 + obytes))
        return CYC_ERR_INVALID_ARG;  // O over an input
    if (dtype != CYC_BF16_F32 || (d != 64 && d != 128)) {
        snprintf(g_err, sizeof g_err, "flash attention: bf16 inputs with head dimension 64 or 128 only");
        return CYC_ERR_UNSUPPORTED;
    }
    if ((q0 | k0 | v0 | o0) % 16) {
        snprintf(g_err, sizeof g_err, "flash attention: Q, K, V and O must be 16-byte aligned");
        return CYC_ERR_UNSUPPORTED;
    }
    const long long tiles_q = (N + FA2_ROWS - 1) / FA2_ROWS;
    if (N > 0x7fffffffll || M > 0x7fffffffll || batch * tiles_q > 0x7fffffffll) return CYC_ERR_UNSUPPORTED;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    if (di.cc_major != 10) {
        snprintf(g_err, sizeof g_err, "tensor-core kernels need an sm_100 device");
        return CYC_ERR_UNSUPPORTED;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return d == 64 ? launch_fa2<64>(batch, N, M, Q, K, V, static_cast<float*>(O), st)
                   : launch_fa2<128>(batch, N, M, Q, K, V, static_cast<float*>(O), st);
}

// tile of SUBS * 4096 elements: 16384 for long rows (the running value of one chain advances by at most 32 tiles per
// descriptor round trip), 8192 when a row has at most 32 such tiles (its look-back never leaves one window; half the
// shared memory per CTA, twice the CTAs per SM)
static int scan_subs(long long n) { return (n + SCAN_SUBS_SHORT * SCAN_SUB - 1) / (SCAN_SUBS_SHORT * SCAN_SUB) <= SCAN_WINDOW ? SCAN_SUBS_SHORT : SCAN_SUBS; }

template <typename T, int SUBS>
static int launch_scan(long long rows, long long n, const void* A, long long sA, void* P, long long sP, cudaStream_t st) {
    constexpr long long TILE = static_cast<long long>(SUBS) * SCAN_SUB;
    ScanParams<T> p;
    p.A = static_cast<const T*>(A);
    p.P = static_cast<T*>(P);
    p.n = n; p.strideA = sA; p.strideP = sP;
    p.tiles_per_row = (n + TILE - 1) / TILE;
    const long long tiles = rows * p.tiles_per_row;
    p.total_tiles = tiles;
    p.vec_ok = (reinterpret_cast<uintptr_t>(A) % 16 == 0 && reinterpret_cast<uintptr_t>(P) % 16 == 0 && (rows == 1 || (sA % 4 == 0 && sP % 4 == 0)))
                   ? 1 : 0;
    if (int rc_ = status_word(&p.status)) return rc_;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(scan_kernel<T, SUBS>), static_cast<int>(TILE * sizeof(T)) + 128)) return rc_;
    cudaMemPool_t pool;
    int rc = workspace_pool(&pool);
    if (rc) return rc;
    void* ws = nullptr;
    const size_t bytes = sizeof(ScanHeader) + static_cast<size_t>(tiles) * sizeof(unsigned long long);
    CYC_CUDA(cudaMallocFromPoolAsync(&ws, bytes, pool, st));
    p.header = static_cast<ScanHeader*>(ws);
    p.desc = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(ws) + sizeof(ScanHeader));
    cudaError_t e = cudaMemsetAsync(ws, 0, bytes, st);  // counter, abort flag and every descriptor start at zero
    if (e == cudaSuccess) {
        // short rows need only their own quarters of the staging buffer: more CTAs fit an SM
        const int quarters = static_cast<int>(std::min<long long>(SUBS, (n + SCAN_SUB - 1) / SCAN_SUB));
        scan_kernel<T, SUBS><<<static_cast<unsigned>(tiles), SCAN_THREADS, quarters * SCAN_SUB * sizeof(T) + 128, st>>>(p);
        e = cudaGetLastError();
        if (e == cudaSuccess) g_launches.fetch_add(1);
    }
    const cudaError_t e2 = cudaFreeAsync(ws, st);
    if (e != cudaSuccess) return cuda_fail(e, "scan_kernel");
    if (e2 != cudaSuccess) return cuda_fail(e2, "cudaFreeAsync");
    return CYC_OK;
}

extern "C" int cyc_prefix_sum(int64_t rows, int64_t n, int dtype, const void* A, int64_t strideA, void* P, int64_t strideP,
                              void* stream, unsigned flags) {
    if (rows <= 0 || n <= 0 || !A || !P || flags != 0 || strideA < 0 || strideP < 0) return CYC_ERR_INVALID_ARG;
    if (dtype != CYC_F32 && dtype != CYC_BF16_F32 && dtype != CYC_I8_I32 && dtype != CYC_I32) return CYC_ERR_INVALID_ARG;
    const long long sA = strideA ? strideA : n, sP = strideP ? strideP : n;
    if (sA < n || sP < n) return CYC_ERR_INVALID_ARG;
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(A), p0 = reinterpret_cast<uintptr_t>(P);
    if ((a0 | p0) % 4) return CYC_ERR_INVALID_ARG;
    if (rows > (1ll << 40) || n > (1ll << 40)) return CYC_ERR_UNSUPPORTED;
    const uintptr_t abytes = (static_cast<uintptr_t>(rows - 1) * sA + n) * 4, pbytes = (static_cast<uintptr_t>(rows - 1) * sP + n) * 4;
    const bool in_place = a0 == p0 && sA == sP;
    if (!in_place && a0 < p0 + pbytes && p0 < a0 + abytes) return CYC_ERR_INVALID_ARG;
    if (dtype != CYC_F32 && dtype != CYC_I32) {
        snprintf(g_err, sizeof g_err, "prefix sum: fp32 or int32 only");
        return CYC_ERR_UNSUPPORTED;
    }
    const int subs = scan_subs(n);
    const long long tiles_per_row = (n + subs * SCAN_SUB - 1) / (subs * SCAN_SUB);
    if (tiles_per_row > 0x7fffffffll / rows) return CYC_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (subs == SCAN_SUBS_SHORT)
        return dtype == CYC_F32 ? launch_scan<float, SCAN_SUBS_SHORT>(rows, n, A, sA, P, sP, st) : launch_scan<int, SCAN_SUBS_SHORT>(rows, n, A, sA, P, sP, st);
    return dtype == CYC_F32 ? launch_scan<float, SCAN_SUBS>(rows, n, A, sA, P, sP, st) : launch_scan<int, SCAN_SUBS>(rows, n, A, sA, P, sP, st);
}

// ------------------------------------------------------------------ tiled Cholesky
// Panel j (columns c0 .. c1 of L), left-looking.  The sums over the panels already factored,
//     W = L[c0:n, 0:c0] L[c0:c1, 0:c0]^T ,
// are recurrence-matmul launches (k cut into slices that run as the batch dimension, then summed in increasing k); the
// diagonal tile A_jj - W is factored by chol_diag_kernel (one SM); the tiles below are the rows of
// X L_jj^T = A[c1:n, c0:c1] - W, solved by trsm_diag_kernel with the right-hand sides addressed as rows.
// The paper describes the recurrence as a wavefront that widens down the column; on a GPU the narrow end of that
// wavefront is the one-SM diagonal tile, so the work is laid on two streams:
//   the caller's stream carries the chain  sum of the diagonal tile -> diagonal tile (j) -> solve of the block row just
//   below it -> sum of the next diagonal tile -> diagonal tile (j+1) ...,
//   a helper stream carries the bulk: solve of the remaining rows of panel j, then the sums of everything below the
//   next diagonal tile -- which run while diagonal tile j+1 is being factored.
// Events order the two; every launch below names the data it needs.
struct CholAux {
    bool ready = false;
    cudaStream_t side = nullptr;
    std::vector<cudaEvent_t> events;
    std::mutex mu;  // one factorisation at a time per device uses the helper stream
};
static int chol_aux(CholAux** out, size_t events) {
    static std::mutex mu;
    static CholAux aux[64];
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CYC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(mu);
    CholAux& a = aux[dev];
    if (!a.ready) {
        CYC_CUDA(cudaStreamCreateWithFlags(&a.side, cudaStreamNonBlocking));
        a.ready = true;
    }
    while (a.events.size() < events) {
        cudaEvent_t e = nullptr;
        CYC_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        a.events.push_back(e);
    }
    *out = &a;
    return CYC_OK;
}

// W (plane 0) = L[r0:r1, 0:c0] L[c0:c0+w, 0:c0]^T on stream `s`; planes of `pstride` floats starting at W.  The k range
// is cut into up to CHOL_MAX_SLICES equal slices (one batched launch: few 256-row tiles, and the slices give every CTA
// pair work) plus one launch for the remainder; the slices' partial sums are then added in increasing k into plane 0.
constexpr int CHOL_MAX_SLICES = 8;        // sums below a diagonal tile: several 256-row tiles share the CTA pairs
constexpr int CHOL_MAX_SLICES_DIAG = 64;  // sum of a diagonal tile: one tile, so every panel of k can be a slice of its own
static int chol_product(cudaStream_t s, float* Lf, long long n, long long T, long long c0, long long w, long long r0, long long r1, float* W,
                        long long pstride, unsigned flags, int max_slices) {
    const long long rows = r1 - r0;
    const long long kblocks = c0 / T, tiles_m = (rows + 255) / 256;
    const long long smax = std::min<long long>({static_cast<long long>(max_slices), kblocks, std::max<long long>(1, kCtaPairs / tiles_m)});
    // slices of ceil(kblocks / smax) panels, so that the remainder (one more launch) is shorter than a slice
    const long long per = (kblocks + smax - 1) / smax, S = kblocks / per;
    const long long kc = per * T, rem = c0 - S * kc;
    const unsigned gflags = (flags & CYC_FLAG_FIXED_K_ORDER) | CYC_FLAG_B_COL_MAJOR;
    Problem q{S, rows, w, kc, CYC_F32, Lf + r0 * n, Lf + c0 * n, W, kc, kc, pstride, gflags, n, n};
    int rc = route(q, s);
    if (rc) return rc;
    int planes = static_cast<int>(S);
    if (rem > 0) {
        Problem r{1, rows, w, rem, CYC_F32, Lf + r0 * n + S * kc, Lf + c0 * n + S * kc, W + S * pstride, rows * n, w * n, pstride, gflags, n, n};
        rc = route(r, s);
        if (rc) return rc;
        ++planes;
    }
    if (planes > 1) {
        DeviceInfo di;
        rc = device_info(&di);
        if (rc) return rc;
        const long long work = pstride / 4;
        const long long blocks = std::min<long long>((work + 127) / 128, 16ll * di.sms);
        cudaError_t e = launch_pdl(splitk_reduce_kernel<float>, static_cast<unsigned>(blocks), 128, 0, s, static_cast<const float*>(W), W, pstride,
                                   pstride, planes, 1ll, 1);
        if (e != cudaSuccess) return cuda_fail(e, "splitk_reduce_kernel");
        g_launches.fetch_add(1);
    }
    return CYC_OK;
}

extern "C" int cyc_cholesky(int64_t n, int64_t tile, int dtype, const void* A, void* L, void* stream, unsigned flags) {
    if (n <= 0 || tile < 0 || tile > CHOL_T_MAX || !A || !L) return CYC_ERR_INVALID_ARG;
    if (dtype != CYC_F32 && dtype != CYC_BF16_F32 && dtype != CYC_I8_I32) return CYC_ERR_INVALID_ARG;
    if (flags & ~CYC_FLAG_FIXED_K_ORDER) return CYC_ERR_INVALID_ARG;
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(A), l0 = reinterpret_cast<uintptr_t>(L);
    if ((a0 | l0) % 4) return CYC_ERR_INVALID_ARG;
    if (n > 0x7fffffffll) return CYC_ERR_UNSUPPORTED;
    if (dtype != CYC_F32) return CYC_ERR_UNSUPPORTED;  // the factorisation is defined for fp32 only
    const uintptr_t bytes = static_cast<uintptr_t>(n) * n * 4;
    if (a0 != l0 && a0 < l0 + bytes && l0 < a0 + bytes) return CYC_ERR_INVALID_ARG;  // overlap other than in place
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float* Af = static_cast<const float*>(A);
    float* Lf = static_cast<float*>(L);
    const long long T = tile ? tile : CHOL_T_MAX;
    const bool in_place = a0 == l0;
    const long long panels = (n + T - 1) / T;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(chol_diag_kernel), CHOL_SMEM_BYTES)) return rc_;
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(trsm_diag_kernel), TRSM_SMEM_BYTES)) return rc_;
    CholAux* aux = nullptr;
    if (int rc_ = chol_aux(&aux, static_cast<size_t>(3 * panels + 2))) return rc_;
    std::lock_guard<std::mutex> aux_lock(aux->mu);
    cudaStream_t side = aux->side;
    auto ev = [&](long long j, int which) { return aux->events[static_cast<size_t>(3 * j + which)]; };  // 0: D(j), 1: near solve (j), 2: sums below (j)
    cudaEvent_t ev_fork = aux->events[static_cast<size_t>(3 * panels)], ev_join = aux->events[static_cast<size_t>(3 * panels + 1)];

    // workspace: planes of the diagonal tile's sums and planes of the sums below it (the two streams never share a plane)
    const long long pd = (T * T + 3) / 4 * 4, pb = ((n - T) * T + 3) / 4 * 4;
    float* Wd = nullptr;
    float* Wb = nullptr;
    if (n > T) {
        cudaMemPool_t pool;
        int rc = workspace_pool(&pool);
        if (rc) return rc;
        void* ws = nullptr;
        CYC_CUDA(cudaMallocFromPoolAsync(&ws, (static_cast<size_t>(CHOL_MAX_SLICES_DIAG + 1) * pd + static_cast<size_t>(CHOL_MAX_SLICES + 1) * pb) * sizeof(float), pool, st));
        Wd = static_cast<float*>(ws);
        Wb = Wd + (CHOL_MAX_SLICES_DIAG + 1) * pd;
    }
    int rc = CYC_OK;
    auto ok = [&](cudaError_t e, const char* what) {
        if (e != cudaSuccess && rc == CYC_OK) rc = cuda_fail(e, what);
        return rc == CYC_OK;
    };
    // rows [r0, r1) of panel (c0, w): X L_jj^T = A - W, the right-hand sides addressed as rows
    auto solve_rows = [&](cudaStream_t s, long long c0, long long w, long long c1, long long r0, long long r1, bool have_w, long long pstride) {
        TrsmDiagParams p;
        p.L = Lf;
        p.B = Af + r0 * n + c0; p.X = Lf + r0 * n + c0; p.W = have_w ? Wb + (r0 - c1) * w : nullptr;
        p.plane = pstride;
        p.b_r = 1; p.b_c = n; p.x_r = 1; p.x_c = n; p.w_r = 1; p.w_c = w;
        p.n = static_cast<int>(n); p.m = static_cast<int>(r1 - r0);
        p.r0 = static_cast<int>(c0); p.rows = static_cast<int>(w);
        p.mask = have_w ? 1u : 0u;
        if (ok(launch_pdl(trsm_diag_kernel, static_cast<unsigned>((r1 - r0 + TRSM_CW - 1) / TRSM_CW), TRSM_THREADS, TRSM_SMEM_BYTES, s, p), "trsm_diag_kernel"))
            g_launches.fetch_add(1);
    };

    ok(cudaEventRecord(ev_fork, st), "cudaEventRecord");
    ok(cudaStreamWaitEvent(side, ev_fork, 0), "cudaStreamWaitEvent");
    for (long long j = 0; j < panels && rc == CYC_OK; ++j) {
        const long long c0 = j * T, c1 = std::min<long long>(n, c0 + T), w = c1 - c0, c2 = std::min<long long>(n, c1 + T);
        // ---- caller's stream: the sum of the diagonal tile (needs row block j of every earlier panel: the near solve of
        // ---- panel j-1 is on this stream, the far solves of older panels were waited for with the sums below panel j-1)
        if (c0 > 0) {
            rc = chol_product(st, Lf, n, T, c0, w, c0, c1, Wd, pd, flags, CHOL_MAX_SLICES_DIAG);
            if (rc) break;
        }
        CholDiagParams d;
        d.A = Af + c0 * n + c0; d.W = Wd; d.L = Lf + c0 * n + c0;
        d.plane = pd; d.planes = c0 > 0 ? 1 : 0;
        d.lda = n; d.ldw = w; d.ldl = n;
        d.rows = static_cast<int>(w);
        d.zero_upper = in_place ? 0 : 1;
        if (!ok(launch_pdl(chol_diag_kernel, 1u, CHOL_THREADS, CHOL_SMEM_BYTES, st, d), "chol_diag_kernel")) break;
        g_launches.fetch_add(1);
        if (c1 >= n) break;
        ok(cudaEventRecord(ev(j, 0), st), "cudaEventRecord");
        const long long pstride_b = ((n - c1) * w + 3) / 4 * 4;
        // ---- caller's stream: the block row just below the diagonal tile (needs its sums, formed on the helper stream)
        if (c0 > 0) ok(cudaStreamWaitEvent(st, ev(j, 2), 0), "cudaStreamWaitEvent");
        if (rc == CYC_OK) solve_rows(st, c0, w, c1, c1, c2, c0 > 0, pstride_b);
        ok(cudaEventRecord(ev(j, 1), st), "cudaEventRecord");
        // ---- helper stream: the remaining rows of the panel (need the diagonal tile; their sums are on this stream)
        ok(cudaStreamWaitEvent(side, ev(j, 0), 0), "cudaStreamWaitEvent");
        if (c2 < n && rc == CYC_OK) solve_rows(side, c0, w, c1, c2, n, c0 > 0, pstride_b);
        if (!in_place)  // zeros above the diagonal: the block row to the right of the diagonal tile
            ok(cudaMemset2DAsync(Lf + c0 * n + c1, static_cast<size_t>(n) * 4, 0, static_cast<size_t>(n - c1) * 4, static_cast<size_t>(w), side), "cudaMemset2DAsync");
        // ---- helper stream: the sums below the NEXT diagonal tile (need block row j+1 of this panel: the near solve)
        if (c2 < n && rc == CYC_OK) {
            const long long w1 = c2 - c1, pstride_n = ((n - c2) * w1 + 3) / 4 * 4;
            ok(cudaStreamWaitEvent(side, ev(j, 1), 0), "cudaStreamWaitEvent");
            if (rc == CYC_OK) rc = chol_product(side, Lf, n, T, c1, w1, c2, n, Wb, pstride_n, flags, CHOL_MAX_SLICES);
            ok(cudaEventRecord(ev(j + 1, 2), side), "cudaEventRecord");
        }
    }
    // the caller's stream continues only after the helper stream has finished
    if (cudaEventRecord(ev_join, side) == cudaSuccess) cudaStreamWaitEvent(st, ev_join, 0);
    else cudaStreamSynchronize(side);
    if (Wd) {
        cudaError_t e = cudaFreeAsync(Wd, st);
        if (e != cudaSuccess && rc == CYC_OK) rc = cuda_fail(e, "cudaFreeAsync");
    }
    return rc;
}

extern "C" int cyc_selftest_bounded_wait(void* stream, int64_t budget_cycles) {
    if (budget_cycles < 1 || budget_cycles > (1ll << 24)) return CYC_ERR_INVALID_ARG;  // at most ~10 ms
    int* status = nullptr;
    CYC_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&status), g_device_status));
    bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(budget_cycles, status);
    CYC_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    return CYC_OK;
}

extern "C" int cyc_last_device_status(void* stream, int* out) {
    CYC_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    int word = 0;
    CYC_CUDA(cudaMemcpyFromSymbol(&word, g_device_status, sizeof word));
    if (word != 0) {
        const int zero = 0;
        tail_scratch_mark_dirty();  // a kernel that gave up may have left strip counters of the sliced tail non-zero
        CYC_CUDA(cudaMemcpyToSymbol(g_device_status, &zero, sizeof zero));
        snprintf(g_err, sizeof g_err, "device wait ran out (code 0x%x)", word);
    }
    if (out) *out = word != 0 ? CYC_ERR_TIMEOUT : CYC_OK;
    return CYC_OK;
}

extern "C" const char* cyc_kernel_for(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B,
                                      const void* C, unsigned flags) {
    if (batch <= 0 || M <= 0 || N <= 0 || K <= 0) return nullptr;
    Problem q{batch, M, N, K, dtype, A, B, const_cast<void*>(C), M * K, K * N, M * N, flags};
    if (validate(q) != CYC_OK) return nullptr;
    switch (choose(q)) {
        case FAM_UMMA: return "tcgen05";
        case FAM_UMMA_PAIR: return "tcgen05_pair";
        case FAM_UMMA_TALL: return "tcgen05_pair_tall";
        case FAM_UMMA_SPLITK: return "tcgen05_pair_splitk";
        case FAM_UMMA_3XTF32: return "tcgen05_3xtf32";
        default: return "simt";
    }
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

extern "C" int64_t cyc_launch_count(void) { return g_launches.load(); }
extern "C" const char* cyc_last_cuda_error(void) { return g_err; }

extern "C" const char* cyc_status_string(int s) {
    switch (s) {
        case CYC_OK: return "ok";
        case CYC_ERR_INVALID_ARG: return "invalid argument";
        case CYC_ERR_UNSUPPORTED: return "unsupported";
        case CYC_ERR_CUDA: return "CUDA error";
        case CYC_ERR_TIMEOUT: return "device wait timed out";
        default: return "unknown status";
    }
}
extern "C" int cyc_version(void) { return 100; }
