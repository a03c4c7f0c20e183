// The prefix-sum recurrence: cyc_prefix_sum.  See include/cyc.h.
#include "api_internal.h"
#include "scan_kernel.cuh"

using namespace cyc;

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
