// The recurrences over two coupled iteration spaces: the block lower-triangular solve (cyc_block_trsm) and the tiled
// Cholesky factorisation (cyc_cholesky).  Both lay their tile products on the matrix-multiply recurrence (route) and
// share the diagonal-space kernel.  See include/cyc.h.
#include "api_internal.h"
#include "splitk_reduce_kernel.cuh"
#include "trsm_diag_kernel.cuh"
#include "chol_diag_kernel.cuh"

namespace cyc {

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

// One launch of the diagonal-space kernel over `columns` right-hand-side columns: 32 columns per CTA, or 8 when 32 would
// occupy at most a quarter of the SMs (the CTA's chain of dependent steps is as long either way, its arithmetic is not).
static cudaError_t launch_trsm_diag(const TrsmDiagParams& p, long long columns, cudaStream_t st) {
    DeviceInfo di;
    const bool narrow = device_info(&di) == CYC_OK && 4 * ((columns + TRSM_CW - 1) / TRSM_CW) <= di.sms;
    if (narrow)
        return launch_pdl(trsm_diag_kernel<TRSM_CW_NARROW>, static_cast<unsigned>((columns + TRSM_CW_NARROW - 1) / TRSM_CW_NARROW), TRSM_THREADS,
                          TRSM_SMEM_BYTES, st, p);
    return launch_pdl(trsm_diag_kernel<TRSM_CW>, static_cast<unsigned>((columns + TRSM_CW - 1) / TRSM_CW), TRSM_THREADS, TRSM_SMEM_BYTES, st, p);
}
static int trsm_diag_smem() {
    if (int rc_ = ensure_dynamic_smem(reinterpret_cast<const void*>(trsm_diag_kernel<TRSM_CW>), TRSM_SMEM_BYTES)) return rc_;
    return ensure_dynamic_smem(reinterpret_cast<const void*>(trsm_diag_kernel<TRSM_CW_NARROW>), TRSM_SMEM_BYTES);
}

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
    CYC_CUDA(launch_trsm_diag(p, t.m, t.st));
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
}  // namespace cyc

using namespace cyc;

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
    if (int rc_ = trsm_diag_smem()) return rc_;
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
    if (int rc_ = trsm_diag_smem()) return rc_;
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
        if (ok(launch_trsm_diag(p, r1 - r0, s), "trsm_diag_kernel"))
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
