/*
 * cyc.h -- C ABI of the B200 (sm_100a) evaluator of the weight-stationary
 * systolic matrix-multiply recurrence
 *
 *        [i,k]_C <- [i,k-1]_C + [i,k]_W * [i,k]_B ,   [i,0-1]_C = 0 ,
 *        C_ij    <- [i,k_end]_C
 *
 * (weight-stationary program of Section "Space-time Mappings of Dataflow
 * Recurrences" and the nine per-cell programs of Figure "perPE": W = A_ik is
 * held in cell (i,k), B_kj is injected at the north boundary and copied along
 * i, the partial sum moves along k, and C_ij = sum_k A_ik B_kj leaves the
 * array at k_end -- the export rule of Section "Explicit Communication and
 * Loads into Iteration Space").
 *
 * All pointers are DEVICE pointers unless a function says otherwise.  The
 * caller owns every buffer; the library reads A and B, overwrites C, and keeps
 * no reference once the kernels it enqueued have completed.  C must not
 * overlap A or B.  Calls are asynchronous: work is enqueued on `stream` and the
 * function returns without synchronising.  The functions never throw, never
 * abort and are safe to call from several host threads.
 *
 * Environment.  CYC_LOG=1 (read once per process): one line on stderr for every
 * kernel selection of the matrix-multiply recurrence -- shape, dtype, flags,
 * pitches and the kernel chosen (the names of cyc_kernel_for) -- including the
 * tile products that the triangular solve and the Cholesky factorisation lay on it,
 * and for every attention launch its grid (units, sliced tail).
 *
 * Device memory the library holds besides the caller's buffers: a 4-byte status word per
 * device; a stream-ordered pool for split-K and solver workspaces (cyc_pool_reserved_bytes);
 * the fixed array of cyc_recurrence_matmul_splitk_static; and, for schedules with a sliced
 * tail, one scratch per (device, stream) -- 19.4 MB for the matrix multiply, 21.3 MB for
 * attention, at most eight of each per device -- allocated the first time such a schedule
 * runs on a stream and kept until the process exits (a stream beyond the eighth, or one that
 * is being captured before it has a scratch, runs the schedule without a sliced tail).  A call
 * captured into a CUDA graph keeps using the scratch of the stream it was captured on: replays
 * of such graphs must not overlap one another.
 *
 * Layouts.  A is [M][K] row-major (K contiguous).  B is [K][N] row-major, or,
 * with CYC_FLAG_B_COL_MAJOR, stored as [N][K] (element B_kj at B[j*K + k]).
 * C is [M][N] row-major and is written completely (the recurrence starts from
 * zero; there is no accumulate-into-C).
 *
 * Arithmetic.
 *   CYC_F32       A, B, C float.   With CYC_FLAG_FIXED_K_ORDER every C_ij is
 *                 the chain acc = fma(A_ik, B_kj, acc), k = 0,1,..,K-1, acc
 *                 starting at +0 (one rounding per cell, round to nearest
 *                 even): bit-reproducible.  Without the flag the library may
 *                 evaluate the sum on tensor cores with each operand split
 *                 into two TF32 parts and fp32 accumulation (error well inside
 *                 1e-5 * sum_k |A_ik||B_kj|).  Infinite or NaN inputs make exactly
 *                 the C_ij they reach non-finite, but an infinite C_ij may come out
 *                 as NaN (an infinite part of one operand meeting a part of the
 *                 other that is exactly zero); the flag gives IEEE results.
 *   CYC_BF16_F32  A, B bfloat16; products exact; fp32 accumulation; C float.
 *                 k-blocks are accumulated in increasing order; results are
 *                 run-to-run identical with or without the flag (no atomics) for
 *                 the same arguments on the same stream.  Without the flag the
 *                 grouping of the fp32 additions follows the schedule (k-slices,
 *                 sliced tail), so a call on a stream that runs another schedule
 *                 (see "Device memory" above) may differ in the last bits.
 *                 Without the flag, problems with few output tiles and a long k
 *                 loop are cut into k-slices whose partial sums are added in
 *                 slice order (split-K; needs a workspace from a stream-ordered
 *                 pool the library owns); with the flag one CTA pair owns each
 *                 C_ij for the whole k loop.
 *   CYC_I8_I32    A, B signed 8-bit; C int32; exact for K <= 131071.
 */
#ifndef CYC_H_
#define CYC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CYC_F32 = 0,
    CYC_BF16_F32 = 1,
    CYC_I8_I32 = 2,
    CYC_I32 = 3 /* int32 in, int32 out, wrap-around: cyc_prefix_sum only */
} cyc_dtype_t;

enum {
    CYC_FLAG_FIXED_K_ORDER = 1u, /* deterministic; one owner per C_ij; k strictly increasing */
    CYC_FLAG_B_COL_MAJOR = 2u    /* B is stored as [N][K] */
};

typedef enum {
    CYC_OK = 0,
    CYC_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, unknown dtype or flag bit, bad stride */
    CYC_ERR_UNSUPPORTED = 2, /* valid request this build cannot serve (e.g. int8 with K > 131071, not an sm_100 device) */
    CYC_ERR_CUDA = 3,        /* a CUDA runtime or driver call failed; see cyc_last_cuda_error */
    CYC_ERR_TIMEOUT = 4      /* a bounded device-side wait ran out; C is undefined */
} cyc_status_t;

/*
 * Evaluate the recurrence for one problem: C[M][N] = sum_k A[M][K] B[K][N]
 * (the whole hot path: weight load, B injection, zero initial partial sum,
 * the multiply-accumulate along k, and the export of C_ij at k_end).
 *
 *   M, N, K  >= 1; any values (no tile-multiple requirement).
 *   dtype    a cyc_dtype_t.
 *   A, B, C  device pointers, aligned to the element size; 16-byte alignment
 *            and row pitches that are multiples of 16 bytes select the
 *            tensor-core kernels, anything else runs on a slower general kernel.
 *   stream   a cudaStream_t (0 = the default stream).
 *   flags    OR of CYC_FLAG_*.
 * Returns a cyc_status_t.  Argument errors are found on the host before any
 * CUDA call is made.
 */
int cyc_recurrence_matmul(int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B, void* C, void* stream,
                          unsigned flags);

/*
 * `batch` independent recurrences in one launch: problem b uses
 * A + b*strideA, B + b*strideB, C + b*strideC (strides in ELEMENTS of the
 * respective type; 0 selects the contiguous default M*K, K*N, M*N).  Strides
 * smaller than one matrix are rejected.  Everything else as above.
 */
int cyc_recurrence_matmul_batched(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A, int64_t strideA,
                                  const void* B, int64_t strideB, void* C, int64_t strideC, void* stream, unsigned flags);

/*
 * HOST-memory convenience: A, B and C are host pointers (same layouts).  The
 * library allocates device buffers, copies A and B in, evaluates the
 * recurrence, copies C out, frees the buffers and synchronises `stream`
 * before returning.  For callers without their own device memory management
 * and for end-to-end timing.
 */
int cyc_recurrence_matmul_host(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A_host,
                               const void* B_host, void* C_host, void* stream, unsigned flags);

/*
 * Split-K evaluation of ONE bf16 or int8 problem that never allocates (the paper has
 * no counterpart; this is a service for hosts of the library).
 *
 * Who needs it: a program that gave all device memory to its own allocator at start-up,
 * or a latency-critical loop that must never enter the driver's allocator (which may
 * block, synchronise the device, or fail under memory pressure), cannot use the split-K
 * path of cyc_recurrence_matmul, whose partial sums go through a stream-ordered pool.
 * Here the partial sums go through a fixed array of CYC_STATIC_WORKSPACE_BYTES that is
 * part of the library image: every device that loads the library holds it until the
 * process exits, used or not.
 *
 *   A, B, C, stream, layouts, dtype: as for cyc_recurrence_matmul, restricted to
 *   CYC_BF16_F32 and CYC_I8_I32, 16-byte aligned bases and row pitches, M > 128, N > 128.
 *   flags: CYC_FLAG_B_COL_MAJOR or 0 (CYC_FLAG_FIXED_K_ORDER contradicts split-K:
 *   CYC_ERR_INVALID_ARG).
 * The k loop is cut into S >= 2 slices (as many as there are idle CTA pairs, >= 8
 * k-blocks each) and S*M*N*4 bytes must fit the array; S is reduced to fit, and a
 * problem for which not even two slices fit (2*M*N*4 > CYC_STATIC_WORKSPACE_BYTES), or
 * whose k loop is shorter than 16 k-blocks, is refused with CYC_ERR_UNSUPPORTED and a
 * message in cyc_last_cuda_error().  Results equal the split-K path of
 * cyc_recurrence_matmul when both pick the same S, and stay within the usual tolerance
 * otherwise (int8: exact).
 * The first call on each device looks up the array's device address with
 * cudaGetSymbolAddress; make that first call outside any stream capture.  The look-up
 * itself requests no memory, but if nothing of the library has run on the device yet,
 * the CUDA runtime loads the library's device code at that moment (lazy module loading),
 * and that is when the device receives its copy of the array: after one warm-up call per
 * device, no call of this function allocates or frees memory -- neither through
 * cudaMalloc / cudaFree nor through the library's pool (cyc_pool_reserved_bytes reports
 * the pool's size for those who want to check).  Nothing in the array needs clearing: every
 * element a call reads was written by the same call.  All calls share the one array, so
 * two calls whose kernels can overlap on the GPU (different streams, no dependency) race
 * on it: order them on one stream or with events.
 */
#define CYC_STATIC_WORKSPACE_BYTES (8u << 20)
int cyc_recurrence_matmul_splitk_static(int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B, void* C,
                                        void* stream, unsigned flags);

/*
 * Bytes the library's stream-ordered workspace pool currently holds from the driver on
 * the current device (cudaMemPoolAttrReservedMemCurrent; 0 if no call has needed the
 * pool yet).  Introspection only (the paper has no counterpart): lets a host verify
 * that a sequence of calls did not grow the library's memory.
 */
int cyc_pool_reserved_bytes(int64_t* out);

/*
 * Block lower-triangular solve  L X = B  (Section "Multiple Iteration Spaces":
 *     X_i = TRSM( L_ii , B_i - sum_{j<i} GEMM(L_ij, X_j) ),
 * recurrences of Figure "deps-tri-solve"): a triangular iteration space of tile products
 * whose accumulators run along j, and a diagonal space of small triangular solves that
 * consume the end of each row and seed the next block column.
 *
 *   n      order of L;  m  number of right-hand sides (columns of B and X);  n, m >= 1
 *   tile   edge T of the square tiles of both spaces, 1 .. 256; 0 selects 256.  The last
 *          tile may be ragged.  T changes only the grouping of the additions (results
 *          differ by roundings), not the mathematical result.
 *   dtype  CYC_F32 (fp32 in, fp32 arithmetic, fp32 out); the other types are refused
 *          with CYC_ERR_UNSUPPORTED
 *   L      DEVICE, [n][n] row-major; only entries on and below the diagonal are read
 *          (the rest may hold anything, NaN included).  A zero on the diagonal gives
 *          infinities or NaN in X, as the division does; it is not an error.
 *   B      DEVICE, [n][m] row-major
 *   X      DEVICE, [n][m] row-major, fully overwritten.  X may be the very same buffer as
 *          B (in place); any other overlap of X with B or L is CYC_ERR_INVALID_ARG.
 *   stream cudaStream_t; every kernel is enqueued there, the call does not synchronise
 *   flags  0, or CYC_FLAG_FIXED_K_ORDER: the tile products then run as per-element fp32
 *          fused-multiply-add chains in increasing k (bit-reproducible, slower); without
 *          it they may run on the tensor cores (fp32 split into TF32 parts).
 * The tile products of the triangular space are evaluated by the same kernels as
 * cyc_recurrence_matmul (operand A = a sub-block of L, row pitch n); their partial sums
 * pass through a workspace of ceil(log2(ceil(n/T))) * n * m * 4 bytes taken from the
 * library's stream-ordered pool for the duration of the call.  The diagonal tiles are
 * solved by forward substitution in fp32 (rows scaled by the correctly rounded reciprocal
 * of their diagonal entry).  Caller owns L, B, X;
 * the library keeps no reference after the kernels complete.  Errors as for
 * cyc_recurrence_matmul.
 */
int cyc_block_trsm(int64_t n, int64_t m, int64_t tile, int dtype, const void* L, const void* B, void* X, void* stream,
                   unsigned flags);

/*
 * FlashAttention-2 recurrence (Section "Simulated Cholesky and Flash Attention"): for every
 * query row i, over key tiles J_t,
 *     S = alpha Q_i K_{J_t}^T,  mh = max(m, max S),  l <- e^(m-mh) l + sum_j e^(S_j-mh),
 *     o <- e^(m-mh) o + sum_j e^(S_j-mh) V_j,  m <- mh;      O_i = o / l,  alpha = 1/sqrt(d),
 * which equals softmax(alpha Q K^T) V.  `batch` independent problems (batch x heads, flattened).
 *
 *   Q      DEVICE, [batch][N][d] bf16, row-major, 16-byte aligned
 *   K, V   DEVICE, [batch][M][d] bf16
 *   O      DEVICE, [batch][N][d] fp32, fully overwritten, 16-byte aligned, must not overlap an input
 *   dtype  CYC_BF16_F32 (bf16 in; scores, normaliser and output accumulated in fp32; the
 *          exponentials enter the second product rounded to bf16); d = 64 or 128.  Anything
 *          else is refused with CYC_ERR_UNSUPPORTED.
 *   flags  0 (the paper's recurrence has no mask and no other scale)
 * N, M >= 1 need not be multiples of the tile sizes (128 queries, 128 keys).  Asynchronous on
 * `stream`; the caller owns all buffers; errors as for cyc_recurrence_matmul.
 * Results are run-to-run identical for the same arguments on the same stream.  Where the last
 * round of the grid is cut by key range (see "Device memory" above) the parts round their
 * exponentials against their own reference maxima, so a call that runs without that cut (a
 * stream without scratch, a capture on such a stream) agrees with one that runs with it to the
 * bf16 rounding of the exponentials, not bit for bit.
 */
int cyc_flash_attention(int64_t batch, int64_t N, int64_t M, int64_t d, int dtype, const void* Q, const void* K, const void* V,
                        void* O, void* stream, unsigned flags);

/*
 * Prefix-sum recurrence (Figure "Representative recurrences"):  P_i = P_{i-1} + A_i, read with
 * P_{-1} = 0, i.e. P_i = A_0 + ... + A_i, for `rows` independent sequences of n elements.
 *
 *   A      DEVICE, element i of sequence r at A[r * strideA + i]
 *   P      DEVICE, same indexing with strideP; fully overwritten for i < n.  P may be the very
 *          same buffer as A with the same stride (in place); any other overlap is
 *          CYC_ERR_INVALID_ARG.
 *   strideA, strideP   in elements, >= n; 0 means n (sequences back to back)
 *   dtype  CYC_F32: sums of neighbouring elements are formed in fp32 inside runs of 128
 *          elements, everything carried further (across a tile of 16384 or 8192 elements and from
 *          tile to tile) is fp64: |P_i - exact| <= 1e-6 * sum_{k<=i} |A_k|, independent of n.  The order in
 *          which tile sums are combined follows their arrival, so the last bit of a result may
 *          differ between runs.
 *          CYC_I32: two's-complement 32-bit integers, wrap-around on overflow; exact and
 *          run-to-run identical.  Other types are refused with CYC_ERR_UNSUPPORTED.
 *   flags  0
 * rows, n >= 1; rows * ceil(n / 8192) < 2^31.  One pass over the data (each element read once,
 * written once) in a single kernel; the tile descriptors (8 bytes per tile of 16384 elements, 8192 for rows of at most 262144 elements) come from
 * the library's stream-ordered pool for the duration of the call.  Asynchronous on `stream`;
 * the caller owns A and P; errors as for cyc_recurrence_matmul.
 */
int cyc_prefix_sum(int64_t rows, int64_t n, int dtype, const void* A, int64_t strideA, void* P, int64_t strideP, void* stream,
                   unsigned flags);

/*
 * Tiled Cholesky recurrence (Section "Simulated Cholesky and Flash Attention"; scalar form in
 * Figure "Representative recurrences"): the lower-triangular L with A = L L^T, panel by panel,
 *     L_jj = CHOL(A_jj - sum_{k<j} SYRK(L_jk)),   L_ij = TRSM(A_ij - sum_{k<j} GEMM(L_ik, L_jk), L_jj),  i > j.
 *
 *   n      order of A;  n >= 1
 *   tile   edge of the square tiles, 1 .. 256; 0 selects 256.  The last tile may be ragged.  The
 *          tile size changes only the grouping of the additions, not the mathematical result.
 *   dtype  CYC_F32 (fp32 in, fp32 arithmetic, fp32 out); other types: CYC_ERR_UNSUPPORTED
 *   A      DEVICE, [n][n] row-major, symmetric positive definite; only entries on and below the
 *          diagonal are read (the rest may hold anything, NaN included)
 *   L      DEVICE, [n][n] row-major.  Entries on and below the diagonal receive the factor.  L may
 *          be the very same buffer as A (in place: entries above the diagonal are then left as
 *          they are); otherwise the two must not overlap and entries above the diagonal are set
 *          to zero.
 *   flags  0, or CYC_FLAG_FIXED_K_ORDER: the SYRK / GEMM sums then run as per-element fp32
 *          fused-multiply-add chains in increasing k (bit-reproducible, slower); without it they
 *          may run on the tensor cores (fp32 split into TF32 parts).
 * A matrix that is not positive definite yields NaN (or infinities) from the square root of a
 * non-positive pivot, as the recurrence does; it is not an error.  The SYRK / GEMM sums are evaluated by the
 * same kernels as cyc_recurrence_matmul (both operands sub-blocks of L with row pitch n) into a
 * workspace of (n - T) * T * 4 bytes from the library's stream-ordered pool; everything
 * else is fp32; L_kk and the divisions by it are products with 1 / sqrt(pivot), computed to
 * about 1e-7 relative (hardware reciprocal square root and one Newton step).
 * Asynchronous on `stream`; the caller owns A and L; errors as for cyc_recurrence_matmul.
 */
int cyc_cholesky(int64_t n, int64_t tile, int dtype, const void* A, void* L, void* stream, unsigned flags);

/*
 * Synchronise `stream` and report whether a kernel enqueued by this library on
 * the current device since the previous call of this function gave up on a
 * bounded wait.  *out (HOST pointer, may be NULL) receives CYC_OK or
 * CYC_ERR_TIMEOUT; the return value is CYC_OK unless the synchronisation
 * itself failed (CYC_ERR_CUDA).
 */
int cyc_last_device_status(void* stream, int* out);

/*
 * Self-test of the failure path (no counterpart in the paper): enqueue a one-CTA kernel whose
 * only wait can never be satisfied and which gives up after `budget_cycles` SM clocks
 * (1 .. 2^24, i.e. at most about ten milliseconds), exactly as the bounded waits of the real
 * kernels do.  The kernel ends normally; the next cyc_last_device_status reports
 * CYC_ERR_TIMEOUT once and the device stays usable.
 */
int cyc_selftest_bounded_wait(void* stream, int64_t budget_cycles);

/* Name of the kernel the dispatcher would pick for these arguments -- "simt" (general
 * kernel), "tcgen05" (one CTA per tile), "tcgen05_pair" (CTA pair, 256x256 tiles),
 * "tcgen05_pair_tall" (CTA pair, 512x256 tiles), "tcgen05_pair_splitk" (few tiles, long k
 * loop: k-slices on different CTA pairs, partial sums added in slice order by a second kernel),
 * "tcgen05_3xtf32" (fp32 split into TF32 parts), "tcgen05_3xtf32_ws" (the same with a small B
 * kept in tensor memory while a long A streams past it) -- or NULL if the arguments are invalid.
 * Host only, makes no CUDA call. */
const char* cyc_kernel_for(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B,
                           const void* C, unsigned flags);

/* Which space-time mapping of the base recurrence the dispatcher would use for these
 * arguments (Section "Space-time Mappings of Dataflow Recurrences" prints a
 * weight-stationary and an output-stationary program for the same recurrence):
 *   "output_stationary"  every block of C stays in place (tensor memory or registers) for
 *                        its whole k loop while A and B stream past it -- k runs in time,
 *                        one owner per C_ij; what CYC_FLAG_FIXED_K_ORDER always selects;
 *   "k_sliced"           the k range of a block is cut into slices held by different CTA
 *                        pairs at the same time (k partly in space) and the slices' partial
 *                        sums are added in increasing k by a second kernel;
 *   "output_stationary+k_sliced_tail"
 *                        output-stationary, except that the blocks left over after the last
 *                        full round of CTA pairs (which would keep only some pairs busy for
 *                        a whole k loop) are cut into k-slices spread over all pairs; for
 *                        each strip of such a block the pair that finishes last adds the
 *                        slices' partial sums in increasing k inside the same kernel
 *                        (assumes a B200's 74 CTA pairs; never under CYC_FLAG_FIXED_K_ORDER).
 * NULL if the arguments are invalid.  Host only, makes no CUDA call. */
const char* cyc_schedule_for(int64_t batch, int64_t M, int64_t N, int64_t K, int dtype, const void* A, const void* B,
                             const void* C, unsigned flags);

/* Number of kernels this library has launched in the calling process (monotonic). */
int64_t cyc_launch_count(void);

/* Text of the last CUDA error this library saw in the calling thread ("" if none). */
const char* cyc_last_cuda_error(void);

const char* cyc_status_string(int status);
int cyc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CYC_H_ */
