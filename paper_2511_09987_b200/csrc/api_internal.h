// Internals shared by the translation units of the library (one per recurrence): the problem description, validation,
// kernel selection of the matrix-multiply recurrence, tensor maps, per-device caches, the workspace pool and the launch
// helper.  Not part of the public interface (that is include/cyc.h).
#pragma once
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

namespace cyc {

extern std::atomic<long long> g_launches;   // kernels launched by this process
extern thread_local char g_err[512];        // text of the last CUDA error seen by the calling thread

int cuda_fail(cudaError_t e, const char* what);
#define CYC_CUDA(call)                                    \
    do {                                                  \
        cudaError_t e_ = (call);                          \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

// Launch with programmatic stream serialisation: the kernel may be scheduled while the kernel before it on the stream
// is still running; each kernel launched this way executes griddepcontrol.wait before it touches global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st, Args&&... args) {
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

inline int elem_bytes(int dtype) { return dtype == CYC_F32 ? 4 : (dtype == CYC_BF16_F32 ? 2 : 1); }

struct Problem {
    long long batch, M, N, K;
    int dtype;
    const void *A, *B;
    void* C;
    long long sA, sB, sC;
    unsigned flags;
    long long lda = 0;  // row pitch of A in elements; 0 = dense (K).  Only internal callers set it (sub-blocks of L).
    long long ldb = 0;  // pitch of B in elements (between rows k, or between columns j when stored [N][K]); 0 = dense
};inline long long lda_of(const Problem& q) { return q.lda ? q.lda : q.K; }
inline long long ldb_of(const Problem& q) { return q.ldb ? q.ldb : ((q.flags & CYC_FLAG_B_COL_MAJOR) ? q.K : q.N); }

constexpr long long kCtaPairs = 74;  // CTA pairs resident on a B200 (148 SMs); used by the tile-shape rule

int validate(const Problem& q);                    // host-side validation; no CUDA call
int route(const Problem& q, cudaStream_t st);      // kernel selection and launch for a validated problem (also for the
                                                   // sub-problems the library builds itself)
int dispatch(const Problem& q, cudaStream_t st);   // validate, then route

// rank-3 tensor map over a [d2][d1][d0] array of the problem's input type (d0 contiguous), box [1][box1][box0]
int make_map(CUtensorMap* m, int dtype, const void* base, long long d0, long long d1, long long d2, long long pitch1_elems,
             long long pitch2_elems, int box0, int box1, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B);
int make_map_raw(CUtensorMap* m, CUtensorMapDataType dt, int eb, const void* base, long long d0, long long d1, long long d2,
                 long long pitch1_elems, long long pitch2_elems, int box0, int box1,
                 CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B);

struct DeviceInfo {
    int sms = 0, cc_major = 0;
    bool known = false;
};
int device_info(DeviceInfo* out);
bool log_enabled();                                       // CYC_LOG=1 in the environment
int status_word(int** out);                               // device address of the status word, cached per device
int ensure_dynamic_smem(const void* kernel, int bytes);   // opt-in to large dynamic shared memory, once per (kernel, device)
int workspace_pool(cudaMemPool_t* out, bool create = true);  // the library's stream-ordered pool on the current device
// Scratch kept for the life of the process, one per (device, stream, purpose): `data_bytes` of partial results and
// `counter_bytes` of arrival counters that are zero when a launch starts and that the kernel leaves zero.  Launches on
// one stream are ordered, launches on different streams are not, hence one scratch per stream; at most eight are made
// per device and purpose.  *data stays nullptr (and the call returns CYC_OK) when none can be had -- the stream is being
// captured and has no scratch yet, the limit is reached, or the allocation failed -- and the caller then runs a
// schedule that needs none.  A purpose always asks for the same sizes.
enum ScratchPurpose { SCRATCH_MATMUL_TAIL = 0, SCRATCH_ATTENTION_TAIL = 1 };
int kept_scratch_for(cudaStream_t st, int purpose, size_t data_bytes, size_t counter_bytes, uint8_t** data, int** counters);
void kept_scratch_mark_dirty();  // after a device-side timeout counters may be non-zero: the next use of each scratch clears them

}  // namespace cyc
