// Shared state and helpers of the library, and the status / introspection entry points.  See include/cyc.h.
#include <cstdlib>

#include "api_internal.h"
#include "ptx.cuh"

namespace cyc {

// raised by a kernel whose bounded wait ran out; one word per device (module scope)
__device__ int g_device_status = 0;
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
std::atomic<long long> g_launches{0};
thread_local char g_err[512] = "";

int cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_err, sizeof g_err, "%s: %s", what, cudaGetErrorString(e));
    return CYC_ERR_CUDA;
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
int make_map_raw(CUtensorMap* m, CUtensorMapDataType dt, int eb, const void* base, long long d0, long long d1, long long d2,
                        long long pitch1_elems, long long pitch2_elems, int box0, int box1,
                        CUtensorMapSwizzle swizzle) {
    // Descriptor cache: a map is a pure function of these arguments, and callers come back with the same buffers step
    // after step, so each host thread keeps the last maps it encoded (direct-mapped, 64 entries) and copies 128 bytes
    // instead of calling the driver.
    struct Key {
        const void* base;
        long long d0, d1, d2, p1, p2;
        int dt, eb, box0, box1, swizzle;
        bool operator==(const Key& o) const {
            return base == o.base && d0 == o.d0 && d1 == o.d1 && d2 == o.d2 && p1 == o.p1 && p2 == o.p2 && dt == o.dt && eb == o.eb &&
                   box0 == o.box0 && box1 == o.box1 && swizzle == o.swizzle;
        }
    };
    struct Entry {
        Key key;
        CUtensorMap map;
        bool valid;
    };
    constexpr int kEntries = 64;
    thread_local Entry cache[kEntries] = {};
    const Key key{base, d0, d1, d2, pitch1_elems, pitch2_elems, static_cast<int>(dt), eb, box0, box1, static_cast<int>(swizzle)};
    unsigned long long h = reinterpret_cast<uintptr_t>(base) * 0x9E3779B97F4A7C15ull;
    h ^= static_cast<unsigned long long>(d0 * 31 + d1 * 131 + d2 * 521 + pitch1_elems * 8191 + box0 * 7 + box1 * 3 + static_cast<int>(swizzle));
    Entry& e = cache[(h ^ (h >> 29)) % kEntries];
    if (e.valid && e.key == key) {
        memcpy(m, &e.map, sizeof(CUtensorMap));
        return CYC_OK;
    }
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
    e.key = key;
    memcpy(&e.map, m, sizeof(CUtensorMap));
    e.valid = true;
    return CYC_OK;
}

// operand map (A or B) in the problem's input type
int make_map(CUtensorMap* m, int dtype, const void* base, long long d0, long long d1, long long d2, long long pitch1_elems,
                    long long pitch2_elems, int box0, int box1, CUtensorMapSwizzle swizzle) {
    const CUtensorMapDataType dt = dtype == CYC_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                    : (dtype == CYC_BF16_F32 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8);
    return make_map_raw(m, dt, elem_bytes(dtype), base, d0, d1, d2, pitch1_elems, pitch2_elems, box0, box1, swizzle);
}

int device_info(DeviceInfo* out) {
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
int status_word(int** out) {
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

int ensure_dynamic_smem(const void* kernel, int bytes) {
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
// Workspace for partial sums and scratch: stream-ordered allocations from a pool the library owns (one per device),
// so that repeated calls reuse the same memory without a synchronising cudaMalloc.
int workspace_pool(cudaMemPool_t* out, bool create) {
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
// CYC_LOG=1 in the environment: one line on stderr per kernel selection (read once per process)
bool log_enabled() {
    static const bool on = [] {
        const char* v = getenv("CYC_LOG");
        return v && *v && *v != '0';
    }();
    return on;
}

// ------------------------------------------------------------------ scratch kept per (device, stream, purpose)
struct KeptScratch {
    int dev = -1;
    cudaStream_t stream = nullptr;
    int purpose = 0;
    uint8_t* data = nullptr;
    int* counters = nullptr;
    size_t counter_bytes = 0;
    bool dirty = false;
};
constexpr int kKeptScratchPerDevice = 8;  // per purpose
constexpr int kKeptScratchMax = 128;
static std::mutex g_scratch_mu;
static KeptScratch g_scratch[kKeptScratchMax];
static int g_scratch_count = 0;

void kept_scratch_mark_dirty() {
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    for (int i = 0; i < g_scratch_count; ++i) g_scratch[i].dirty = true;
}

int kept_scratch_for(cudaStream_t st, int purpose, size_t data_bytes, size_t counter_bytes, uint8_t** data, int** counters) {
    *data = nullptr;
    *counters = nullptr;
    int dev = 0;
    CYC_CUDA(cudaGetDevice(&dev));
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); return CYC_OK; }
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    KeptScratch* found = nullptr;
    int on_dev = 0;
    for (int i = 0; i < g_scratch_count; ++i) {
        if (g_scratch[i].dev != dev || g_scratch[i].purpose != purpose) continue;
        ++on_dev;
        if (g_scratch[i].stream == st) found = &g_scratch[i];
    }
    if (!found) {
        // creating one allocates and clears memory: not while the stream is being captured into a graph
        if (cap != cudaStreamCaptureStatusNone || on_dev >= kKeptScratchPerDevice || g_scratch_count >= kKeptScratchMax) return CYC_OK;
        const size_t data_padded = (data_bytes + 255) & ~static_cast<size_t>(255);
        void* mem = nullptr;
        if (cudaMalloc(&mem, data_padded + counter_bytes) != cudaSuccess) { cudaGetLastError(); return CYC_OK; }
        if (cudaMemset(static_cast<uint8_t*>(mem) + data_padded, 0, counter_bytes) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(mem);
            return CYC_OK;
        }
        found = &g_scratch[g_scratch_count++];
        found->dev = dev;
        found->stream = st;
        found->purpose = purpose;
        found->data = static_cast<uint8_t*>(mem);
        found->counters = reinterpret_cast<int*>(found->data + data_padded);
        found->counter_bytes = counter_bytes;
        found->dirty = false;
    }
    if (found->dirty) {
        if (cap != cudaStreamCaptureStatusNone) return CYC_OK;
        CYC_CUDA(cudaMemsetAsync(found->counters, 0, found->counter_bytes, st));
        found->dirty = false;
    }
    *data = found->data;
    *counters = found->counters;
    return CYC_OK;
}

}  // namespace cyc

using namespace cyc;

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
        kept_scratch_mark_dirty();  // a kernel that gave up may have left arrival counters of a sliced tail non-zero
        CYC_CUDA(cudaMemcpyToSymbol(g_device_status, &zero, sizeof zero));
        snprintf(g_err, sizeof g_err, "device wait ran out (code 0x%x)", word);
    }
    if (out) *out = word != 0 ? CYC_ERR_TIMEOUT : CYC_OK;
    return CYC_OK;
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
