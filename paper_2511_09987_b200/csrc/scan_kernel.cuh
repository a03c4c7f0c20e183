// Prefix-sum recurrence P_i = P_{i-1} + A_i, P_{-1} = 0 (Figure "Representative recurrences"), for many independent
// rows in one pass over the data: 4 bytes read and 4 bytes written per element.
//
// The dependency of the recurrence runs along i.  A CTA owns a tile of 4096 consecutive elements of one row; inside the
// tile the running value is carried from thread to thread through registers and shuffles, and from tile to tile through
// one 64-bit descriptor per tile in global memory: a tile first publishes the sum of its own elements ("partial"), then
// looks back over its predecessors -- adding partial sums until it meets a tile that already knows its running value
// ("inclusive") -- and publishes its own running value.  Tiles take their index from a counter in launch order, so every
// predecessor of a tile is resident and makes progress; every wait is bounded.
//
// fp32: sums inside a tile are fp32, the value carried between tiles is fp64 (descriptor = the double with its two
// lowest significand bits replaced by the state), and P_i is the carried value plus the in-tile prefix rounded once.
// int32: two's-complement wrap-around, exact (descriptor = value << 32 | state).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace cyc {

constexpr int SCAN_THREADS = 256, SCAN_CHUNKS = 4, SCAN_TILE = SCAN_THREADS * SCAN_CHUNKS * 4;  // 4096 elements
constexpr int SCAN_WARPS = SCAN_THREADS / 32;
constexpr long long SCAN_WAIT_CYCLES = 1ll << 31;
constexpr unsigned long long SCAN_PARTIAL = 1, SCAN_INCLUSIVE = 2;

// header of the scratch block, followed by one descriptor per tile; zeroed before every launch
struct ScanHeader {
    unsigned int next_tile;
    int abort;
    unsigned long long pad;
};

template <typename T>
struct ScanParams {
    const T* A;
    T* P;
    long long n, strideA, strideP;
    long long tiles_per_row;
    ScanHeader* header;
    unsigned long long* desc;  // [rows * tiles_per_row]
    int* status;               // device status word
    int vec_ok;                // every row of A and P starts on a 16-byte boundary
};

template <typename T> struct ScanCarry;
template <> struct ScanCarry<float> {
    using type = double;
    static __device__ __forceinline__ unsigned long long pack(double v, unsigned long long state) {
        return (static_cast<unsigned long long>(__double_as_longlong(v)) & ~3ull) | state;
    }
    static __device__ __forceinline__ double value(unsigned long long w) { return __longlong_as_double(static_cast<long long>(w & ~3ull)); }
    static __device__ __forceinline__ float finish(double carry, float local) { return static_cast<float>(carry + static_cast<double>(local)); }
};
template <> struct ScanCarry<int> {
    using type = unsigned int;
    static __device__ __forceinline__ unsigned long long pack(unsigned int v, unsigned long long state) {
        return (static_cast<unsigned long long>(v) << 32) | state;
    }
    static __device__ __forceinline__ unsigned int value(unsigned long long w) { return static_cast<unsigned int>(w >> 32); }
    static __device__ __forceinline__ int finish(unsigned int carry, int local) { return static_cast<int>(carry + static_cast<unsigned int>(local)); }
};

__device__ __forceinline__ unsigned long long scan_ld_desc(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void scan_st_desc(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// wrap-around addition for int (signed overflow is undefined in C++), plain addition for float
__device__ __forceinline__ float scan_add(float a, float b) { return a + b; }
__device__ __forceinline__ int scan_add(int a, int b) { return static_cast<int>(static_cast<unsigned int>(a) + static_cast<unsigned int>(b)); }

template <typename T>
__global__ void __launch_bounds__(SCAN_THREADS) scan_kernel(const ScanParams<T> p) {
    using Carry = typename ScanCarry<T>::type;
    using V4 = typename std::conditional<std::is_same<T, float>::value, float4, int4>::type;
    __shared__ unsigned int s_tile;
    __shared__ T s_warp_total[SCAN_CHUNKS][SCAN_WARPS];
    __shared__ T s_warp_offset[SCAN_CHUNKS][SCAN_WARPS];
    __shared__ Carry s_carry;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        s_tile = atomicAdd(&p.header->next_tile, 1u);
        s_abort = 0;
    }
    __syncthreads();
    const long long tile = s_tile;
    const long long row = tile / p.tiles_per_row, tr = tile - row * p.tiles_per_row;
    const long long base = tr * SCAN_TILE;
    const int len = static_cast<int>(min(static_cast<long long>(SCAN_TILE), p.n - base));
    const T* a = p.A + row * p.strideA + base;
    T* out = p.P + row * p.strideP + base;

    // ---- load: chunk j of thread t holds elements (j * THREADS + t) * 4 .. + 3 (coalesced 16-byte accesses)
    T x[SCAN_CHUNKS][4];
#pragma unroll
    for (int j = 0; j < SCAN_CHUNKS; ++j) {
        const int at = (j * SCAN_THREADS + tid) * 4;
        if (p.vec_ok && at + 4 <= len) {
            const V4 v = __ldcs(reinterpret_cast<const V4*>(a + at));
            x[j][0] = v.x; x[j][1] = v.y; x[j][2] = v.z; x[j][3] = v.w;
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) x[j][c] = at + c < len ? __ldcs(a + at + c) : T(0);
        }
    }
    // ---- running value inside each chunk, then across the lanes of the warp (chunk by chunk)
    T incl[SCAN_CHUNKS], excl[SCAN_CHUNKS];
#pragma unroll
    for (int j = 0; j < SCAN_CHUNKS; ++j) {
        x[j][1] = scan_add(x[j][0], x[j][1]);
        x[j][2] = scan_add(x[j][1], x[j][2]);
        x[j][3] = scan_add(x[j][2], x[j][3]);
        T w = x[j][3];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const T up = __shfl_up_sync(0xffffffffu, w, d);
            if (lane >= d) w = scan_add(up, w);
        }
        incl[j] = w;
        const T before = __shfl_up_sync(0xffffffffu, w, 1);
        excl[j] = lane ? before : T(0);
        if (lane == 31) s_warp_total[j][warp] = w;
    }
    __syncthreads();

    // ---- warp 0: running value over the (chunk, warp) totals in element order, the tile's sum, and the look-back
    if (warp == 0) {
        static_assert(SCAN_CHUNKS * SCAN_WARPS == 32, "one lane per (chunk, warp) total");
        const T mine = s_warp_total[lane / SCAN_WARPS][lane % SCAN_WARPS];
        T w = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const T up = __shfl_up_sync(0xffffffffu, w, d);
            if (lane >= d) w = scan_add(up, w);
        }
        const T before = __shfl_up_sync(0xffffffffu, w, 1);
        s_warp_offset[lane / SCAN_WARPS][lane % SCAN_WARPS] = lane ? before : T(0);
        const T tile_sum = __shfl_sync(0xffffffffu, w, 31);
        const Carry own = static_cast<Carry>(tile_sum);

        Carry carry = Carry(0);
        bool ok = true;
        if (tr == 0) {
            if (lane == 0) scan_st_desc(&p.desc[tile], ScanCarry<T>::pack(own, SCAN_INCLUSIVE));
        } else {
            if (lane == 0) scan_st_desc(&p.desc[tile], ScanCarry<T>::pack(own, SCAN_PARTIAL));
            const long long first = tile - tr;  // first tile of this row
            long long pos = tile - 1;           // nearest predecessor not yet added
            const long long t0 = clock64();
            while (true) {
                const long long idx = pos - lane;
                const bool in_row = idx >= first;
                // a lane past the start of the row behaves like a finished tile with value zero: the walk ends there
                unsigned long long word = ScanCarry<T>::pack(Carry(0), SCAN_INCLUSIVE);
                unsigned int spins = 0;
                while (true) {
                    if (in_row) word = scan_ld_desc(&p.desc[idx]);
                    if (__all_sync(0xffffffffu, (word & 3ull) != 0)) break;
                    if ((++spins & 63u) == 0) {
                        int give_up = 0;
                        if (lane == 0) {
                            give_up = *reinterpret_cast<volatile int*>(&p.header->abort);
                            if (!give_up && clock64() - t0 > SCAN_WAIT_CYCLES) {
                                atomicExch(&p.header->abort, 1);
                                atomicExch(p.status, 0x400);
                                give_up = 1;
                            }
                        }
                        if (__shfl_sync(0xffffffffu, give_up, 0)) { ok = false; break; }
                    }
                }
                if (!ok) break;
                const unsigned int done = __ballot_sync(0xffffffffu, (word & 3ull) == SCAN_INCLUSIVE);
                const int stop = done ? __ffs(done) - 1 : 32;  // nearest tile that knows its running value
                Carry v = lane <= stop ? ScanCarry<T>::value(word) : Carry(0);
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
                carry += v;
                if (done) break;
                pos -= 32;
            }
            if (ok && lane == 0) scan_st_desc(&p.desc[tile], ScanCarry<T>::pack(carry + own, SCAN_INCLUSIVE));
        }
        if (lane == 0) {
            s_carry = carry;
            s_abort = ok ? 0 : 1;
        }
    }
    __syncthreads();
    if (s_abort) return;

    // ---- P_i = carried value + prefix inside the tile
    const Carry carry = s_carry;
#pragma unroll
    for (int j = 0; j < SCAN_CHUNKS; ++j) {
        const int at = (j * SCAN_THREADS + tid) * 4;
        const T before = scan_add(s_warp_offset[j][warp], excl[j]);
        T r[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) r[c] = ScanCarry<T>::finish(carry, scan_add(before, x[j][c]));
        if (p.vec_ok && at + 4 <= len) {
            V4 v;
            v.x = r[0]; v.y = r[1]; v.z = r[2]; v.w = r[3];
            __stcs(reinterpret_cast<V4*>(out + at), v);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (at + c < len) __stcs(out + at + c, r[c]);
        }
    }
    (void)incl;
}

}  // namespace cyc
