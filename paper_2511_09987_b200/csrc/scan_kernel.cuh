// Prefix-sum recurrence P_i = P_{i-1} + A_i, P_{-1} = 0 (Figure "Representative recurrences"), for many independent
// rows in one pass over the data: 4 bytes read and 4 bytes written per element.
//
// The dependency of the recurrence runs along i.  A CTA owns a tile of 16384 consecutive elements of one row, fetched
// into shared memory as four bulk copies of 16 KB (one mbarrier each, so the arithmetic starts when the first quarter
// has landed).  Inside the tile the running value is carried through registers and shuffles (groups of four elements,
// then the lanes of a warp) and the 128 warp-level sums of a tile are combined in element order by one warp; from tile
// to tile it is carried through one 64-bit descriptor per tile in global memory: a tile first publishes the sum of its
// own elements ("partial"), then looks back over its predecessors -- adding partial sums until it meets a tile that
// already knows its running value ("inclusive") -- and publishes its own running value.  Along one long row the running
// value advances by at most one look-back window per descriptor round trip (about a microsecond under load), which is
// why tiles are this large.  Tiles take their index from a counter
// in launch order, so every predecessor of a tile is resident and makes progress; every wait is bounded.
//
// fp32: sums inside a warp's 128 elements are fp32; warp-level sums, tile sums and the value carried between tiles are
// fp64 (descriptor = the double with its two lowest significand bits replaced by the state); P_i is rounded to fp32 at
// the end.  int32: two's-complement wrap-around, exact (descriptor = value << 32 | state).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "ptx.cuh"

namespace cyc {

constexpr int SCAN_THREADS = 256, SCAN_CHUNKS = 4, SCAN_SUB = SCAN_THREADS * SCAN_CHUNKS * 4;  // 4096 elements per quarter
constexpr int SCAN_SUBS = 4, SCAN_TILE = SCAN_SUBS * SCAN_SUB;                                     // 16384 elements per tile (long rows)
constexpr int SCAN_SUBS_SHORT = 2;  // 8192-element tiles for rows of at most SCAN_WINDOW such tiles: twice the CTAs per SM
constexpr int SCAN_WARPS = SCAN_THREADS / 32;
constexpr int SCAN_SMEM_BYTES = SCAN_TILE * 4 + 128;
constexpr int SCAN_WINDOW = 32;  // predecessors examined per round of the look-back (128 measured slower: 3.6 against 4.0 TB/s)
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
    long long tiles_per_row, total_tiles;
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
    // P = base + y[c] for the four elements of a group, base = carried value + offset of the group's warp in fp64:
    // base is split into an fp32 head and tail once per group; head + (tail + y) then costs two fp32 additions per
    // element and, beyond the final rounding of P, loses only the rounding of (tail + y)
    static __device__ __forceinline__ void finish4(double base, const float (&y)[4], float (&r)[4]) {
        const float head = static_cast<float>(base);
        const float tail = static_cast<float>(base - static_cast<double>(head));
#pragma unroll
        for (int c = 0; c < 4; ++c) r[c] = head + (tail + y[c]);
    }
};
template <> struct ScanCarry<int> {
    using type = unsigned int;
    static __device__ __forceinline__ unsigned long long pack(unsigned int v, unsigned long long state) {
        return (static_cast<unsigned long long>(v) << 32) | state;
    }
    static __device__ __forceinline__ unsigned int value(unsigned long long w) { return static_cast<unsigned int>(w >> 32); }
    static __device__ __forceinline__ void finish4(unsigned int base, const int (&y)[4], int (&r)[4]) {
#pragma unroll
        for (int c = 0; c < 4; ++c) r[c] = static_cast<int>(base + static_cast<unsigned int>(y[c]));
    }
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


// 16 KB from global to shared memory by one bulk copy that reports to an mbarrier (no multicast)
__device__ __forceinline__ void scan_bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(ptx::smem_u32(smem_dst)),
                 "l"(gmem_src), "r"(bytes), "r"(ptx::smem_u32(bar))
                 : "memory");
}

// ask L2 for 16 KB that a later tile will copy to shared memory (no destination, nobody waits for it)
__device__ __forceinline__ void scan_bulk_prefetch_l2(const void* gmem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(gmem_src), "r"(bytes) : "memory");
}

#ifndef CYC_SCAN_PREFETCH_TILES
#define CYC_SCAN_PREFETCH_TILES 256
#endif
// A tile also requests, into L2, the input of the tile that far ahead in the order tiles are handed out: about as many
// tiles as are resident at once, so that the copies of a tile that starts later find their data in L2 -- shorter and more
// even copy times, which is what the look-back of the successors waits for.  Measured: 4.0 -> 4.6 TB/s on one row of 2^28,
// 5.5 -> 6.3 TB/s on 4096 rows of 65536; 192 to 384 tiles ahead are alike, 64 less (4.5 / 6.0), 1024 worse than none.
constexpr long long SCAN_PREFETCH_TILES = CYC_SCAN_PREFETCH_TILES;

template <typename T, int SUBS>
__global__ void __launch_bounds__(SCAN_THREADS) scan_kernel(const ScanParams<T> p) {
    using Carry = typename ScanCarry<T>::type;
    using V4 = typename std::conditional<std::is_same<T, float>::value, float4, int4>::type;
    constexpr int ENTRIES = SUBS * SCAN_CHUNKS * SCAN_WARPS;  // warp-level sums of a tile, in element order
    extern __shared__ uint8_t scan_smem_raw[];
    T* buf = reinterpret_cast<T*>((reinterpret_cast<uintptr_t>(scan_smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    __shared__ uint64_t s_bar[SUBS];
    __shared__ unsigned int s_tile;
    __shared__ T s_total[ENTRIES];
    __shared__ Carry s_offset[ENTRIES];
    __shared__ Carry s_carry;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < SUBS; ++s) ptx::mbar_init(&s_bar[s], 1);
        ptx::fence_mbar_init();
        s_abort = 0;
        const unsigned int t = atomicAdd(&p.header->next_tile, 1u);
        s_tile = t;
        // quarters that lie completely inside the row come by bulk copy; a ragged or unaligned quarter is read by the threads
        if (p.vec_ok) {
            const long long row = t / p.tiles_per_row, tr = t - row * p.tiles_per_row;
            const long long base = tr * (SUBS * SCAN_SUB);
            const T* a = p.A + row * p.strideA + base;
#pragma unroll
            for (int s = 0; s < SUBS; ++s)
                if (base + (s + 1) * SCAN_SUB <= p.n) {
                    ptx::mbar_arrive_expect_tx(&s_bar[s], SCAN_SUB * sizeof(T));
                    scan_bulk_load(buf + s * SCAN_SUB, a + s * SCAN_SUB, SCAN_SUB * sizeof(T), &s_bar[s]);
                }
            const long long ahead = static_cast<long long>(t) + SCAN_PREFETCH_TILES;
            if (SCAN_PREFETCH_TILES > 0 && ahead < p.total_tiles) {
                const long long prow = ahead / p.tiles_per_row, ptr_ = ahead - prow * p.tiles_per_row;
                const long long pbase = ptr_ * (SUBS * SCAN_SUB);
                const T* pa = p.A + prow * p.strideA + pbase;
#pragma unroll
                for (int s = 0; s < SUBS; ++s)
                    if (pbase + (s + 1) * SCAN_SUB <= p.n) scan_bulk_prefetch_l2(pa + s * SCAN_SUB, SCAN_SUB * sizeof(T));
            }
        }
    }
    __syncthreads();
    const long long tile = s_tile;
    const long long row = tile / p.tiles_per_row, tr = tile - row * p.tiles_per_row;
    const long long base = tr * (SUBS * SCAN_SUB);
    const int len = static_cast<int>(min(static_cast<long long>((SUBS * SCAN_SUB)), p.n - base));
    const int subs = (len + SCAN_SUB - 1) / SCAN_SUB;
    const T* a = p.A + row * p.strideA + base;
    T* out = p.P + row * p.strideP + base;
    bool ok = true;

    // ---- quarter by quarter: running value inside each group of four, then across the lanes of the warp; the prefix
    // ---- relative to the start of the warp's 128 elements goes back to shared memory, the warp's sum to the table
    for (int s = 0; s < subs; ++s) {
        const bool bulk = p.vec_ok && (s + 1) * SCAN_SUB <= len;
        if (bulk && ok) {
            if (!ptx::mbar_try_wait(&s_bar[s], 0)) {
                const long long t0 = clock64();
                while (!ptx::mbar_try_wait(&s_bar[s], 0)) {
                    if (clock64() - t0 > SCAN_WAIT_CYCLES) {
                        atomicExch(&p.header->abort, 1);
                        atomicExch(p.status, 0x401);
                        s_abort = 1;
                        ok = false;
                        break;
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < SCAN_CHUNKS; ++j) {
            const int at = s * SCAN_SUB + (j * SCAN_THREADS + tid) * 4;
            T x[4];
            if (bulk) {
                const V4 v = *reinterpret_cast<const V4*>(buf + at);
                x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) x[c] = at + c < len ? __ldcs(a + at + c) : T(0);
            }
            x[1] = scan_add(x[0], x[1]);
            x[2] = scan_add(x[1], x[2]);
            x[3] = scan_add(x[2], x[3]);
            T w = x[3];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const T up = __shfl_up_sync(0xffffffffu, w, d);
                if (lane >= d) w = scan_add(up, w);
            }
            T before = __shfl_up_sync(0xffffffffu, w, 1);
            if (lane == 0) before = T(0);
            V4 y;
            y.x = scan_add(before, x[0]); y.y = scan_add(before, x[1]); y.z = scan_add(before, x[2]); y.w = scan_add(before, x[3]);
            *reinterpret_cast<V4*>(buf + at) = y;
            if (lane == 31) s_total[(s * SCAN_CHUNKS + j) * SCAN_WARPS + warp] = w;
        }
    }
    __syncthreads();

    // ---- warp 0: running value over the warp-level sums in element order, the tile's sum, and the look-back
    if (warp == 0) {
        constexpr int PER_LANE = ENTRIES / 32;
        const int used = subs * SCAN_CHUNKS * SCAN_WARPS;
        Carry run[PER_LANE];
        Carry mine = Carry(0);
#pragma unroll
        for (int e = 0; e < PER_LANE; ++e) {
            const int at = lane * PER_LANE + e;
            run[e] = mine;  // sum of this lane's entries before e
            if (at < used) mine += static_cast<Carry>(s_total[at]);
        }
        Carry w = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const Carry up = __shfl_up_sync(0xffffffffu, w, d);
            if (lane >= d) w += up;
        }
        Carry before = __shfl_up_sync(0xffffffffu, w, 1);
        if (lane == 0) before = Carry(0);
#pragma unroll
        for (int e = 0; e < PER_LANE; ++e) s_offset[lane * PER_LANE + e] = before + run[e];
        const Carry own = __shfl_sync(0xffffffffu, w, 31);

        Carry carry = Carry(0);
        bool wok = true;
        if (tr == 0) {
            if (lane == 0) scan_st_desc(&p.desc[tile], ScanCarry<T>::pack(own, SCAN_INCLUSIVE));
        } else {
            if (lane == 0) scan_st_desc(&p.desc[tile], ScanCarry<T>::pack(own, SCAN_PARTIAL));
            const long long first = tile - tr;  // first tile of this row
            long long pos = tile - 1;           // nearest predecessor not yet added
            const long long t0 = clock64();
            while (true) {
                // one round looks at the SCAN_WINDOW nearest predecessors not yet added, SCAN_WINDOW / 32 per lane (group e of a
                // lane is predecessor e * 32 + lane of the round); a slot past the start of the row behaves like a
                // finished tile with value zero, so the walk ends there
                unsigned long long word[SCAN_WINDOW / 32];
                unsigned int spins = 0;
                while (true) {
                    bool ready = true;
#pragma unroll
                    for (int e = 0; e < SCAN_WINDOW / 32; ++e) {
                        const long long idx = pos - (e * 32 + lane);
                        word[e] = idx >= first ? scan_ld_desc(&p.desc[idx]) : ScanCarry<T>::pack(Carry(0), SCAN_INCLUSIVE);
                    }
#pragma unroll
                    for (int e = 0; e < SCAN_WINDOW / 32; ++e) ready = ready && (word[e] & 3ull) != 0;
                    if (__all_sync(0xffffffffu, ready)) break;
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
                        if (__shfl_sync(0xffffffffu, give_up, 0)) { wok = false; break; }
                    }
                }
                if (!wok) break;
                bool found = false;
#pragma unroll
                for (int e = 0; e < SCAN_WINDOW / 32; ++e) {
                    if (found) continue;
                    const unsigned int done = __ballot_sync(0xffffffffu, (word[e] & 3ull) == SCAN_INCLUSIVE);
                    const int stop = done ? __ffs(done) - 1 : 32;  // nearest tile that knows its running value
                    Carry v = lane <= stop ? ScanCarry<T>::value(word[e]) : Carry(0);
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
                    carry += v;
                    found = done != 0;
                }
                if (found) break;
                pos -= SCAN_WINDOW;
            }
            if (wok && lane == 0) scan_st_desc(&p.desc[tile], ScanCarry<T>::pack(carry + own, SCAN_INCLUSIVE));
        }
        if (lane == 0) {
            s_carry = carry;
            if (!wok) s_abort = 1;
        }
    }
    __syncthreads();
    if (s_abort) {
        // leave no copy in flight: wait (bounded) for the quarters that were requested
        if (tid == 0 && p.vec_ok)
            for (int s = 0; s < SUBS; ++s)
                if (base + (s + 1) * SCAN_SUB <= p.n) {
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(&s_bar[s], 0) && clock64() - t0 < SCAN_WAIT_CYCLES) {}
                }
        return;
    }

    // ---- P_i = carried value + offset of the warp's 128 elements + prefix inside them
    const Carry carry = s_carry;
    for (int s = 0; s < subs; ++s) {
#pragma unroll
        for (int j = 0; j < SCAN_CHUNKS; ++j) {
            const int at = s * SCAN_SUB + (j * SCAN_THREADS + tid) * 4;
            const V4 v = *reinterpret_cast<const V4*>(buf + at);
            const T y[4] = {v.x, v.y, v.z, v.w};
            T r[4];
            ScanCarry<T>::finish4(carry + s_offset[(s * SCAN_CHUNKS + j) * SCAN_WARPS + warp], y, r);
            if (p.vec_ok && at + 4 <= len) {
                V4 o;
                o.x = r[0]; o.y = r[1]; o.z = r[2]; o.w = r[3];
                __stcs(reinterpret_cast<V4*>(out + at), o);
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (at + c < len) __stcs(out + at + c, r[c]);
            }
        }
    }
}

}  // namespace cyc
