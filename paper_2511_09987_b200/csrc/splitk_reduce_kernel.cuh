// Second step of the split-K schedule: the k loop of each tile was cut into S slices whose
// partial sums sit in S consecutive planes of a workspace; C_ij is their sum taken in
// increasing slice (= increasing k) order, so the result does not depend on timing.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "ptx.cuh"

namespace cyc {

// ws: [batch][S][plane] ; C: [batch] planes with stride sC ; plane = M*N elements.
// C may be plane 0 of ws (the sum taken in place): every thread reads the S values of its own index before it writes
// that index and touches no other, so the pointers carry no no-alias promise.
template <typename T>
__global__ void __launch_bounds__(128) splitk_reduce_kernel(const T* ws, T* C, long long plane, long long sC, int S,
                                                            long long batch, int vec4) {
    // launched with programmatic stream serialisation: only the launch itself overlaps the previous kernel
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const long long per_batch = vec4 ? plane / 4 : plane;
    const long long total = per_batch * batch;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long b = i / per_batch, r = i - b * per_batch;
        const T* src = ws + b * S * plane;
        if (vec4) {
            using V = typename std::conditional<sizeof(T) == 4 && std::is_floating_point<T>::value, float4, int4>::type;
            V acc = reinterpret_cast<const V*>(src)[r];
            int s = 1;
            for (; s + 8 <= S; s += 8) {  // eight loads in flight, added in slice order
                V v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = reinterpret_cast<const V*>(src + static_cast<long long>(s + u) * plane)[r];
#pragma unroll
                for (int u = 0; u < 8; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
            }
            for (; s < S; ++s) {
                const V v = reinterpret_cast<const V*>(src + static_cast<long long>(s) * plane)[r];
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
            reinterpret_cast<V*>(C + b * sC)[r] = acc;
        } else {
            T acc = src[r];
            for (int s = 1; s < S; ++s) acc += src[static_cast<long long>(s) * plane + r];
            C[b * sC + r] = acc;
        }
    }
}

}  // namespace cyc
