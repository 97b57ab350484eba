// Shared device/host helpers of the LinSimp kernels (no arithmetic of the method here).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace linsimp {

typedef __nv_bfloat16 bf16;

template <typename T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ldf<bf16>(const bf16 *p) { return __bfloat162float(*p); }

template <typename T> __device__ __forceinline__ void stf(T *p, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<bf16>(bf16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Workspace layout helpers shared by the host API and the kernels' launchers.
struct Shape {
    int B, H, T, d, m, W;
    int C;        // chunk length in tokens
    int NC;       // number of chunks = ceil(T / C)
    long E;       // floats per boundary state: m*d (state) + m (normaliser)
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Streaming multiprocessors of the current device (launch heuristics size their grids by it); 148 if the query fails.
inline int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 148;
    return n;
}

}  // namespace linsimp
