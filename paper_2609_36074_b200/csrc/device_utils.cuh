// Small device helpers: fixed-order warp and block sums.
#pragma once
#include <cuda_runtime.h>

namespace gemnlr {

// Butterfly sum: every lane ends with the same bits (a + b == b + a at every level).
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over a block of NT threads; warp totals are added in warp order, every thread returns
// the same value.  sred must hold NT/32 doubles; safe to call repeatedly with the same buffer.
template <int NT>
__device__ __forceinline__ double block_sum(double v, double* sred)
{
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sred[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < NT / 32; ++w) t += sred[w];
    return t;
}

}  // namespace gemnlr
