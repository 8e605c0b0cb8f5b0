// Small device-side helpers shared by the kernels: warp / CTA reductions.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace qllm {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum_int(int v) { return __reduce_add_sync(0xffffffffu, v); }
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// CTA-wide sum; `red` holds at least 32 floats.  Every thread returns the total.
// blockDim.x must be a multiple of 32.  Safe to call back to back with the same `red`.
__device__ __forceinline__ float block_sum(float v, float* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    v = warp_sum(v);
    __syncthreads();                 // previous users of `red` are done
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = lane < nw ? red[lane] : 0.f;
    return warp_sum(t);
}
__device__ __forceinline__ int block_sum_int(int v, int* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    v = warp_sum_int(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    int t = lane < nw ? red[lane] : 0;
    return warp_sum_int(t);
}
// CTA-wide min and max in one pass; `red` holds at least 64 floats.
__device__ __forceinline__ void block_minmax(float& lo, float& hi, float* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    lo = warp_min(lo);
    hi = warp_max(hi);
    __syncthreads();
    if (lane == 0) { red[warp] = lo; red[32 + warp] = hi; }
    __syncthreads();
    float a = lane < nw ? red[lane] : INFINITY;
    float b = lane < nw ? red[32 + lane] : -INFINITY;
    lo = warp_min(a);
    hi = warp_max(b);
}

}  // namespace qllm
