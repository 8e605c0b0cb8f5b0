// One token row through LayerNorm -> reassembly map -> per-token quantization (QLLM Eq. 2-4) by a whole CTA,
// for any channel count: the normalised row lives in shared memory and the CSR map is read through L2.  Used
// by the shape-agnostic kernel and by the fused decode step (where a CTA quantizes one token before it
// starts multiplying).
#pragma once

#include <cuda_bf16.h>

#include "device_utils.cuh"

namespace qllm {

template <typename XT>
__device__ __forceinline__ float load_as_float(const XT* p, int64_t i);
template <>
__device__ __forceinline__ float load_as_float<float>(const float* p, int64_t i) { return p[i]; }
template <>
__device__ __forceinline__ float load_as_float<__nv_bfloat16>(const __nv_bfloat16* p, int64_t i) {
    return __bfloat162float(p[i]);
}

// LayerNorm of one row into shared memory y[0..C).  All threads of the CTA take part.
// gamma == nullptr: no normalisation, the row is copied as it is (the caller's input already is the
// linear layer's input, Appendix B).
template <typename XT>
__device__ void layernorm_row(const XT* __restrict__ xrow, int C, const float* __restrict__ gamma,
                              const float* __restrict__ beta, float eps, float* y, float* red) {
    if (!gamma) {
        for (int k = threadIdx.x; k < C; k += blockDim.x) y[k] = load_as_float<XT>(xrow, k);
        __syncthreads();
        return;
    }
    float s = 0.f;
    for (int k = threadIdx.x; k < C; k += blockDim.x) {
        float v = load_as_float<XT>(xrow, k);
        y[k] = v;
        s += v;
    }
    const float mean = block_sum(s, red) / float(C);
    float q = 0.f;
    for (int k = threadIdx.x; k < C; k += blockDim.x) {
        float d = y[k] - mean;
        q = fmaf(d, d, q);
    }
    const float var = block_sum(q, red) / float(C);
    const float rstd = 1.0f / sqrtf(var + eps);
    for (int k = threadIdx.x; k < C; k += blockDim.x) {
        float d = (y[k] - mean) * rstd;
        y[k] = fmaf(d, gamma[k], beta ? beta[k] : 0.f);
    }
    __syncthreads();
}

__device__ __forceinline__ float map_row(const float* y, const int32_t* __restrict__ ptr,
                                         const int32_t* __restrict__ src,
                                         const float* __restrict__ coef, int c) {
    int j = ptr[c];
    const int e = ptr[c + 1];
    float v = coef[j] * y[src[j]];
    for (++j; j < e; ++j) v = fmaf(coef[j], y[src[j]], v);
    return v;
}

// Token row m: x row -> codes (4-bit: two per byte), scale, zero, code sum.  y: C floats of shared memory,
// red: 64 floats.  All threads of the CTA take part; ends with the CTA synchronised.
template <typename XT>
__device__ void quantize_token_row(const XT* __restrict__ xrow, int64_t m, int C, const float* __restrict__ gamma,
                                   const float* __restrict__ beta, float eps, const int32_t* __restrict__ ptr,
                                   const int32_t* __restrict__ src, const float* __restrict__ coef, int bits,
                                   uint8_t* __restrict__ codes, float* __restrict__ a_scale,
                                   float* __restrict__ a_zero, int32_t* __restrict__ a_rowsum, float* y, float* red) {
    const float qmax = float((1 << bits) - 1);
    layernorm_row<XT>(xrow, C, gamma, beta, eps, y, red);
    float lo = INFINITY, hi = -INFINITY;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        float v = map_row(y, ptr, src, coef, c);
        lo = fminf(lo, v);
        hi = fmaxf(hi, v);
    }
    block_minmax(lo, hi, red);
    float alpha = (hi - lo) / qmax;
    if (!(hi > lo)) alpha = lo != 0.f ? fabsf(lo) : 1.f;
    const float zero = -rintf(lo / alpha);
    int sum = 0;
    if (bits == 4) {
        uint8_t* out = codes + m * (C / 2);
        for (int p = threadIdx.x; p < C / 2; p += blockDim.x) {
            float v0 = map_row(y, ptr, src, coef, 2 * p);
            float v1 = map_row(y, ptr, src, coef, 2 * p + 1);
            int q0 = int(fminf(fmaxf(rintf(v0 / alpha) + zero, 0.f), qmax));
            int q1 = int(fminf(fmaxf(rintf(v1 / alpha) + zero, 0.f), qmax));
            out[p] = uint8_t(q0 | (q1 << 4));
            sum += q0 + q1;
        }
    } else {
        uint8_t* out = codes + m * C;
        for (int c = threadIdx.x; c < C; c += blockDim.x) {
            float v = map_row(y, ptr, src, coef, c);
            int q = int(fminf(fmaxf(rintf(v / alpha) + zero, 0.f), qmax));
            out[c] = uint8_t(q);
            sum += q;
        }
    }
    const int total = block_sum_int(sum, reinterpret_cast<int*>(red));
    if (threadIdx.x == 0) {
        a_scale[m] = alpha;
        a_zero[m] = zero;
        if (a_rowsum) a_rowsum[m] = total;
    }
    __syncthreads();   // y is rewritten by the next row
}

}  // namespace qllm
