// Shape-agnostic kernels of the pre-GEMM stage: LayerNorm -> reassembly map ->
// per-token asymmetric quantization (Eq. 2-4 of QLLM), and the calibration
// statistic (per-channel max |LayerNorm(x)|).  One CTA walks whole token rows; the
// normalised row lives in shared memory and the CSR map is read through L2.  These
// kernels accept any C the boundary allows and serve shapes the specialised kernel
// does not cover.

#include <cuda_bf16.h>

#include "common.h"
#include "device_utils.cuh"

namespace qllm {

namespace {

constexpr int kThreads = 256;

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

template <typename XT>
__global__ void __launch_bounds__(kThreads)
reassemble_quant_generic(const XT* __restrict__ x, int64_t M, int C, const float* __restrict__ gamma,
                         const float* __restrict__ beta, float eps, const int32_t* __restrict__ ptr,
                         const int32_t* __restrict__ src, const float* __restrict__ coef, int bits,
                         uint8_t* __restrict__ codes, float* __restrict__ a_scale,
                         float* __restrict__ a_zero, int32_t* __restrict__ a_rowsum,
                         const int* __restrict__ skip_if_nonzero) {
    extern __shared__ float y[];
    __shared__ float red[2 * 32];
    // launched behind a specialised kernel that may have served the call already (it says so in this word)
    if (skip_if_nonzero && *skip_if_nonzero != 0) return;
    const float qmax = float((1 << bits) - 1);
    for (int64_t m = blockIdx.x; m < M; m += gridDim.x) {
        layernorm_row<XT>(x + m * C, C, gamma, beta, eps, y, red);
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
}

// Per-channel running maximum of |LayerNorm(x)| over the rows this CTA walks, merged into
// absmax with one atomic per channel (non-negative floats order like their bit patterns).
template <typename XT>
__global__ void __launch_bounds__(kThreads)
calib_absmax_kernel(const XT* __restrict__ x, int64_t M, int C, const float* __restrict__ gamma,
                    const float* __restrict__ beta, float eps, float* __restrict__ absmax) {
    extern __shared__ float smem[];
    float* y = smem;
    float* amax = smem + C;
    __shared__ float red[2 * 32];
    for (int k = threadIdx.x; k < C; k += blockDim.x) amax[k] = 0.f;
    for (int64_t m = blockIdx.x; m < M; m += gridDim.x) {
        layernorm_row<XT>(x + m * C, C, gamma, beta, eps, y, red);
        for (int k = threadIdx.x; k < C; k += blockDim.x) amax[k] = fmaxf(amax[k], fabsf(y[k]));
        __syncthreads();
    }
    for (int k = threadIdx.x; k < C; k += blockDim.x)
        atomicMax(reinterpret_cast<int*>(absmax + k), __float_as_int(amax[k]));
}

}  // namespace

int launch_reassemble_quant_generic(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                                    const float* beta, float eps, const int32_t* ptr,
                                    const int32_t* src, const float* coef, int bits, uint8_t* codes,
                                    float* a_scale, float* a_zero, int32_t* a_rowsum, cudaStream_t st,
                                    const int* skip_if_nonzero) {
    const size_t smem = size_t(C) * sizeof(float);
    if (smem > 200 * 1024) return QLLM_ERR_UNSUPPORTED;
    const int grid = int(std::min<int64_t>(M, int64_t(device_sm_count()) * 4));
    if (x_dtype == QLLM_F32) {
        auto k = reassemble_quant_generic<float>;
        if (smem > 48 * 1024) QLLM_CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
        k<<<grid, kThreads, smem, st>>>(static_cast<const float*>(x), M, C, gamma, beta, eps, ptr, src,
                                        coef, bits, codes, a_scale, a_zero, a_rowsum, skip_if_nonzero);
    } else {
        auto k = reassemble_quant_generic<__nv_bfloat16>;
        if (smem > 48 * 1024) QLLM_CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
        k<<<grid, kThreads, smem, st>>>(static_cast<const __nv_bfloat16*>(x), M, C, gamma, beta, eps,
                                        ptr, src, coef, bits, codes, a_scale, a_zero, a_rowsum, skip_if_nonzero);
    }
    return after_launch();
}

int launch_calib_absmax(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                        const float* beta, float eps, float* absmax, cudaStream_t st) {
    const size_t smem = 2 * size_t(C) * sizeof(float);
    if (smem > 200 * 1024) return QLLM_ERR_UNSUPPORTED;
    const int grid = int(std::min<int64_t>(M, int64_t(device_sm_count())));
    if (x_dtype == QLLM_F32) {
        auto k = calib_absmax_kernel<float>;
        if (smem > 48 * 1024) QLLM_CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
        k<<<grid, kThreads, smem, st>>>(static_cast<const float*>(x), M, C, gamma, beta, eps, absmax);
    } else {
        auto k = calib_absmax_kernel<__nv_bfloat16>;
        if (smem > 48 * 1024) QLLM_CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
        k<<<grid, kThreads, smem, st>>>(static_cast<const __nv_bfloat16*>(x), M, C, gamma, beta, eps, absmax);
    }
    return after_launch();
}

}  // namespace qllm
