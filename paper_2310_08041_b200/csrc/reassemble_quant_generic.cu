// Shape-agnostic kernels of the pre-GEMM stage: LayerNorm -> reassembly map ->
// per-token asymmetric quantization (Eq. 2-4 of QLLM), and the calibration
// statistic (per-channel max |LayerNorm(x)|).  One CTA walks whole token rows; the
// normalised row lives in shared memory and the CSR map is read through L2.  These
// kernels accept any C the boundary allows and serve shapes the specialised kernel
// does not cover.

#include <cuda_bf16.h>

#include "common.h"
#include "device_utils.cuh"
#include "reassemble_generic.cuh"

namespace qllm {

namespace {

constexpr int kThreads = 256;

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
    for (int64_t m = blockIdx.x; m < M; m += gridDim.x)
        quantize_token_row<XT>(x + m * C, m, C, gamma, beta, eps, ptr, src, coef, bits, codes, a_scale, a_zero, a_rowsum,
                               y, red);
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
