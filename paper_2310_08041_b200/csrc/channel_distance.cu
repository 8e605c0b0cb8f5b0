// Build-time kernels on calibration data: the linear layer's input y = LayerNorm(x) in fp32, and the
// table of Eq. 5,
//     D(i, j) = || (x_i (W_i - W_j) + x_j (W_j - W_i)) / 2 ||_F^2 = 1/4 ||y_i - y_j||^2 ||W_i - W_j||^2,
// the output error of assembling channels i and j, which bipartite soft matching uses as its distance
// (Sec. 4.1.2; the paper names the pairwise distances as the main cost of reassembly).  The table
// decides an argmin, so its arithmetic is fixed: float32, rows taken in order with one fused
// multiply-add each (dx = fma(e, e, dx), e = y[t][i] - y[t][j]), D = (0.25f * dx) * dw.

#include <cuda_bf16.h>

#include "common.h"
#include "device_utils.cuh"

namespace qllm {

namespace {

template <typename XT>
__global__ void __launch_bounds__(256)
layernorm_rows_kernel(const XT* __restrict__ x, int C, const float* __restrict__ gamma, const float* __restrict__ beta,
                      float eps, float* __restrict__ y) {
    __shared__ float red[32];
    const XT* xr = x + size_t(blockIdx.x) * C;
    float* yr = y + size_t(blockIdx.x) * C;
    float s = 0.f;
    for (int c = threadIdx.x; c < C; c += blockDim.x) s += float(xr[c]);
    const float mean = block_sum(s, red) / float(C);
    float sq = 0.f;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const float d = float(xr[c]) - mean;
        sq = fmaf(d, d, sq);
    }
    const float rstd = rsqrtf(block_sum(sq, red) / float(C) + eps);
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const float v = (float(xr[c]) - mean) * rstd * gamma[c];
        yr[c] = beta ? v + beta[c] : v;
    }
}

// One 32 x 32 tile of channel pairs per CTA; a thread owns 4 pairs (i = i0 + ty + 8k, j = j0 + tx) and walks
// the rows of `a` ([rows][C]) in order, 32 at a time through shared memory.  Rows past the end are staged as
// zeros: fma(0, 0, acc) leaves acc unchanged, so the result is that of the exact row count.
__device__ __forceinline__ void pair_sq_dist(const float* __restrict__ a, int64_t rows, int C, int i0, int j0,
                                             float (&si)[32][33], float (&sj)[32][33], float (&acc)[4]) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int64_t r0 = 0; r0 < rows; r0 += 32) {
        __syncthreads();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int rr = ty + 8 * q;
            const bool in = r0 + rr < rows;
            si[rr][tx] = (in && i0 + tx < C) ? a[(r0 + rr) * C + i0 + tx] : 0.f;
            sj[rr][tx] = (in && j0 + tx < C) ? a[(r0 + rr) * C + j0 + tx] : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int rr = 0; rr < 32; ++rr) {
            const float bj = sj[rr][tx];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float e = si[rr][ty + 8 * k] - bj;
                acc[k] = fmaf(e, e, acc[k]);
            }
        }
    }
}

__global__ void __launch_bounds__(256)
channel_distance_kernel(const float* __restrict__ y, int64_t T, const float* __restrict__ w, int N, int C,
                        float* __restrict__ D) {
    __shared__ float si[32][33], sj[32][33];
    const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    float dx[4] = {0.f, 0.f, 0.f, 0.f}, dw[4] = {0.f, 0.f, 0.f, 0.f};
    pair_sq_dist(y, T, C, i0, j0, si, sj, dx);
    pair_sq_dist(w, int64_t(N), C, i0, j0, si, sj, dw);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int i = i0 + ty + 8 * k, j = j0 + tx;
        if (i < C && j < C) D[size_t(i) * C + j] = (0.25f * dx[k]) * dw[k];
    }
}

}  // namespace

int launch_layernorm_rows(const void* x, int x_dtype, int64_t T, int C, const float* gamma, const float* beta,
                          float eps, float* y, cudaStream_t st) {
    if (T == 0) return QLLM_OK;
    if (x_dtype == QLLM_BF16)
        layernorm_rows_kernel<__nv_bfloat16><<<unsigned(T), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), C,
                                                                         gamma, beta, eps, y);
    else
        layernorm_rows_kernel<float><<<unsigned(T), 256, 0, st>>>(static_cast<const float*>(x), C, gamma, beta, eps, y);
    return after_launch();
}

}  // namespace qllm

using namespace qllm;

extern "C" int qllm_layernorm_rows(const void* x, int x_dtype, int64_t T, int C, const float* ln_gamma,
                                   const float* ln_beta, float ln_eps, float* y, void* stream) {
    if (!dtype_ok(x_dtype)) return QLLM_ERR_DTYPE;
    if (T < 0 || C <= 0 || T > (int64_t(1) << 30)) return QLLM_ERR_SHAPE;
    if (T == 0) return QLLM_OK;
    if (!x || !ln_gamma || !y) return QLLM_ERR_NULL;
    return launch_layernorm_rows(x, x_dtype, T, C, ln_gamma, ln_beta, ln_eps, y, static_cast<cudaStream_t>(stream));
}

extern "C" int qllm_channel_distance(const float* y, int64_t T, const float* W, int N, int C, float* D, void* stream) {
    if (T <= 0 || N <= 0 || C <= 0 || C > 65535 * 32) return QLLM_ERR_SHAPE;
    if (!y || !W || !D) return QLLM_ERR_NULL;
    const unsigned g = unsigned((C + 31) / 32);
    channel_distance_kernel<<<dim3(g, g), 256, 0, static_cast<cudaStream_t>(stream)>>>(y, T, W, N, C, D);
    return after_launch();
}
