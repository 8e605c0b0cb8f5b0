// Adaptive threshold search (Algorithm 1): for P thresholds theta_p = min(m) + p/P (max(m) - min(m)) build
// the reassembly, run the calibration tokens through the reassembled, quantized layer (the hot-path
// kernels) and keep the threshold with the smallest reassembly error
//     L(theta) = || LN(x) W^T  -  quant(X^) quant(W^) ||_F^2
// (Eq. 6, taken on the layer's own output).  An offline, host-orchestrated routine: it builds on the
// host, allocates, and waits for the device after every candidate.  The full-precision reference output
// is computed once with a plain fp32 GEMM; the error is summed in fp64.

#include <cuda_bf16.h>

#include <cmath>
#include <limits>
#include <vector>

#include "common.h"
#include "device_utils.cuh"

namespace qllm {

namespace {

// out[t][n] = sum_c y[t][c] * w[n][c]; 64 x 64 tiles, 16 channels per step, 4 x 4 outputs per thread.
__global__ void __launch_bounds__(256)
dense_ref_kernel(const float* __restrict__ y, const float* __restrict__ w, int T, int N, int C, float* __restrict__ out) {
    __shared__ float ys[16][65], ws[16][65];
    const int t0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4] = {};
    for (int c0 = 0; c0 < C; c0 += 16) {
        for (int i = threadIdx.x; i < 64 * 16; i += 256) {
            const int r = i >> 4, k = i & 15;
            ys[k][r] = (t0 + r < T && c0 + k < C) ? y[size_t(t0 + r) * C + c0 + k] : 0.f;
            ws[k][r] = (n0 + r < N && c0 + k < C) ? w[size_t(n0 + r) * C + c0 + k] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = ys[k][ty * 4 + i]; b[i] = ws[k][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t = t0 + ty * 4 + i, n = n0 + tx * 4 + j;
            if (t < T && n < N) out[size_t(t) * N + n] = acc[i][j];
        }
}

// *total += sum (a - b)^2, accumulated in fp64
__global__ void __launch_bounds__(256)
sqerr_kernel(const float* __restrict__ a, const float* __restrict__ b, int64_t n, double* __restrict__ total) {
    __shared__ double red[8];
    double s = 0.0;
    for (int64_t i = int64_t(blockIdx.x) * 256 + threadIdx.x; i < n; i += int64_t(gridDim.x) * 256) {
        const double d = double(a[i]) - double(b[i]);
        s += d * d;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        atomicAdd(total, t);
    }
}

struct DevBuf {
    void* p = nullptr;
    ~DevBuf() { if (p) cudaFree(p); }
    int alloc(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 1) == cudaSuccess ? QLLM_OK : cuda_fail(cudaGetLastError()); }
};

}  // namespace

}  // namespace qllm

using namespace qllm;

extern "C" int qllm_search_theta(const void* calib_x, int x_dtype, int64_t T, int C, const float* ln_gamma,
                                 const float* ln_beta, float ln_eps, const float* calib_absmax, const float* W,
                                 int N, int a_bits, int w_bits, int P, float* theta_out, double* losses_out,
                                 void* stream) {
    if (!calib_x || !ln_gamma || !calib_absmax || !W || !theta_out) return QLLM_ERR_NULL;
    if (!bits_ok(a_bits) || !bits_ok(w_bits)) return QLLM_ERR_BITS;
    if (!dtype_ok(x_dtype)) return QLLM_ERR_DTYPE;
    if (T <= 0 || C <= 0 || N <= 0 || P <= 0 || T > (int64_t(1) << 24)) return QLLM_ERR_SHAPE;
    if (!aligned16(calib_x)) return QLLM_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // full-precision reference output of the calibration tokens, once
    DevBuf d_gamma, d_beta, d_w, d_y, d_ref, d_out, d_loss;
    int rc = d_gamma.alloc(size_t(C) * 4);
    if (rc == QLLM_OK && ln_beta) rc = d_beta.alloc(size_t(C) * 4);
    if (rc == QLLM_OK) rc = d_w.alloc(size_t(N) * C * 4);
    if (rc == QLLM_OK) rc = d_y.alloc(size_t(T) * C * 4);
    if (rc == QLLM_OK) rc = d_ref.alloc(size_t(T) * N * 4);
    if (rc == QLLM_OK) rc = d_out.alloc(size_t(T) * N * 4);
    if (rc == QLLM_OK) rc = d_loss.alloc(sizeof(double));
    if (rc != QLLM_OK) return rc;
    QLLM_CUDA_TRY(cudaMemcpyAsync(d_gamma.p, ln_gamma, size_t(C) * 4, cudaMemcpyHostToDevice, st));
    if (ln_beta) QLLM_CUDA_TRY(cudaMemcpyAsync(d_beta.p, ln_beta, size_t(C) * 4, cudaMemcpyHostToDevice, st));
    QLLM_CUDA_TRY(cudaMemcpyAsync(d_w.p, W, size_t(N) * C * 4, cudaMemcpyHostToDevice, st));
    rc = launch_layernorm_rows(calib_x, x_dtype, T, C, static_cast<const float*>(d_gamma.p),
                               static_cast<const float*>(d_beta.p), ln_eps, static_cast<float*>(d_y.p), st);
    if (rc != QLLM_OK) return rc;
    dense_ref_kernel<<<dim3(unsigned((N + 63) / 64), unsigned((T + 63) / 64)), 256, 0, st>>>(
        static_cast<const float*>(d_y.p), static_cast<const float*>(d_w.p), int(T), N, C, static_cast<float*>(d_ref.p));
    rc = after_launch();
    if (rc != QLLM_OK) return rc;

    float lo = calib_absmax[0], hi = calib_absmax[0];
    for (int c = 1; c < C; ++c) { lo = std::fmin(lo, calib_absmax[c]); hi = std::fmax(hi, calib_absmax[c]); }
    double best = std::numeric_limits<double>::infinity();
    float best_theta = hi;
    for (int p = 1; p <= P; ++p) {
        const float theta = float(double(lo) + (double(p) / double(P)) * (double(hi) - double(lo)));
        double loss = std::numeric_limits<double>::infinity();
        qllm_reassembly_t* h = nullptr;
        rc = theta > 0.f ? qllm_build_reassembly(calib_absmax, C, theta, W, N, nullptr, nullptr, 0, w_bits, &h)
                         : QLLM_ERR_INFEASIBLE;
        if (rc == QLLM_OK) {
            qllm_layer_t* layer = nullptr;
            rc = qllm_layer_create(h, ln_gamma, ln_beta, ln_eps, nullptr, a_bits, x_dtype, QLLM_F32, T, &layer);
            if (rc == QLLM_OK) rc = qllm_layer_forward(layer, calib_x, T, d_out.p, stream);
            if (rc == QLLM_OK && cudaMemsetAsync(d_loss.p, 0, sizeof(double), st) != cudaSuccess) rc = QLLM_ERR_CUDA;
            if (rc == QLLM_OK) {
                sqerr_kernel<<<device_sm_count() * 4, 256, 0, st>>>(static_cast<const float*>(d_out.p),
                                                                   static_cast<const float*>(d_ref.p), int64_t(T) * N,
                                                                   static_cast<double*>(d_loss.p));
                rc = after_launch();
            }
            if (rc == QLLM_OK &&
                (cudaMemcpyAsync(&loss, d_loss.p, sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
                 cudaStreamSynchronize(st) != cudaSuccess))
                rc = cuda_fail(cudaGetLastError());
            else if (rc != QLLM_OK)
                cudaStreamSynchronize(st);               // nothing of this candidate may outlive its buffers
            if (layer) qllm_layer_destroy(layer);
            qllm_free_reassembly(h);
            if (rc != QLLM_OK) return rc;
        } else if (rc != QLLM_ERR_INFEASIBLE) {
            return rc;                                   // a threshold that cannot restore C channels is skipped
        }
        if (losses_out) losses_out[p - 1] = loss;
        if (loss < best) { best = loss; best_theta = theta; }
    }
    *theta_out = best_theta;
    return QLLM_OK;
}
