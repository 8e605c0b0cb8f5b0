// Build-time kernels on calibration data: the linear layer's input y = LayerNorm(x) in fp32, and the
// table of Eq. 5,
//     D(i, j) = || (x_i (W_i - W_j) + x_j (W_j - W_i)) / 2 ||_F^2 = 1/4 ||y_i - y_j||^2 ||W_i - W_j||^2,
// the output error of assembling channels i and j, which bipartite soft matching uses as its distance
// (Sec. 4.1.2; the paper names the pairwise distances as the main cost of reassembly).  The table
// decides an argmin, so its arithmetic is fixed: float32, rows taken in order with one fused
// multiply-add each (dx = fma(e, e, dx), e = y[t][i] - y[t][j]), D = (0.25f * dx) * dw.

#include <cuda_bf16.h>

#include <algorithm>

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

// ---- nearest channel of set B for every channel of set A (Appendix A step 2) ---------------------------------
// The bipartite matching needs, for every entry a of A, only argmin_b D(a, b) and that distance.  A CTA owns 32
// channels of A (a_idx) and walks a chunk of B (b_idx) 32 channels at a time with the table kernel's arithmetic;
// each thread keeps the best of its 4 rows over the tiles, a warp then reduces over its 32 columns.  Ties go
// to the lowest index in b_idx (the lists are in list-position order).  No table is written.
__device__ __forceinline__ void pair_sq_dist_cols(const float* __restrict__ a, int64_t rows, int C, const int* icol,
                                                  const int* jcol, float (&si)[32][33], float (&sj)[32][33],
                                                  float (&acc)[4]) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int ci = icol[tx], cj = jcol[tx];                // -1: past the end of the list
    for (int64_t r0 = 0; r0 < rows; r0 += 32) {
        __syncthreads();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int rr = ty + 8 * q;
            const bool in = r0 + rr < rows;
            si[rr][tx] = (in && ci >= 0) ? a[(r0 + rr) * C + ci] : 0.f;
            sj[rr][tx] = (in && cj >= 0) ? a[(r0 + rr) * C + cj] : 0.f;
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
eq5_nearest_partial_kernel(const float* __restrict__ y, int64_t T, const float* __restrict__ w, int N, int C,
                           const int* __restrict__ a_idx, int nA, const int* __restrict__ b_idx, int nB,
                           int tiles_per_chunk, float* __restrict__ pd, int* __restrict__ pi) {
    __shared__ float si[32][33], sj[32][33];
    __shared__ int icol[32], jcol[32];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int i0 = blockIdx.y * 32, chunk = blockIdx.x, nchunks = gridDim.x;
    if (threadIdx.x < 32) icol[threadIdx.x] = i0 + threadIdx.x < nA ? a_idx[i0 + threadIdx.x] : -1;
    float best[4] = {INFINITY, INFINITY, INFINITY, INFINITY};
    int bi[4] = {-1, -1, -1, -1};
    const int tile0 = chunk * tiles_per_chunk, tile1 = min((nB + 31) / 32, tile0 + tiles_per_chunk);
    for (int tile = tile0; tile < tile1; ++tile) {
        const int j0 = tile * 32;
        __syncthreads();
        if (threadIdx.x < 32) jcol[threadIdx.x] = j0 + threadIdx.x < nB ? b_idx[j0 + threadIdx.x] : -1;
        __syncthreads();
        float dx[4] = {0.f, 0.f, 0.f, 0.f}, dw[4] = {0.f, 0.f, 0.f, 0.f};
        pair_sq_dist_cols(y, T, C, icol, jcol, si, sj, dx);
        pair_sq_dist_cols(w, int64_t(N), C, icol, jcol, si, sj, dw);
        if (j0 + tx < nB) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float d = (0.25f * dx[k]) * dw[k];
                if (d < best[k]) { best[k] = d; bi[k] = j0 + tx; }     // tiles in ascending order: ties keep the first
            }
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        float d = best[k];
        int j = bi[k];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float d2 = __shfl_xor_sync(0xffffffffu, d, o);
            const int j2 = __shfl_xor_sync(0xffffffffu, j, o);
            if (j2 >= 0 && (j < 0 || d2 < d || (d2 == d && j2 < j))) { d = d2; j = j2; }
        }
        const int a = i0 + ty + 8 * k;
        if (tx == 0 && a < nA) { pd[size_t(a) * nchunks + chunk] = d; pi[size_t(a) * nchunks + chunk] = j; }
    }
}

__global__ void eq5_nearest_final_kernel(const float* __restrict__ pd, const int* __restrict__ pi, int nA, int nchunks,
                                         int* __restrict__ best, float* __restrict__ best_d) {
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= nA) return;
    float d = INFINITY;
    int j = -1;
    for (int c = 0; c < nchunks; ++c) {                    // chunks cover ascending indices: ties keep the first
        const int jc = pi[size_t(a) * nchunks + c];
        const float dc = pd[size_t(a) * nchunks + c];
        if (jc >= 0 && (j < 0 || dc < d)) { d = dc; j = jc; }
    }
    best[a] = j;
    best_d[a] = d;
}

}  // namespace

// For every a_idx[i] (source channel of an entry of A) the index into b_idx of its nearest channel under Eq. 5,
// and that distance.  y [T][C] and w [N][C] are device arrays, the index lists and results host arrays; the few
// small device buffers this needs are allocated and freed here (an offline build step).  best[i] = -1 when no
// distance of the row is a number below +inf.
int eq5_nearest_device(const float* y, int64_t T, const float* w, int N, int C, const int* a_idx, int nA,
                       const int* b_idx, int nB, int* best, float* best_d, cudaStream_t st) {
    if (nA <= 0 || nB <= 0) return QLLM_OK;
    const int tiles = (nB + 31) / 32;
    int nchunks = std::min(tiles, std::max(1, (4 * device_sm_count() + (nA + 31) / 32 - 1) / ((nA + 31) / 32)));
    const int tpc = (tiles + nchunks - 1) / nchunks;
    nchunks = (tiles + tpc - 1) / tpc;
    int *d_a = nullptr, *d_b = nullptr, *d_pi = nullptr, *d_best = nullptr;
    float *d_pd = nullptr, *d_bd = nullptr;
    auto release = [&]() { cudaFree(d_a); cudaFree(d_b); cudaFree(d_pi); cudaFree(d_best); cudaFree(d_pd); cudaFree(d_bd); };
    cudaError_t e = cudaMalloc(&d_a, sizeof(int) * nA);
    if (e == cudaSuccess) e = cudaMalloc(&d_b, sizeof(int) * nB);
    if (e == cudaSuccess) e = cudaMalloc(&d_pi, sizeof(int) * size_t(nA) * nchunks);
    if (e == cudaSuccess) e = cudaMalloc(&d_pd, sizeof(float) * size_t(nA) * nchunks);
    if (e == cudaSuccess) e = cudaMalloc(&d_best, sizeof(int) * nA);
    if (e == cudaSuccess) e = cudaMalloc(&d_bd, sizeof(float) * nA);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_a, a_idx, sizeof(int) * nA, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_b, b_idx, sizeof(int) * nB, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { release(); return cuda_fail(e); }
    eq5_nearest_partial_kernel<<<dim3(nchunks, (nA + 31) / 32), 256, 0, st>>>(y, T, w, N, C, d_a, nA, d_b, nB, tpc, d_pd, d_pi);
    eq5_nearest_final_kernel<<<(nA + 255) / 256, 256, 0, st>>>(d_pd, d_pi, nA, nchunks, d_best, d_bd);
    int rc = after_launch(2);
    if (rc == QLLM_OK) {
        e = cudaMemcpyAsync(best, d_best, sizeof(int) * nA, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(best_d, d_bd, sizeof(float) * nA, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) rc = cuda_fail(e);
    }
    release();
    return rc;
}

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
