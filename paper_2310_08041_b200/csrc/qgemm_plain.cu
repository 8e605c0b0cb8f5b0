// Shape-agnostic integer GEMM with the dequantizing epilogue, and the row code-sum
// pre-pass.  One thread per output element, operands read code by code: this is the
// path for shapes the tensor-core and weight-streaming kernels do not take (odd K,
// unaligned rows) and the on-device cross-check of those kernels.

#include "common.h"
#include "epilogue.cuh"

namespace qllm {

namespace {

__device__ __forceinline__ int code_at(const uint8_t* row, int k, int bits) {
    if (bits == 4) {
        const int b = row[k >> 1];
        return (k & 1) ? (b >> 4) : (b & 0xF);
    }
    return row[k];
}

// Eight consecutive codes starting at k (k % 8 == 0) as two words of four byte lanes:
// lanes of `even` = codes k, k+2, k+4, k+6; lanes of `odd` = codes k+1, k+3, k+5, k+7.
// Both operands use the same order, so the dot product is unchanged.
__device__ __forceinline__ void eight_codes(const uint8_t* row, int k, int bits, uint32_t& even, uint32_t& odd) {
    if (bits == 4) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(row + (k >> 1));
        even = w & 0x0F0F0F0Fu;
        odd = (w >> 4) & 0x0F0F0F0Fu;
    } else {
        const uint2 w = *reinterpret_cast<const uint2*>(row + k);
        even = __byte_perm(w.x, w.y, 0x6420);
        odd = __byte_perm(w.x, w.y, 0x7531);
    }
}

template <bool WORDS>
__global__ void __launch_bounds__(256)
qgemm_plain_kernel(const uint8_t* __restrict__ a, const uint8_t* __restrict__ w, int64_t M, int N, int K,
                   int a_bits, int w_bits, EpilogueArgs ep) {
    const int n = blockIdx.x * 32 + (threadIdx.x & 31);
    const int64_t m = int64_t(blockIdx.y) * 8 + (threadIdx.x >> 5);
    if (n >= N || m >= M) return;
    const uint8_t* arow = a + m * (a_bits == 4 ? K / 2 : K);
    const uint8_t* wrow = w + int64_t(n) * (w_bits == 4 ? K / 2 : K);
    int acc = 0;
    if (WORDS) {
        for (int k = 0; k < K; k += 8) {
            uint32_t ae, ao, we, wo;
            eight_codes(arow, k, a_bits, ae, ao);
            eight_codes(wrow, k, w_bits, we, wo);
            acc = int(__dp4a(ae, we, uint32_t(acc)));      // unsigned lanes
            acc = int(__dp4a(ao, wo, uint32_t(acc)));
        }
    } else {
        for (int k = 0; k < K; ++k) acc += code_at(arow, k, a_bits) * code_at(wrow, k, w_bits);
    }
    if (ep.raw_acc) {
        static_cast<int32_t*>(ep.out)[m * N + n] = acc;
        return;
    }
    const RowTerm r = make_row_term(ep.a_scale, ep.a_zero, ep.a_rowsum, m);
    const ColTerm c = make_col_term(ep.w_scale, ep.w_zero, ep.w_colsum, ep.bias, K, n);
    const float o = dequant(acc, r, c);
    if (ep.out_dtype == QLLM_F32) static_cast<float*>(ep.out)[m * N + n] = o;
    else static_cast<__nv_bfloat16*>(ep.out)[m * N + n] = __float2bfloat16_rn(o);
}

// One warp per row: sum of the row's codes.
__global__ void __launch_bounds__(256)
rowsum_kernel(const uint8_t* __restrict__ codes, int64_t M, int K, int bits, int32_t* __restrict__ rowsum) {
    const int64_t m = int64_t(blockIdx.x) * 8 + (threadIdx.x >> 5);
    if (m >= M) return;
    const int lane = threadIdx.x & 31;
    const int nbytes = bits == 4 ? K / 2 : K;
    const uint8_t* row = codes + m * nbytes;
    int s = 0;
    for (int i = lane; i < nbytes; i += 32) {
        const int b = row[i];
        s += bits == 4 ? (b & 0xF) + (b >> 4) : b;
    }
    s = __reduce_add_sync(0xffffffffu, s);
    if (lane == 0) rowsum[m] = s;
}

// Packed nibbles [rows][K/2] -> byte codes [rows][K] in natural K order.  A 16-byte chunk (32 codes) becomes 32
// contiguous bytes; purely bandwidth-bound.  The kernel often runs beside a kernel that leaves it few warps per
// SM, so a thread keeps kExpandUnroll loads in flight, and a lane pair swaps halves so that every store instruction
// of a warp writes whole 32-byte sectors instead of half of each.
constexpr int kExpandUnroll = 4;
__device__ __forceinline__ void expand_chunk(const uint4& w, uint32_t (&o)[8]) {
    const uint32_t in[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t lo = in[k] & 0x0F0F0F0Fu, hi = (in[k] >> 4) & 0x0F0F0F0Fu;
        o[2 * k] = __byte_perm(lo, hi, 0x5140);
        o[2 * k + 1] = __byte_perm(lo, hi, 0x7362);
    }
}
__global__ void __launch_bounds__(256)
expand_codes_kernel(const uint4* __restrict__ packed, int64_t chunks, uint4* __restrict__ bytes) {
    const int lane = threadIdx.x & 31;
    const bool odd = lane & 1;
    const int64_t step = int64_t(gridDim.x) * 256;
    // whole warps stay in the loop (the exchange below needs both lanes of a pair); chunks beyond the end are
    // loaded as zeros and not stored
    const int64_t first = int64_t(blockIdx.x) * 256 + (threadIdx.x & ~31);
    for (int64_t i0 = first; i0 < chunks; i0 += step * kExpandUnroll) {
        uint4 w[kExpandUnroll];
#pragma unroll
        for (int u = 0; u < kExpandUnroll; ++u) {
            const int64_t i = i0 + u * step + lane;
            w[u] = i < chunks ? __ldcs(packed + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kExpandUnroll; ++u) {
            const int64_t i = i0 + u * step + lane;
            uint32_t o[8];
            expand_chunk(w[u], o);
            // even lane: keeps its first half, takes the odd lane's first half; odd lane: takes the even lane's
            // second half, keeps its own second half.  Store 1 then covers the even lane's chunk, store 2 the odd's.
            uint32_t a[4], b[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t got = __shfl_xor_sync(0xffffffffu, odd ? o[k] : o[4 + k], 1);
                a[k] = odd ? got : o[k];                     // 16 bytes of the even lane's chunk
                b[k] = odd ? o[4 + k] : got;                 // 16 bytes of the odd lane's chunk
            }
            const int64_t ie = i & ~int64_t(1);              // the pair's even chunk
            if (ie < chunks) bytes[2 * ie + (odd ? 1 : 0)] = make_uint4(a[0], a[1], a[2], a[3]);
            if (ie + 1 < chunks) bytes[2 * ie + 2 + (odd ? 1 : 0)] = make_uint4(b[0], b[1], b[2], b[3]);
        }
    }
}

}  // namespace

int launch_expand_codes(const uint8_t* packed, int64_t rows, int K, uint8_t* bytes, cudaStream_t st) {
    const int64_t chunks = rows * (K / 32);
    if (chunks == 0) return QLLM_OK;
    const int64_t per_cta = 256 * kExpandUnroll;
    const int grid = int(std::min<int64_t>((chunks + per_cta - 1) / per_cta, int64_t(device_sm_count()) * 16));
    expand_codes_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const uint4*>(packed), chunks,
                                              reinterpret_cast<uint4*>(bytes));
    return after_launch();
}

int launch_rowsum(const uint8_t* codes, int64_t M, int K, int bits, int32_t* rowsum, cudaStream_t st) {
    if (M == 0) return QLLM_OK;
    rowsum_kernel<<<unsigned((M + 7) / 8), 256, 0, st>>>(codes, M, K, bits, rowsum);
    return after_launch();
}

int launch_qgemm_plain(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, int a_bits, int w_bits,
                       const EpilogueArgs& ep, cudaStream_t st) {
    if (M == 0) return QLLM_OK;
    if ((M + 7) / 8 > 65535) return QLLM_ERR_UNSUPPORTED;
    dim3 grid(unsigned((N + 31) / 32), unsigned((M + 7) / 8));
    // word loads need 4-byte aligned rows for both operands
    const bool words = (K % 8 == 0);
    if (words) qgemm_plain_kernel<true><<<grid, 256, 0, st>>>(a, w, M, N, K, a_bits, w_bits, ep);
    else qgemm_plain_kernel<false><<<grid, 256, 0, st>>>(a, w, M, N, K, a_bits, w_bits, ep);
    return after_launch();
}

}  // namespace qllm
