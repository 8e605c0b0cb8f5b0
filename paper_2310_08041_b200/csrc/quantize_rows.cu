// qllm_quantize_rows: the per-token asymmetric quantizer of Eq. 2 alone.
//
// When the reassembly has been folded into the layer that produces the activation (Appendix B: that layer's
// output channels are duplicated / averaged offline, qllm_fold_previous), the run-time half of the pre-GEMM stage
// is only this: range of the row, alpha, zero-point, codes, code sum.  HBM roofline: a row is read once and its
// codes written once.  One to four warps own a row: the row stays in registers between the range pass and the code
// pass (bf16 rows up to 8192 channels, fp32 rows up to 4096), the reductions are warp shuffles, nothing touches
// shared memory but the two exchanges between the warps of a row.  Other shapes take a CTA per row and read the row
// twice (the second time from L2).

#include <cuda_bf16.h>

#include "common.h"
#include "device_utils.cuh"
#include "reassemble_quant_common.cuh"

namespace qllm {

namespace {

template <typename XT>
struct RowVec;                                             // 8 consecutive channels of a row
template <>
struct RowVec<__nv_bfloat16> {
    uint4 r;
    // running range of a lane's channels: bf16 pairs, compared as they are (no widening; a NaN operand is ignored)
    struct Range {
        __nv_bfloat162 lo, hi;
        __device__ __forceinline__ Range() {
            const uint32_t pinf = 0x7F807F80u, ninf = 0xFF80FF80u;
            lo = *reinterpret_cast<const __nv_bfloat162*>(&pinf);
            hi = *reinterpret_cast<const __nv_bfloat162*>(&ninf);
        }
        __device__ __forceinline__ void get(float& l, float& h) const {
            const uint32_t a = *reinterpret_cast<const uint32_t*>(&lo), b = *reinterpret_cast<const uint32_t*>(&hi);
            l = fminf(__uint_as_float(a << 16), __uint_as_float(a & 0xFFFF0000u));
            h = fmaxf(__uint_as_float(b << 16), __uint_as_float(b & 0xFFFF0000u));
        }
    };
    __device__ __forceinline__ void extend(Range& g) const {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const __nv_bfloat162 p = *reinterpret_cast<const __nv_bfloat162*>(&w[k]);
            g.lo = __hmin2(g.lo, p);
            g.hi = __hmax2(g.hi, p);
        }
    }
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { r = __ldcs(reinterpret_cast<const uint4*>(p)); }
    __device__ __forceinline__ void get(float (&f)[8]) const {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            f[2 * k] = __uint_as_float(w[k] << 16);
            f[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
};
template <>
struct RowVec<float> {
    float4 a, b;
    struct Range {
        float lo = INFINITY, hi = -INFINITY;
        __device__ __forceinline__ void get(float& l, float& h) const { l = lo; h = hi; }
    };
    __device__ __forceinline__ void extend(Range& g) const {
        g.lo = min3(g.lo, a.x, a.y); g.lo = min3(g.lo, a.z, a.w); g.lo = min3(g.lo, b.x, b.y); g.lo = min3(g.lo, b.z, b.w);
        g.hi = max3(g.hi, a.x, a.y); g.hi = max3(g.hi, a.z, a.w); g.hi = max3(g.hi, b.x, b.y); g.hi = max3(g.hi, b.z, b.w);
    }
    __device__ __forceinline__ void load(const float* p) {
        a = __ldcs(reinterpret_cast<const float4*>(p));
        b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    }
    __device__ __forceinline__ void get(float (&f)[8]) const {
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
};

// Eq. 2 from the row's range: alpha, 1 / alpha, zero-point (a constant row takes alpha = |value|, 1 if it is 0)
__device__ __forceinline__ void eq2_params(float lo, float hi, float qmax, float& alpha, float& inv, float& zero) {
    alpha = (hi - lo) / qmax;
    if (!(hi > lo)) alpha = lo != 0.f ? fabsf(lo) : 1.f;
    inv = __frcp_rn(alpha);
    zero = -rintf(lo * inv);
}

// How a row's codes are made from its Eq. 2 parameters.  round(f / alpha) + zero is taken as the low bits of
// fma(f, 1 / alpha, 1.5 * 2^23) plus an integer constant (one rounding, to nearest even, no conversion
// instruction: those run at a sixteenth of the arithmetic rate and would bound the kernel); quotients or
// zero-points too large for that constant take the plain form.
struct RowQuant {
    float inv, zero, qmax;
    int zadd, top;
    bool big;
    __device__ __forceinline__ RowQuant(float lo, float hi, float inv_, float zero_, float qmax_)
        : inv(inv_), zero(zero_), qmax(qmax_), zadd(int(zero_) - kMagicBits), top(int(qmax_)),
          big(fmaxf(fabsf(lo), fabsf(hi)) * inv_ >= 2097152.f || fabsf(zero_) >= 2097152.f) {}
};

// 8 codes of consecutive channels -> stored (4 bit: one 32-bit word, else two); returns their sum
__device__ __forceinline__ int store_codes8(const float (&f)[8], const RowQuant& q, int bits, uint8_t* out_row, int g) {
    int n[8];
    if (!q.big) {
#pragma unroll
        for (int j = 0; j < 8; ++j) n[j] = __float_as_int(fmaf(f[j], q.inv, kMagic)) + q.zadd;
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) n[j] = int(fminf(fmaxf(rintf(f[j] * q.inv) + q.zero, 0.f), q.qmax));
    }
    if (bits == 4) {
        uint32_t p = 0;                                    // saturating packs clamp to 0 .. 15
#pragma unroll
        for (int k = 3; k >= 0; --k) p = pack_sat_u4(n[2 * k + 1], n[2 * k], p);
        reinterpret_cast<uint32_t*>(out_row)[g] = p;
        const uint32_t nib = (p & 0x0F0F0F0Fu) + ((p >> 4) & 0x0F0F0F0Fu);
        return int(__dp4a(nib, 0x01010101u, 0u));
    }
    // saturating packs clamp to 0 .. 255; 6-bit codes are cut at 63 first
    uint32_t p0 = pack_sat_u8(min(n[3], q.top), min(n[2], q.top), 0u);
    p0 = pack_sat_u8(min(n[1], q.top), min(n[0], q.top), p0);
    uint32_t p1 = pack_sat_u8(min(n[7], q.top), min(n[6], q.top), 0u);
    p1 = pack_sat_u8(min(n[5], q.top), min(n[4], q.top), p1);
    reinterpret_cast<uint2*>(out_row)[g] = make_uint2(p0, p1);
    return int(__dp4a(p1, 0x01010101u, __dp4a(p0, 0x01010101u, 0u)));
}

// WPR warps per row (1, 2, 4 or 8 of the CTA's 8), the row in registers: NVL vectors of 8 channels per lane.
// Few registers per thread (at most 8 vectors) keep four CTAs on an SM, so that the loads of some warps overlap
// the arithmetic and the stores of others.  The warps of a row meet twice in shared memory (range, code sum).
template <typename XT, int NVL, int WPR>
__global__ void __launch_bounds__(256, 4)
quantize_rows_warp(const XT* __restrict__ x, int64_t M, int bits, uint8_t* __restrict__ codes,
                   float* __restrict__ a_scale, float* __restrict__ a_zero, int32_t* __restrict__ a_rowsum) {
    constexpr int C = NVL * 256 * WPR;
    constexpr int RPC = 8 / WPR;                            // rows per CTA
    __shared__ float s_lo[8], s_hi[8];
    __shared__ int s_sum[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wsub = warp % WPR;
    const int64_t m = int64_t(blockIdx.x) * RPC + warp / WPR;
    const bool live = m < M;
    const XT* xr = x + (live ? m : 0) * C;
    RowVec<XT> v[NVL];
    float lo = INFINITY, hi = -INFINITY;
    if (live) {
#pragma unroll
        for (int i = 0; i < NVL; ++i) v[i].load(xr + 8 * (lane + 32 * (wsub + WPR * i)));
        typename RowVec<XT>::Range range;
#pragma unroll
        for (int i = 0; i < NVL; ++i) v[i].extend(range);
        range.get(lo, hi);
    }
    lo = redux_min(lo);
    hi = redux_max(hi);
    if (WPR > 1) {
        if (lane == 0) { s_lo[warp] = lo; s_hi[warp] = hi; }
        __syncthreads();
#pragma unroll
        for (int w = 0; w < WPR; ++w) {
            lo = fminf(lo, s_lo[warp - wsub + w]);
            hi = fmaxf(hi, s_hi[warp - wsub + w]);
        }
    }
    const float qmax = float((1 << bits) - 1);
    float alpha, inv, zero;
    eq2_params(lo, hi, qmax, alpha, inv, zero);
    const RowQuant rq(lo, hi, inv, zero, qmax);
    int sum = 0;
    if (live) {
        uint8_t* out_row = codes + m * (bits == 4 ? C / 2 : C);
#pragma unroll
        for (int i = 0; i < NVL; ++i) {
            float f[8];
            v[i].get(f);
            sum += store_codes8(f, rq, bits, out_row, lane + 32 * (wsub + WPR * i));
        }
    }
    sum = __reduce_add_sync(0xffffffffu, sum);
    if (WPR > 1) {
        if (lane == 0) s_sum[warp] = sum;
        __syncthreads();
        sum = 0;
#pragma unroll
        for (int w = 0; w < WPR; ++w) sum += s_sum[warp - wsub + w];
    }
    if (live && wsub == 0 && lane == 0) {
        a_scale[m] = alpha;
        a_zero[m] = zero;
        if (a_rowsum) a_rowsum[m] = sum;
    }
}

// Any channel count: a CTA per row, two reads of the row.
template <typename XT>
__global__ void __launch_bounds__(256)
quantize_rows_cta(const XT* __restrict__ x, int64_t M, int C, int bits, uint8_t* __restrict__ codes,
                  float* __restrict__ a_scale, float* __restrict__ a_zero, int32_t* __restrict__ a_rowsum) {
    __shared__ float red[64];
    const float qmax = float((1 << bits) - 1);
    for (int64_t m = blockIdx.x; m < M; m += gridDim.x) {
        const XT* xr = x + m * C;
        float lo = INFINITY, hi = -INFINITY;
        for (int k = threadIdx.x; k < C; k += blockDim.x) {
            const float f = float(xr[k]);
            lo = fminf(lo, f);
            hi = fmaxf(hi, f);
        }
        block_minmax(lo, hi, red);
        float alpha, inv, zero;
        eq2_params(lo, hi, qmax, alpha, inv, zero);
        int sum = 0;
        if (bits == 4) {
            uint8_t* out = codes + m * (C / 2);
            for (int p = threadIdx.x; p < C / 2; p += blockDim.x) {
                const int q0 = int(fminf(fmaxf(rintf(float(xr[2 * p]) * inv) + zero, 0.f), qmax));
                const int q1 = int(fminf(fmaxf(rintf(float(xr[2 * p + 1]) * inv) + zero, 0.f), qmax));
                out[p] = uint8_t(q0 | (q1 << 4));
                sum += q0 + q1;
            }
        } else {
            uint8_t* out = codes + m * C;
            for (int k = threadIdx.x; k < C; k += blockDim.x) {
                const int q = int(fminf(fmaxf(rintf(float(xr[k]) * inv) + zero, 0.f), qmax));
                out[k] = uint8_t(q);
                sum += q;
            }
        }
        const int total = block_sum_int(sum, reinterpret_cast<int*>(red));
        if (threadIdx.x == 0) {
            a_scale[m] = alpha;
            a_zero[m] = zero;
            if (a_rowsum) a_rowsum[m] = total;
        }
        __syncthreads();
    }
}

template <typename XT, int NVL, int WPR>
int launch_warp_rows(const XT* xp, int64_t M, int bits, uint8_t* codes, float* a_scale, float* a_zero, int32_t* a_rowsum,
                     cudaStream_t st) {
    constexpr int RPC = 8 / WPR;
    quantize_rows_warp<XT, NVL, WPR><<<unsigned((M + RPC - 1) / RPC), 256, 0, st>>>(xp, M, bits, codes, a_scale, a_zero,
                                                                                  a_rowsum);
    return after_launch();
}

template <typename XT>
int launch_rows(const void* x, int64_t M, int C, int bits, uint8_t* codes, float* a_scale, float* a_zero,
                int32_t* a_rowsum, cudaStream_t st) {
    const XT* xp = static_cast<const XT*>(x);
#define QLLM_QR(NVL, WPR) return launch_warp_rows<XT, NVL, WPR>(xp, M, bits, codes, a_scale, a_zero, a_rowsum, st)
    if (C % 256 == 0 && M <= (int64_t(1) << 32)) {
        // vectors of 8 channels per lane of one warp, split over as many warps as keep it at 8 (bf16) / 4 (fp32)
        const int nv = C / 256;
        if (sizeof(XT) == 2) {
            switch (nv) {
                case 1: QLLM_QR(1, 1); case 2: QLLM_QR(2, 1); case 4: QLLM_QR(4, 1); case 8: QLLM_QR(8, 1);
                case 16: QLLM_QR(8, 2); case 20: QLLM_QR(5, 4); case 32: QLLM_QR(8, 4); default: break;
            }
        } else {
            switch (nv) {
                case 1: QLLM_QR(1, 1); case 2: QLLM_QR(2, 1); case 4: QLLM_QR(4, 1); case 8: QLLM_QR(4, 2);
                case 16: QLLM_QR(4, 4); default: break;
            }
        }
    }
#undef QLLM_QR
    const int g2 = int(std::min<int64_t>(M, int64_t(device_sm_count()) * 8));
    quantize_rows_cta<XT><<<g2, 256, 0, st>>>(xp, M, C, bits, codes, a_scale, a_zero, a_rowsum);
    return after_launch();
}

}  // namespace
}  // namespace qllm

extern "C" int qllm_quantize_rows(const void* x, int x_dtype, int64_t M, int C, int bits, uint8_t* codes,
                                  float* a_scale, float* a_zero, int32_t* a_rowsum, void* stream) {
    using namespace qllm;
    if (!bits_ok(bits)) return QLLM_ERR_BITS;
    if (!dtype_ok(x_dtype)) return QLLM_ERR_DTYPE;
    if (M < 0 || C <= 0 || (bits == 4 && (C & 1))) return QLLM_ERR_SHAPE;
    if (M == 0) return QLLM_OK;
    if (!x || !codes || !a_scale || !a_zero) return QLLM_ERR_NULL;
    if (!aligned16(x) || !aligned16(codes)) return QLLM_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return x_dtype == QLLM_BF16 ? launch_rows<__nv_bfloat16>(x, M, C, bits, codes, a_scale, a_zero, a_rowsum, st)
                                : launch_rows<float>(x, M, C, bits, codes, a_scale, a_zero, a_rowsum, st);
}
