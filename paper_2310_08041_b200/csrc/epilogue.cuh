// Dequantizing epilogue of the integer GEMM (Eq. 2 inverted on both operands):
//   I   = acc - zw[n]*rs[m] - za[m]*cs[n] + K*za[m]*zw[n]      (exact, int32 ring)
//   out = (a_scale[m] * w_scale[n]) * I + bias[n]
// Row terms (m) and column terms (n) are prepared once per row / column by the caller.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace qllm {

struct RowTerm { float scale; int zero; int rowsum; };     // a_scale, za, rs
struct ColTerm { float scale; int zero; int corr; float bias; };  // w_scale, zw, cs - K*zw, bias

__device__ __forceinline__ ColTerm make_col_term(const float* w_scale, const float* w_zero,
                                                 const int32_t* w_colsum, const float* bias, int K, int n) {
    ColTerm c;
    c.scale = w_scale[n];
    c.zero = __float2int_rn(w_zero[n]);
    c.corr = w_colsum[n] - K * c.zero;
    c.bias = bias ? bias[n] : 0.f;
    return c;
}
__device__ __forceinline__ RowTerm make_row_term(const float* a_scale, const float* a_zero,
                                                 const int32_t* a_rowsum, int64_t m) {
    RowTerm r;
    r.scale = a_scale[m];
    r.zero = __float2int_rn(a_zero[m]);
    r.rowsum = a_rowsum[m];
    return r;
}
__device__ __forceinline__ float dequant(int acc, const RowTerm& r, const ColTerm& c) {
    // acc - zw*rs - za*(cs - K*zw)
    const int I = acc - c.zero * r.rowsum - r.zero * c.corr;
    return fmaf(r.scale * c.scale, float(I), c.bias);
}

}  // namespace qllm
