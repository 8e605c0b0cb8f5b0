// Pieces shared by the tcgen05 GEMM kernels: bounded mbarrier waits, the nibble -> byte tile
// expansion, the dequantizing store of an accumulator chunk, tensor-map construction.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.h"
#include "epilogue.cuh"
#include "ptx_sm100.cuh"

namespace qllm {
namespace tc {

constexpr int BM = 128;              // tile rows (tokens) per CTA = MMA M
constexpr int BK = 128;              // codes of K per pipeline stage = one 128-byte swizzle row
constexpr int kUnpackWarps = 8;
constexpr int kFirstEpiWarp = 2, kFirstUnpackWarp = 6;
constexpr long long kWaitCycles = 1ll << 32;   // ~2 s at 2 GHz

struct Abort {
    volatile int* flag;     // shared: some role gave up
    int* status;            // global status word of the library
};

// Waits for a phase of an mbarrier for at most `limit` cycles.  On expiry the CTA's abort flag and the library's
// status word are set and the caller leaves its loop (false); a role that sees the flag set by another gives up too.
__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity, const Abort& ab,
                                             long long limit = kWaitCycles) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 1;; ++i) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 0) {
            if (*ab.flag) return false;
            if (clock64() - t0 > limit) {
                *ab.flag = 1;
                atomicExch(ab.status, QLLM_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// Expand a ROWS x 64-byte tile of packed nibbles into a ROWS x 128-byte swizzled byte tile.
// 16-byte chunk j of row r (codes 32j .. 32j+31) fills units 2j and 2j+1 of the row, each unit
// stored at position unit ^ (r & 7).  PAIRED (both operands 4-bit): even nibbles to unit 2j,
// odd nibbles to unit 2j+1 -- a permutation of K shared by both operands.  Otherwise (the other
// operand holds byte codes in natural order) the nibbles are interleaved back into K order.
template <int ROWS, bool PAIRED>
__device__ __forceinline__ void unpack_tile(const uint8_t* __restrict__ raw, uint8_t* __restrict__ op, int t) {
    constexpr int PER_THREAD = (ROWS * 4 + 32 * kUnpackWarps - 1) / (32 * kUnpackWarps);
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
        const int q = t + i * 32 * kUnpackWarps;
        if (PER_THREAD * 32 * kUnpackWarps != ROWS * 4 && q >= ROWS * 4) break;   // last round of a tile that does not split evenly
        const int r = q >> 2, j = q & 3;
        const uint4 w = *reinterpret_cast<const uint4*>(raw + q * 16);
        uint4 lo, hi;
        lo.x = w.x & 0x0F0F0F0Fu; hi.x = (w.x >> 4) & 0x0F0F0F0Fu;
        lo.y = w.y & 0x0F0F0F0Fu; hi.y = (w.y >> 4) & 0x0F0F0F0Fu;
        lo.z = w.z & 0x0F0F0F0Fu; hi.z = (w.z >> 4) & 0x0F0F0F0Fu;
        lo.w = w.w & 0x0F0F0F0Fu; hi.w = (w.w >> 4) & 0x0F0F0F0Fu;
        uint4 u0 = lo, u1 = hi;
        if (!PAIRED) {
            u0.x = __byte_perm(lo.x, hi.x, 0x5140); u0.y = __byte_perm(lo.x, hi.x, 0x7362);
            u0.z = __byte_perm(lo.y, hi.y, 0x5140); u0.w = __byte_perm(lo.y, hi.y, 0x7362);
            u1.x = __byte_perm(lo.z, hi.z, 0x5140); u1.y = __byte_perm(lo.z, hi.z, 0x7362);
            u1.z = __byte_perm(lo.w, hi.w, 0x5140); u1.w = __byte_perm(lo.w, hi.w, 0x7362);
        }
        uint8_t* row = op + r * 128;
        const int sw = r & 7;
        *reinterpret_cast<uint4*>(row + (((2 * j) ^ sw) << 4)) = u0;
        *reinterpret_cast<uint4*>(row + (((2 * j + 1) ^ sw) << 4)) = u1;
    }
}


// Epilogue of one 32-column chunk of one accumulator row: r[c] = acc[m][nb + c].  Either stores the raw
// int32 accumulators or dequantizes with the row term and the staged column terms and stores f32 / bf16.
// N is a multiple of 8, so 16-byte groups never straddle the end of a row.
__device__ __forceinline__ void store_chunk(const EpilogueArgs& ep, const uint32_t (&r)[32], const int4* colterm,
                                            const RowTerm& rt, int64_t m, int N, int nb) {
    if (ep.raw_acc) {
        int32_t* o = static_cast<int32_t*>(ep.out) + m * N + nb;
#pragma unroll
        for (int v = 0; v < 8; ++v)
            if (nb + 4 * v < N)
                *reinterpret_cast<int4*>(o + 4 * v) = make_int4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
        return;
    }
    float f[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        const int4 ct = colterm[c];
        const int I = int(r[c]) - ct.y * rt.rowsum - rt.zero * ct.z;
        f[c] = fmaf(rt.scale * __int_as_float(ct.x), float(I), __int_as_float(ct.w));
    }
    if (ep.out_dtype == QLLM_F32) {
        float* o = static_cast<float*>(ep.out) + m * N + nb;
#pragma unroll
        for (int v = 0; v < 8; ++v)
            if (nb + 4 * v < N)
                *reinterpret_cast<float4*>(o + 4 * v) = make_float4(f[4 * v], f[4 * v + 1], f[4 * v + 2], f[4 * v + 3]);
    } else {
        __nv_bfloat16* o = static_cast<__nv_bfloat16*>(ep.out) + m * N + nb;
#pragma unroll
        for (int v = 0; v < 4; ++v)
            if (nb + 8 * v < N) {
                uint4 pk;
                __nv_bfloat162 h0 = __floats2bfloat162_rn(f[8 * v], f[8 * v + 1]);
                __nv_bfloat162 h1 = __floats2bfloat162_rn(f[8 * v + 2], f[8 * v + 3]);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(f[8 * v + 4], f[8 * v + 5]);
                __nv_bfloat162 h3 = __floats2bfloat162_rn(f[8 * v + 6], f[8 * v + 7]);
                pk.x = *reinterpret_cast<uint32_t*>(&h0); pk.y = *reinterpret_cast<uint32_t*>(&h1);
                pk.z = *reinterpret_cast<uint32_t*>(&h2); pk.w = *reinterpret_cast<uint32_t*>(&h3);
                *reinterpret_cast<uint4*>(o + 8 * v) = pk;
            }
    }
}

// A 32-row x 32-column chunk of the accumulator, staged for a bulk tensor store.  The values arrive in the
// 16x256b fragment layout (lo: TMEM lanes 0..15 of the warp's quarter, hi: lanes 16..31): thread t holds rows
// t/4 + {0, 8, 16, 24} and, per column group j, columns 8j + 2(t%4), +1 -- so it needs the terms of 8 of the
// chunk's 32 columns instead of all of them.  (With one row per thread every thread read every column's terms:
// 32 broadcast reads per chunk that queue behind the tensor core's operand reads in the same shared memory;
// they took half of the epilogue's time.)  The warp's 32 rows x 64 bytes go to shared memory in the 64-byte
// swizzle of the output tensor map (16-byte unit u of row r at unit u ^ ((r >> 1) & 3); the four rows of a
// thread share that term), which makes the 4- and 8-byte stores of a warp conflict-free, one box per 64 bytes
// of a row; the global writes are whole lines issued by the copy engine.
// box(b) returns the buffer for the b-th box of this chunk (waiting until it is free), send(b, x_bytes) issues it.
template <typename BoxFn, typename SendFn>
__device__ __forceinline__ void stage_chunk(const EpilogueArgs& ep, const uint32_t (&lo)[16], const uint32_t (&hi)[16],
                                            const int4* colterm, const RowTerm (&rt)[4], int lane, int nb, BoxFn box,
                                            SendFn send) {
    const int q = lane & 3, r0 = lane >> 2, sw = (r0 >> 1) & 3;
    auto acc = [&](int i, int j, int e) -> uint32_t { return i < 2 ? lo[4 * j + 2 * i + e] : hi[4 * j + 2 * (i - 2) + e]; };
    auto deq = [&](uint32_t a, const RowTerm& r, const int4& ct) -> float {
        const int I = int(a) - ct.y * r.rowsum - r.zero * ct.z;
        return fmaf(r.scale * __int_as_float(ct.x), float(I), __int_as_float(ct.w));
    };
    if (ep.raw_acc || ep.out_dtype == QLLM_F32) {
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            uint8_t* buf = box(b) + r0 * 64 + (q & 1) * 8;
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                const int j = 2 * b + jj;
                int4 c0 = make_int4(0, 0, 0, 0), c1 = c0;
                if (!ep.raw_acc) { c0 = colterm[8 * j + 2 * q]; c1 = colterm[8 * j + 2 * q + 1]; }
                const int unit = ((2 * jj + (q >> 1)) ^ sw) << 4;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint2 v;
                    if (ep.raw_acc) {
                        v = make_uint2(acc(i, j, 0), acc(i, j, 1));
                    } else {
                        v = make_uint2(__float_as_uint(deq(acc(i, j, 0), rt[i], c0)), __float_as_uint(deq(acc(i, j, 1), rt[i], c1)));
                    }
                    *reinterpret_cast<uint2*>(buf + i * 8 * 64 + unit) = v;
                }
            }
            send(b, nb * 4 + b * 64);
        }
    } else {
        uint8_t* buf = box(0) + r0 * 64 + q * 4;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int4 c0 = colterm[8 * j + 2 * q], c1 = colterm[8 * j + 2 * q + 1];
            const int unit = (j ^ sw) << 4;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                __nv_bfloat162 v2 = __floats2bfloat162_rn(deq(acc(i, j, 0), rt[i], c0), deq(acc(i, j, 1), rt[i], c1));
                *reinterpret_cast<uint32_t*>(buf + i * 8 * 64 + unit) = *reinterpret_cast<uint32_t*>(&v2);
            }
        }
        send(0, nb * 2);
    }
}

// Column terms of the tile's output channels -> shared memory (scale, zero, colsum - K*zero, bias).
__device__ __forceinline__ void stage_col_terms(const EpilogueArgs& ep, int4* colterm, int bn, int n0, int N, int K,
                                                int et, int nthreads) {
    if (ep.raw_acc) return;
    for (int c = et; c < bn; c += nthreads) {
        const int n = n0 + c;
        int4 v = make_int4(0, 0, 0, 0);
        if (n < N) {
            const ColTerm ct = make_col_term(ep.w_scale, ep.w_zero, ep.w_colsum, ep.bias, K, n);
            v = make_int4(__float_as_int(ct.scale), ct.zero, ct.corr, __float_as_int(ct.bias));
        }
        colterm[c] = v;
    }
}

// ---- host side ----------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// uint8 matrix [rows][row_bytes]; box = box_rows x box_bytes; out-of-range parts read as zero.
inline bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t row_bytes, uint32_t box_rows,
              uint32_t box_bytes, bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {box_bytes, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Output matrix [rows][row_bytes] as bytes; box = 32 rows x 64 bytes in the 64-byte swizzle (stage_chunk).
inline bool make_store_map(CUtensorMap* map, void* base, uint64_t rows, uint64_t row_bytes) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {64, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace qllm
