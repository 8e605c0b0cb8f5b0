// Fused pre-GEMM kernel, one warp per token: LayerNorm -> channel reassembly -> per-token
// asymmetric quantization (QLLM Eq. 2-4; the fusion the paper leaves as future work, Sec. 6).
//
// HBM roofline: a token row of x is read from DRAM once (a second pass hits L1/L2) and its codes
// are written once.  Design:
//  * a warp owns a token from load to store, so no CTA barrier sits on the per-token path; the
//    three row reductions (sum, sum of squares, min/max) are warp shuffles / redux.  A CTA is
//    as many warps as shared memory holds rows for, one CTA per SM, tokens dealt round-robin.
//  * the reassembly map is compiled (once per layer, or per call) into per-output-channel
//    records {16-bit position in the row, weight = coef * gamma[src], bias = sum coef * beta[src]}
//    that the CTA keeps in shared memory.  Rows with several entries (merged channels, Eq. 4)
//    become "virtual slots": once per token a lane sums their entries into a slot appended to the
//    row, so that every output channel is ONE gather:   x'_c = rstd * w_c * d[pos_c] + b_c.
//  * the centred row d = x - mean lives in the warp's shared-memory row in 8 planes
//    (channel k at plane k % 8, index k / 8): a lane owns 8 consecutive channels per step, so
//    both the plane stores and the gathers of mostly order-preserving maps walk consecutive banks,
//    and a lane packs whole 32-bit (4-bit codes) or 64-bit (byte lanes) words of output.
//  * the gathers run twice (min/max pass, quantize pass) instead of keeping C / 32 values per
//    lane in registers: registers stay low for any C and the second pass re-reads shared memory.
//  * rounding by the 1.5 * 2^23 magic constant (nearest-even, as cvt.rni), saturating cvt.pack
//    for the clamp and the nibble / byte packing.
// A map with more multi-entry rows than the row has slots for makes the whole launch walk the CSR
// arrays instead (correct, slow; the specialised path covers every map the builder produces for
// LLM-like outlier statistics).

#include <cuda_bf16.h>

#include "common.h"
#include "device_utils.cuh"

namespace qllm {

namespace {

constexpr int kSlotCap = 2048;                 // virtual slots an image can describe
constexpr int kInline = 4;                     // entries held inside a slot record
constexpr int kLongCap = 512;                  // entries of longer rows kept as (position, weight) pairs
constexpr int kLongRows = 256;                 // longer rows listed by slot (more: the slot pass scans for them)
constexpr int kMaxWarps = 16;
constexpr int kSmemBudget = 227 * 1024;
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23
constexpr int kMagicBits = 0x4B400000;

// position of channel k in a warp's row
__host__ __device__ __forceinline__ int dplane(int k, int C) { return (k & 7) * (C >> 3) + (k >> 3); }

__device__ __forceinline__ float redux_min(float v) {
    float r;
    asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float redux_max(float v) {
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// d = sat_u4(a) << 4 | sat_u4(b) | c << 8
__device__ __forceinline__ uint32_t pack_sat_u4(int a, int b, uint32_t c) {
    uint32_t d;
    asm("cvt.pack.sat.u4.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// d = sat_u8(a) << 8 | sat_u8(b) | c << 16
__device__ __forceinline__ uint32_t pack_sat_u8(int a, int b, uint32_t c) {
    uint32_t d;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(uint32_t(__cvta_generic_to_shared(smem))), "l"(gmem)
                 : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// Compiled map: one allocation, in this order.
//   idx  uint16[C]      word position in the row of the channel's (first or only) source, or C + slot
//   wlo  float[C/8][4]  weights of channels 8g .. 8g+3        whi: channels 8g+4 .. 8g+7
//   blo, bhi            bias terms in the same layout (zero without beta)
//   olo, ohi uint32[C/8][4]  the positions again as byte offsets (4 * idx), in the weights' layout
//   vrec uint4[kSlotCap][2]  slot s: {pos0 | pos1 << 16, pos2 | pos3 << 16, w0, w1}, {w2, w3, n, 0}
//                            for n <= kInline entries; {first CSR entry, -, -, -}, {-, -, n, 0} otherwise
//                            for n <= kInline entries; {0, 0, 0, 0}, {first entry in lent, 0, n, 1} for a longer
//                            row whose entries fit lent; {0, 0, 0, 0}, {first CSR entry, 0, n, 0} otherwise (the
//                            inline fields of such a record are harmless when evaluated: positions 0)
//   lent uint2[kLongCap]     entries of the longer rows: {position, weight bits}
//   lrow int[kLongRows]      slots of the longer rows, in no particular order
//   head int[4]         [0] = slots handed out (more than kSlotCap: the map does not fit), [1] = entries handed
//                       out in lent, [2] = rows longer than kInline
struct WarpImage {
    uint16_t* idx;
    float *wlo, *whi, *blo, *bhi;
    uint32_t *olo, *ohi;
    uint4* vrec;
    uint2* lent;
    int* lrow;
    int* head;
};
__host__ __device__ inline size_t warp_image_bytes(int C) {
    return size_t(C) * 14 + size_t(kSlotCap) * 32 + size_t(kLongCap) * 8 + size_t(kLongRows) * 4 + 16;
}
__host__ __device__ inline WarpImage warp_image_at(void* base, int C) {
    WarpImage im;
    uint8_t* b = static_cast<uint8_t*>(base);
    im.idx = reinterpret_cast<uint16_t*>(b);
    im.wlo = reinterpret_cast<float*>(b + size_t(C) * 2);
    im.whi = im.wlo + C / 2;
    im.blo = im.whi + C / 2;
    im.bhi = im.blo + C / 2;
    im.olo = reinterpret_cast<uint32_t*>(im.bhi + C / 2);
    im.ohi = im.olo + C / 2;
    im.vrec = reinterpret_cast<uint4*>(im.ohi + C / 2);
    im.lent = reinterpret_cast<uint2*>(im.vrec + 2 * size_t(kSlotCap));
    im.lrow = reinterpret_cast<int*>(im.lent + kLongCap);
    im.head = im.lrow + kLongRows;
    return im;
}

// One thread per output channel.  im.head[0] must be zero at launch.
__global__ void __launch_bounds__(256)
compile_map_warp_kernel(int C, const float* __restrict__ gamma, const float* __restrict__ beta,
                        const int32_t* __restrict__ ptr, const int32_t* __restrict__ src,
                        const float* __restrict__ coef, WarpImage im) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    const int j0 = __ldg(ptr + c), n = __ldg(ptr + c + 1) - j0;
    const int s0 = __ldg(src + j0);
    const float c0 = __ldg(coef + j0);
    uint32_t pos = uint32_t(dplane(s0, C));
    float w = c0 * __ldg(gamma + s0);
    float b = beta ? c0 * __ldg(beta + s0) : 0.f;
    if (n > 1) {                                          // merged row
        if (beta)
            for (int j = j0 + 1; j < j0 + n; ++j) b = fmaf(__ldg(coef + j), __ldg(beta + __ldg(src + j)), b);
        const int vi = atomicAdd(im.head, 1);
        if (vi < kSlotCap) {
            if (n <= kInline) {
                uint32_t o[kInline] = {0, 0, 0, 0};
                float ww[kInline] = {0.f, 0.f, 0.f, 0.f};
                for (int e = 0; e < n; ++e) {
                    const int sj = __ldg(src + j0 + e);
                    o[e] = uint32_t(dplane(sj, C));
                    ww[e] = __ldg(coef + j0 + e) * __ldg(gamma + sj);
                }
                im.vrec[2 * vi] = make_uint4(o[0] | (o[1] << 16), o[2] | (o[3] << 16), __float_as_uint(ww[0]),
                                             __float_as_uint(ww[1]));
                im.vrec[2 * vi + 1] = make_uint4(__float_as_uint(ww[2]), __float_as_uint(ww[3]), uint32_t(n), 0u);
            } else {
                const int first = atomicAdd(im.head + 1, n);
                if (first + n <= kLongCap) {              // entries as (position, weight) pairs for shared memory
                    for (int e = 0; e < n; ++e) {
                        const int sj = __ldg(src + j0 + e);
                        im.lent[first + e] = make_uint2(uint32_t(dplane(sj, C)),
                                                        __float_as_uint(__ldg(coef + j0 + e) * __ldg(gamma + sj)));
                    }
                    im.vrec[2 * vi] = make_uint4(0u, 0u, 0u, 0u);
                    im.vrec[2 * vi + 1] = make_uint4(uint32_t(first), 0u, uint32_t(n), 1u);
                } else {                                  // walks the CSR arrays at run time
                    im.vrec[2 * vi] = make_uint4(0u, 0u, 0u, 0u);
                    im.vrec[2 * vi + 1] = make_uint4(uint32_t(j0), 0u, uint32_t(n), 0u);
                }
                const int li = atomicAdd(im.head + 2, 1);   // number of longer rows
                if (li < kLongRows) im.lrow[li] = vi;
            }
            pos = uint32_t(C + vi);
            w = 1.0f;
        }
    }
    im.idx[c] = uint16_t(pos);
    const int g = c >> 3, j = c & 7;
    (j < 4 ? im.wlo : im.whi)[4 * g + (j & 3)] = w;
    (j < 4 ? im.blo : im.bhi)[4 * g + (j & 3)] = b;
    (j < 4 ? im.olo : im.ohi)[4 * g + (j & 3)] = pos * 4u;
}

// 8 consecutive channels of a row as floats
template <typename XT>
__device__ __forceinline__ void load8(const XT* p, float (&f)[8]);
template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, float (&f)[8]) {
    const uint4 r = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        f[2 * k] = __uint_as_float(w[k] << 16);
        f[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
    }
}
template <>
__device__ __forceinline__ void load8<float>(const float* p, float (&f)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
    f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

struct RawMap {
    const float* gamma;
    const int32_t* ptr;
    const int32_t* src;
    const float* coef;
};

// sum_j coef_j gamma[src_j] d[pos(src_j)] over CSR entries [j0, j0 + n)
__device__ __forceinline__ float csr_row(const RawMap& rm, const float* d, int C, int j0, int n) {
    float e = 0.f;
    for (int j = j0; j < j0 + n; ++j) {
        const int sj = __ldg(rm.src + j);
        e = fmaf(__ldg(rm.coef + j) * __ldg(rm.gamma + sj), d[dplane(sj, C)], e);
    }
    return e;
}

// sum of a longer row's entries kept as (position, weight) pairs
__device__ __forceinline__ float pair_row(const uint2* ent, const float* d, int first, int n) {
    float e = 0.f;
    for (int k = 0; k < n; ++k) {
        const uint2 pw = ent[first + k];
        e = fmaf(__uint_as_float(pw.y), d[pw.x], e);
    }
    return e;
}

// the whole CSR row of output channel c (kept out of line: it serves only maps that do not fit the slots)
__device__ __noinline__ float csr_channel(const RawMap& rm, const float* d, int C, int c) {
    const int j0 = __ldg(rm.ptr + c);
    return csr_row(rm, d, C, j0, __ldg(rm.ptr + c + 1) - j0);
}

// u[j] = w_c d[pos_c] for the 8 channels c = 8g + j of group g (before rstd and bias)
template <bool SLOW>
__device__ __forceinline__ void gather8(int g, const uint16_t* s_idx, const float* s_wlo, const float* s_whi,
                                        const float* d, const RawMap& rm, int C, float (&u)[8]) {
    if (SLOW) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = 8 * g + j, j0 = __ldg(rm.ptr + c);
            u[j] = csr_row(rm, d, C, j0, __ldg(rm.ptr + c + 1) - j0);
        }
        return;
    }
    const uint4 iw = *reinterpret_cast<const uint4*>(s_idx + 8 * g);
    const float4 wl = *reinterpret_cast<const float4*>(s_wlo + 4 * g);
    const float4 wh = *reinterpret_cast<const float4*>(s_whi + 4 * g);
    u[0] = wl.x * d[iw.x & 0xFFFFu]; u[1] = wl.y * d[iw.x >> 16];
    u[2] = wl.z * d[iw.y & 0xFFFFu]; u[3] = wl.w * d[iw.y >> 16];
    u[4] = wh.x * d[iw.z & 0xFFFFu]; u[5] = wh.y * d[iw.z >> 16];
    u[6] = wh.z * d[iw.w & 0xFFFFu]; u[7] = wh.w * d[iw.w >> 16];
}

template <typename XT, bool HAS_BETA, bool PACKED>
__global__ void __launch_bounds__(32 * kMaxWarps, 1)
reassemble_quant_warp(const XT* __restrict__ x, int64_t M, int C, float eps, int bits, WarpImage im,
                      int row_words, RawMap rm, uint8_t* __restrict__ codes, float* __restrict__ a_scale,
                      float* __restrict__ a_zero, int32_t* __restrict__ a_rowsum) {
    extern __shared__ __align__(16) uint8_t smem_bytes[];
    uint16_t* s_idx = reinterpret_cast<uint16_t*>(smem_bytes);
    float* s_wlo = reinterpret_cast<float*>(smem_bytes + size_t(C) * 2);
    float* s_whi = s_wlo + C / 2;
    float* s_blo = s_whi + C / 2;                          // bias arrays only with beta
    float* s_bhi = s_blo + C / 2;
    float* rows = HAS_BETA ? s_bhi + C / 2 : s_blo;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, W = blockDim.x >> 5;
    {   // records -> shared memory (the image holds idx | wlo | whi | blo | bhi back to back)
        const uint4* g4 = reinterpret_cast<const uint4*>(im.idx);
        uint4* s4 = reinterpret_cast<uint4*>(smem_bytes);
        const int n16 = (HAS_BETA ? 10 : 6) * C / 16;
        for (int i = threadIdx.x; i < n16; i += blockDim.x) s4[i] = __ldg(g4 + i);
    }
    const int slots_total = __ldg(im.head);
    const int slot_room = row_words - C;
    const bool slow = slots_total > slot_room;             // uniform over the grid
    const int nslots = slow ? 0 : slots_total;
    __syncthreads();

    float* d = rows + size_t(warp) * row_words;
    const int G = C >> 3;                                  // groups of 8 channels
    const int P = C >> 3;                                  // plane stride in words
    const float invC = 1.0f / float(C);
    const float qmax = float((1 << bits) - 1);
    const float inv_qmax = 1.0f / qmax;
    const int64_t stride = int64_t(gridDim.x) * W;

    for (int64_t m = int64_t(blockIdx.x) * W + warp; m < M; m += stride) {
        const XT* xr = x + m * C;
        // -- mean
        float s = 0.f;
#pragma unroll 4
        for (int g = lane; g < G; g += 32) {
            float f[8];
            load8<XT>(xr + 8 * g, f);
            s += ((f[0] + f[1]) + (f[2] + f[3])) + ((f[4] + f[5]) + (f[6] + f[7]));
        }
        const float mean = warp_sum(s) * invC;
        // -- centred row to the warp's planes, variance
        float sq = 0.f;
#pragma unroll 4
        for (int g = lane; g < G; g += 32) {
            float f[8];
            load8<XT>(xr + 8 * g, f);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                f[j] -= mean;
                sq = fmaf(f[j], f[j], sq);
                d[j * P + g] = f[j];
            }
        }
        const float rstd = rsqrtf(warp_sum(sq) * invC + eps);   // a common factor of the whole row: its
                                                                 // last-bit error rescales alpha, codes unchanged
        if (m + stride < M) {                                    // next row of this warp towards L2
            const char* xn = reinterpret_cast<const char*>(x + (m + stride) * C);
            for (int o = lane * 128; o < C * int(sizeof(XT)); o += 32 * 128) prefetch_l2(xn + o);
        }
        __syncwarp();
        // -- merged rows: a lane per row sums the entries into the row's virtual slot
        for (int vi = lane; vi < nslots; vi += 32) {
            const uint4 r0 = __ldg(im.vrec + 2 * vi), r1 = __ldg(im.vrec + 2 * vi + 1);
            float e;
            if (r1.z <= uint32_t(kInline)) {
                e = __uint_as_float(r0.z) * d[r0.x & 0xFFFFu];
                e = fmaf(__uint_as_float(r0.w), d[r0.x >> 16], e);
                if (r1.z > 2u) {
                    e = fmaf(__uint_as_float(r1.x), d[r0.y & 0xFFFFu], e);
                    if (r1.z > 3u) e = fmaf(__uint_as_float(r1.y), d[r0.y >> 16], e);
                }
            } else if (r1.w) {
                e = pair_row(im.lent, d, int(r1.x), int(r1.z));
            } else {
                e = csr_row(rm, d, C, int(r1.x), int(r1.z));
            }
            d[C + vi] = e;
        }
        __syncwarp();
        // -- row range of x' (first gather pass)
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll 2
        for (int g = lane; g < G; g += 32) {
            float u[8];
            if (slow) gather8<true>(g, s_idx, s_wlo, s_whi, d, rm, C, u);
            else gather8<false>(g, s_idx, s_wlo, s_whi, d, rm, C, u);
            if (HAS_BETA) {
                const float4 bl = *reinterpret_cast<const float4*>(s_blo + 4 * g);
                const float4 bh = *reinterpret_cast<const float4*>(s_bhi + 4 * g);
                u[0] = fmaf(rstd, u[0], bl.x); u[1] = fmaf(rstd, u[1], bl.y);
                u[2] = fmaf(rstd, u[2], bl.z); u[3] = fmaf(rstd, u[3], bl.w);
                u[4] = fmaf(rstd, u[4], bh.x); u[5] = fmaf(rstd, u[5], bh.y);
                u[6] = fmaf(rstd, u[6], bh.z); u[7] = fmaf(rstd, u[7], bh.w);
            }
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                lo = min3(lo, u[j], u[j + 1]);
                hi = max3(hi, u[j], u[j + 1]);
            }
        }
        if (!HAS_BETA) { lo *= rstd; hi *= rstd; }         // rstd > 0: scaling commutes with min / max
        lo = redux_min(lo);
        hi = redux_max(hi);
        // -- Eq. 2
        float alpha = (hi - lo) * inv_qmax;
        if (!(hi > lo)) alpha = lo != 0.f ? fabsf(lo) : 1.f;
        const float inv = __frcp_rn(alpha);
        const float zero = -rintf(lo * inv);
        const bool big = fmaxf(fabsf(lo), fabsf(hi)) * inv >= 2097152.f || fabsf(zero) >= 2097152.f;
        const int zadd = int(zero) - kMagicBits;
        const int top = int(qmax);
        int csum = 0;
        // -- codes (second gather pass)
#pragma unroll 2
        for (int g = lane; g < G; g += 32) {
            float u[8];
            if (slow) gather8<true>(g, s_idx, s_wlo, s_whi, d, rm, C, u);
            else gather8<false>(g, s_idx, s_wlo, s_whi, d, rm, C, u);
            if (HAS_BETA) {
                const float4 bl = *reinterpret_cast<const float4*>(s_blo + 4 * g);
                const float4 bh = *reinterpret_cast<const float4*>(s_bhi + 4 * g);
                u[0] = fmaf(rstd, u[0], bl.x); u[1] = fmaf(rstd, u[1], bl.y);
                u[2] = fmaf(rstd, u[2], bl.z); u[3] = fmaf(rstd, u[3], bl.w);
                u[4] = fmaf(rstd, u[4], bh.x); u[5] = fmaf(rstd, u[5], bh.y);
                u[6] = fmaf(rstd, u[6], bh.z); u[7] = fmaf(rstd, u[7], bh.w);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] *= rstd;
            }
            int n[8];
            if (!big) {
#pragma unroll
                for (int j = 0; j < 8; ++j) n[j] = __float_as_int(fmaf(u[j], inv, kMagic)) + zadd;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) n[j] = int(fminf(fmaxf(rintf(u[j] * inv) + zero, 0.f), qmax));
            }
            if (PACKED) {
                // one byte per channel pair: low nibble = even channel
                uint32_t p = 0;
#pragma unroll
                for (int i = 3; i >= 0; --i) p = pack_sat_u4(n[2 * i + 1], n[2 * i], p);
                const uint32_t nib = (p & 0x0F0F0F0Fu) + ((p >> 4) & 0x0F0F0F0Fu);
                csum = int(__dp4a(nib, 0x01010101u, uint32_t(csum)));
                *reinterpret_cast<uint32_t*>(codes + m * (C / 2) + 4 * g) = p;
            } else {
                uint32_t p0 = pack_sat_u8(min(n[3], top), min(n[2], top), 0u);
                p0 = pack_sat_u8(min(n[1], top), min(n[0], top), p0);
                uint32_t p1 = pack_sat_u8(min(n[7], top), min(n[6], top), 0u);
                p1 = pack_sat_u8(min(n[5], top), min(n[4], top), p1);
                csum = int(__dp4a(p0, 0x01010101u, uint32_t(csum)));
                csum = int(__dp4a(p1, 0x01010101u, uint32_t(csum)));
                *reinterpret_cast<uint2*>(codes + m * C + 8 * g) = make_uint2(p0, p1);
            }
        }
        csum = __reduce_add_sync(0xffffffffu, csum);
        if (lane == 0) {
            a_scale[m] = alpha;
            a_zero[m] = zero;
            if (a_rowsum) a_rowsum[m] = csum;
        }
        __syncwarp();                                      // the row is rewritten by the next token
    }
}

// ---- compile-time channel counts ---------------------------------------------------------
// Same algorithm with the shape fixed at compile time (LLaMA hidden sizes): G warps share a token,
// a lane owns NPL = C / (32 G) channels, 8 consecutive ones per step.  The whole row is loaded
// with all its 16-byte loads in flight, converted once, and the reassembled values x' stay in
// registers between the range pass and the quantize pass, so each channel is gathered once.
// Records are kept as 32-bit byte offsets so that a gather is one shared load at [offset + row].
template <int G>
__device__ __forceinline__ void token_sync(int barid) {
    if (G == 1) __syncwarp();
    else asm volatile("bar.sync %0, %1;" ::"r"(barid), "n"(32 * G) : "memory");
}
// Sum over the G warps of a token; every lane returns the total.  ex: [2][G] floats, parity-buffered.
template <int G>
__device__ __forceinline__ float token_sum(float v, float* ex, int& par, int wsub, int lane, int barid) {
    v = warp_sum(v);
    if (G == 1) { __syncwarp(); return v; }
    if (lane == 0) ex[par * G + wsub] = v;
    token_sync<G>(barid);
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < G; ++w) t += ex[par * G + w];
    par ^= 1;
    return t;
}

template <int NPL, int G, bool HAS_BETA, bool PACKED, int MAXW>
__global__ void __launch_bounds__(32 * MAXW, 1)
reassemble_quant_token(const __nv_bfloat16* __restrict__ x, int64_t M, float eps, int bits, WarpImage im,
                       int row_words, int TOK /* tokens in flight per CTA */, RawMap rm, uint8_t* __restrict__ codes, float* __restrict__ a_scale,
                       float* __restrict__ a_zero, int32_t* __restrict__ a_rowsum) {
    constexpr int C = NPL * 32 * G;
    constexpr int NIT = NPL / 8;                           // steps of 8 channels per lane
    constexpr int P = C / 8;                               // plane stride in words
    constexpr int GS = 32 * G;                             // groups per step over the token's lanes
    extern __shared__ __align__(16) uint8_t smem_bytes[];
    float* s_wA = reinterpret_cast<float*>(smem_bytes);    // [C/8][4] weights of channels 8g..8g+3
    float* s_wB = s_wA + C / 2;                            //                      channels 8g+4..8g+7
    float* s_bA = s_wB + C / 2;                            // bias arrays only with beta
    float* s_bB = s_bA + C / 2;
    uint32_t* s_offA = reinterpret_cast<uint32_t*>(HAS_BETA ? s_bB + C / 2 : s_bA);   // byte offsets, same layout
    uint32_t* s_offB = s_offA + C / 2;
    float* s_ex = reinterpret_cast<float*>(s_offB + C / 2);             // [MAXW / G][8 G] exchange words per token slot
    uint4* s_vrec = reinterpret_cast<uint4*>(s_ex + (MAXW / G) * 8 * G);   // [row_words - C][2] slot records
    uint2* s_lent = reinterpret_cast<uint2*>(s_vrec + 2 * size_t(row_words - C));   // [kLongCap] entries of longer rows
    int* s_lrow = reinterpret_cast<int*>(s_lent + kLongCap);                    // [kLongRows] their slots
    float* rows = reinterpret_cast<float*>(s_lrow + kLongRows);

    const int lane = threadIdx.x & 31;
    const int warp = __shfl_sync(0xffffffffu, int(threadIdx.x >> 5), 0);   // warp-uniform for the compiler
    if (warp / G < TOK) {                                  // first row of this token slot towards L2
        const int64_t m0 = int64_t(blockIdx.x) * TOK + warp / G;
        if (m0 < M) {
            const char* x0 = reinterpret_cast<const char*>(x + m0 * C);
            for (int o = ((warp % G) * 32 + lane) * 128; o < C * 2; o += GS * 128) prefetch_l2(x0 + o);
        }
    }
    {   // records -> shared memory, asynchronously: they are first needed after the first row's statistics
        const uint4* gw = reinterpret_cast<const uint4*>(im.wlo);       // wlo | whi | blo | bhi back to back
        const int nw16 = (HAS_BETA ? 8 : 4) * C / 16;
        for (int i = threadIdx.x; i < nw16; i += blockDim.x) cp_async16(reinterpret_cast<uint4*>(s_wA) + i, gw + i);
        const uint4* go = reinterpret_cast<const uint4*>(im.olo);       // olo | ohi back to back
        for (int i = threadIdx.x; i < 4 * C / 16; i += blockDim.x) cp_async16(reinterpret_cast<uint4*>(s_offA) + i, go + i);
        for (int i = threadIdx.x; i < 2 * (row_words - C); i += blockDim.x) cp_async16(s_vrec + i, im.vrec + i);
        for (int i = threadIdx.x; i < kLongCap / 2; i += blockDim.x)
            cp_async16(reinterpret_cast<uint4*>(s_lent) + i, reinterpret_cast<const uint4*>(im.lent) + i);
        for (int i = threadIdx.x; i < kLongRows / 4; i += blockDim.x)
            cp_async16(reinterpret_cast<uint4*>(s_lrow) + i, reinterpret_cast<const uint4*>(im.lrow) + i);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const int slots_total = __ldg(im.head);
    const bool slow = slots_total > row_words - C;         // uniform over the grid: walk the CSR arrays
    const int nslots = slow ? 0 : slots_total;
    const int nlong = __ldg(im.head + 2);                  // rows longer than a slot record
    bool records_pending = true;

    const int tslot = warp / G, wsub = warp % G;
    if (tslot >= TOK) {                                    // spare warps only helped with the copy
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        return;
    }
    const int barid = 1 + tslot;
    float* d = rows + size_t(tslot) * row_words;
    float* ex = s_ex + tslot * 8 * G;
    float* exr = ex + 2 * G;                               // range exchange: [2][G][2]
    const char* dbytes = reinterpret_cast<const char*>(d);
    const int g0 = wsub * 32 + lane;                       // this lane's group in step 0
    const float invC = 1.0f / float(C);
    const float qmax = float((1 << bits) - 1);
    const float inv_qmax = 1.0f / qmax;
    const int top = int(qmax);
    const int64_t stride = int64_t(gridDim.x) * TOK;
    int par = 0;

    for (int64_t m = int64_t(blockIdx.x) * TOK + tslot; m < M; m += stride) {
        const __nv_bfloat16* xr = x + m * C + 8 * g0;
        uint4 raw[NIT];
#pragma unroll
        for (int i = 0; i < NIT; ++i) raw[i] = *reinterpret_cast<const uint4*>(xr + i * 8 * GS);
        // -- mean
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
            float t = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) t += __uint_as_float(w[k] << 16) + __uint_as_float(w[k] & 0xFFFF0000u);
            s += t;
        }
        const float mean = token_sum<G>(s, ex, par, wsub, lane, barid) * invC;
        // -- centred row to the token's planes, variance
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float a = __uint_as_float(w[k] << 16) - mean;
                const float b = __uint_as_float(w[k] & 0xFFFF0000u) - mean;
                sq = fmaf(a, a, sq);
                sq = fmaf(b, b, sq);
                d[(2 * k) * P + g0 + i * GS] = a;
                d[(2 * k + 1) * P + g0 + i * GS] = b;
            }
        }
        // the exchange inside token_sum also makes the row visible to the token's lanes
        const float rstd = rsqrtf(token_sum<G>(sq, ex, par, wsub, lane, barid) * invC + eps);
        if (m + stride < M) {                              // next row of this token slot towards L2
            const char* xn = reinterpret_cast<const char*>(x + (m + stride) * C);
#pragma unroll
            for (int o = 0; o < C * 2; o += GS * 128)
                if (o + g0 * 128 < C * 2) prefetch_l2(xn + o + g0 * 128);
        }
        if (records_pending) {                             // first token of this warp: the records have landed
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncthreads();
            records_pending = false;
        }
        // -- merged rows: a lane per row sums the entries into the row's virtual slot
        if (nslots > 0) {
            // the inline form is evaluated for every record (a longer row's record carries zero weights there), so
            // that the loads of several records are in flight together; longer rows are patched afterwards
#pragma unroll 4
            for (int vi = g0; vi < nslots; vi += GS) {
                const uint4 r0 = s_vrec[2 * vi], r1 = s_vrec[2 * vi + 1];
                float e = __uint_as_float(r0.z) * d[r0.x & 0xFFFFu];
                e = fmaf(__uint_as_float(r0.w), d[r0.x >> 16], e);
                e = fmaf(__uint_as_float(r1.x), d[r0.y & 0xFFFFu], e);
                e = fmaf(__uint_as_float(r1.y), d[r0.y >> 16], e);
                d[C + vi] = e;
            }
            if (nlong > 0) {                               // uniform over the grid; few rows
                const bool listed = nlong <= kLongRows;
                for (int k = g0; k < (listed ? nlong : nslots); k += GS) {
                    const int vi = listed ? s_lrow[k] : k;
                    const uint4 r1 = s_vrec[2 * vi + 1];
                    if (r1.z > uint32_t(kInline))
                        d[C + vi] = r1.w ? pair_row(s_lent, d, int(r1.x), int(r1.z)) : csr_row(rm, d, C, int(r1.x), int(r1.z));
                }
            }
            token_sync<G>(barid);
        }
        // -- reassembly: one gather per channel; row range
        float v[NPL];
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const int g = g0 + i * GS;
            const uint4 oa = reinterpret_cast<const uint4*>(s_offA)[g], ob = reinterpret_cast<const uint4*>(s_offB)[g];
            const float4 wa = reinterpret_cast<const float4*>(s_wA)[g], wb = reinterpret_cast<const float4*>(s_wB)[g];
            float* u = v + 8 * i;
            if (slow) {
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] = csr_channel(rm, d, C, 8 * g + j);
            } else {
            u[0] = wa.x * *reinterpret_cast<const float*>(dbytes + oa.x);
            u[1] = wa.y * *reinterpret_cast<const float*>(dbytes + oa.y);
            u[2] = wa.z * *reinterpret_cast<const float*>(dbytes + oa.z);
            u[3] = wa.w * *reinterpret_cast<const float*>(dbytes + oa.w);
            u[4] = wb.x * *reinterpret_cast<const float*>(dbytes + ob.x);
            u[5] = wb.y * *reinterpret_cast<const float*>(dbytes + ob.y);
            u[6] = wb.z * *reinterpret_cast<const float*>(dbytes + ob.z);
            u[7] = wb.w * *reinterpret_cast<const float*>(dbytes + ob.w);
            }
            if (HAS_BETA) {
                const float4 ba = reinterpret_cast<const float4*>(s_bA)[g], bb = reinterpret_cast<const float4*>(s_bB)[g];
                u[0] = fmaf(rstd, u[0], ba.x); u[1] = fmaf(rstd, u[1], ba.y);
                u[2] = fmaf(rstd, u[2], ba.z); u[3] = fmaf(rstd, u[3], ba.w);
                u[4] = fmaf(rstd, u[4], bb.x); u[5] = fmaf(rstd, u[5], bb.y);
                u[6] = fmaf(rstd, u[6], bb.z); u[7] = fmaf(rstd, u[7], bb.w);
            }
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                lo = min3(lo, u[j], u[j + 1]);
                hi = max3(hi, u[j], u[j + 1]);
            }
        }
        if (!HAS_BETA) { lo *= rstd; hi *= rstd; }         // rstd > 0: scaling commutes with min / max
        lo = redux_min(lo);
        hi = redux_max(hi);
        if (G > 1) {
            if (lane == 0) { exr[par * 2 * G + 2 * wsub] = lo; exr[par * 2 * G + 2 * wsub + 1] = hi; }
            token_sync<G>(barid);
#pragma unroll
            for (int w = 0; w < G; ++w) {
                lo = fminf(lo, exr[par * 2 * G + 2 * w]);
                hi = fmaxf(hi, exr[par * 2 * G + 2 * w + 1]);
            }
        }
        // -- Eq. 2
        float alpha = (hi - lo) * inv_qmax;
        if (!(hi > lo)) alpha = lo != 0.f ? fabsf(lo) : 1.f;
        const float inv = __frcp_rn(alpha);
        const float zero = -rintf(lo * inv);
        const bool big = fmaxf(fabsf(lo), fabsf(hi)) * inv >= 2097152.f || fabsf(zero) >= 2097152.f;
        const int zadd = int(zero) - kMagicBits;
        const float sc = HAS_BETA ? inv : rstd * inv;      // without beta v holds x' / rstd
        int csum = 0;
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const int g = g0 + i * GS;
            const float* u = v + 8 * i;
            int n[8];
            if (!big) {
#pragma unroll
                for (int j = 0; j < 8; ++j) n[j] = __float_as_int(fmaf(u[j], sc, kMagic)) + zadd;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) n[j] = int(fminf(fmaxf(rintf(u[j] * sc) + zero, 0.f), qmax));
            }
            if (PACKED) {
                uint32_t p = 0;
#pragma unroll
                for (int k = 3; k >= 0; --k) p = pack_sat_u4(n[2 * k + 1], n[2 * k], p);
                const uint32_t nib = (p & 0x0F0F0F0Fu) + ((p >> 4) & 0x0F0F0F0Fu);
                csum = int(__dp4a(nib, 0x01010101u, uint32_t(csum)));
                *reinterpret_cast<uint32_t*>(codes + m * (C / 2) + 4 * g) = p;
            } else {
                uint32_t p0 = pack_sat_u8(min(n[3], top), min(n[2], top), 0u);
                p0 = pack_sat_u8(min(n[1], top), min(n[0], top), p0);
                uint32_t p1 = pack_sat_u8(min(n[7], top), min(n[6], top), 0u);
                p1 = pack_sat_u8(min(n[5], top), min(n[4], top), p1);
                csum = int(__dp4a(p0, 0x01010101u, uint32_t(csum)));
                csum = int(__dp4a(p1, 0x01010101u, uint32_t(csum)));
                *reinterpret_cast<uint2*>(codes + m * C + 8 * g) = make_uint2(p0, p1);
            }
        }
        csum = __reduce_add_sync(0xffffffffu, csum);
        if (G == 1) {
            if (lane == 0) {
                a_scale[m] = alpha;
                a_zero[m] = zero;
                if (a_rowsum) a_rowsum[m] = csum;
            }
            __syncwarp();
        } else {
            // partial code sums meet in the parity slot that the range exchange just used; the next
            // token's first exchange uses the other parity, and its barrier orders these reads before
            // any later write of this slot
            int* exi = reinterpret_cast<int*>(exr + par * 2 * G);
            token_sync<G>(barid);                          // everyone has read the range
            if (lane == 0) exi[wsub] = csum;
            token_sync<G>(barid);
            if (wsub == 0 && lane == 0) {
                int tot = 0;
#pragma unroll
                for (int w = 0; w < G; ++w) tot += exi[w];
                a_scale[m] = alpha;
                a_zero[m] = zero;
                if (a_rowsum) a_rowsum[m] = tot;
            }
            par ^= 1;                                      // min/max exchange used parity `par`
        }
    }
    if (records_pending) {                                 // a warp without tokens still joins the CTA barrier
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
    }
}

// warps per CTA that fit with the given slot room (0: does not fit)
int warps_that_fit(int C, bool has_beta, int slot_room) {
    const int64_t rec = int64_t(has_beta ? 10 : 6) * C;
    const int64_t row = int64_t(C + slot_room) * 4;
    const int64_t w = (kSmemBudget - rec) / row;
    return int(w < 0 ? 0 : (w > kMaxWarps ? kMaxWarps : w));
}

template <typename XT, bool HAS_BETA, bool PACKED>
int launch_warp(const void* x, int64_t M, int C, float eps, int bits, const WarpImage& im, int slot_room,
                const RawMap& rm, uint8_t* codes, float* a_scale, float* a_zero, int32_t* a_rowsum,
                cudaStream_t st) {
    auto kern = reassemble_quant_warp<XT, HAS_BETA, PACKED>;
    const int wfit = warps_that_fit(C, HAS_BETA, slot_room);
    const int sms = device_sm_count();
    const int grid = int(M < sms ? M : sms);
    const int64_t per_cta = (M + grid - 1) / grid;        // tokens a CTA gets
    const int W = int(per_cta < wfit ? per_cta : wfit);
    const int row_words = C + slot_room;
    const size_t smem = size_t(HAS_BETA ? 10 : 6) * C + size_t(W) * row_words * 4;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
    kern<<<grid, 32 * W, smem, st>>>(static_cast<const XT*>(x), M, C, eps, bits, im, row_words, rm, codes, a_scale,
                                     a_zero, a_rowsum);
    return after_launch();
}


template <int NPL, int G, bool HAS_BETA, bool PACKED, int MAXW>
int launch_token(const void* x, int64_t M, float eps, int bits, const WarpImage& im, int slot_room, const RawMap& rm,
                 uint8_t* codes, float* a_scale, float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool share_sm) {
    constexpr int C = NPL * 32 * G;
    auto kern = reassemble_quant_token<NPL, G, HAS_BETA, PACKED, MAXW>;
    const int row_words = C + slot_room;
    const int64_t fixed = int64_t(HAS_BETA ? 12 : 8) * C + (MAXW / G) * 8 * G * 4 + int64_t(slot_room) * 32 +
                          kLongCap * 8 + kLongRows * 4;   // records, exchange, slot records, longer rows
    int tok_fit = int((kSmemBudget - fixed) / (int64_t(row_words) * 4));
    if (tok_fit > MAXW / G) tok_fit = MAXW / G;
    if (share_sm) {
        // leave a fifth of the register file free: the layer expands its 4-bit weights for the coming GEMM
        // on a second stream meanwhile, and that bandwidth-bound kernel needs room on every SM to keep
        // enough loads in flight (this kernel is latency-bound and does not miss the token slot)
        static int regs = 0;
        if (regs == 0) {
            cudaFuncAttributes fa;
            QLLM_CUDA_TRY(cudaFuncGetAttributes(&fa, kern));
            regs = fa.numRegs > 0 ? fa.numRegs : 128;
        }
        const int w_cap = int(0.8 * 65536 / (regs * 32));
        if (tok_fit > w_cap / G && w_cap / G >= 1) tok_fit = w_cap / G;
    }
    if (tok_fit < 1) return QLLM_ERR_UNSUPPORTED;
    const int sms = device_sm_count();
    const int grid = int(M < sms ? M : sms);
    const int64_t per_cta = (M + grid - 1) / grid;
    const int tok = int(per_cta < tok_fit ? per_cta : tok_fit);
    int W = tok * G;
    if (W < 4) W = 4;                                       // spare warps help copy the records
    const size_t smem = size_t(fixed) + size_t(tok) * row_words * 4;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
    kern<<<grid, 32 * W, smem, st>>>(static_cast<const __nv_bfloat16*>(x), M, eps, bits, im, row_words, tok, rm,
                                     codes, a_scale, a_zero, a_rowsum);
    return after_launch();
}

// Channels per lane, warps per token, most warps per CTA of the compile-time shapes (measured best).
#ifndef QLLM_RQ_4096
#define QLLM_RQ_4096 64
#define QLLM_RQ_4096_G 2
#define QLLM_RQ_4096_W 20
#endif
#ifndef QLLM_RQ_5120
#define QLLM_RQ_5120 80
#define QLLM_RQ_5120_G 2
#define QLLM_RQ_5120_W 16
#endif
#ifndef QLLM_RQ_8192
#define QLLM_RQ_8192 64
#define QLLM_RQ_8192_G 4
#define QLLM_RQ_8192_W 16
#endif

template <int NPL, int G, int MAXW>
int launch_token_variant(bool has_beta, bool packed, const void* x, int64_t M, float eps, int bits,
                         const WarpImage& im, int slot_room, const RawMap& rm, uint8_t* codes, float* a_scale,
                         float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool share_sm) {
#define QLLM_RQT(B, P) launch_token<NPL, G, B, P, MAXW>(x, M, eps, bits, im, slot_room, rm, codes, a_scale, a_zero, a_rowsum, st, share_sm)
    if (has_beta) return packed ? QLLM_RQT(true, true) : QLLM_RQT(true, false);
    return packed ? QLLM_RQT(false, true) : QLLM_RQT(false, false);
#undef QLLM_RQT
}

}  // namespace

// ---- host entry points -----------------------------------------------------------------------
// The warp kernel serves a channel count when the records (with bias terms) and at least one row with
// the full slot allowance fit into shared memory; other shapes take the shape-agnostic kernel.
static bool warp_kernel_serves(int C) {
    return C % 256 == 0 && C + kSlotCap <= 65535 && warps_that_fit(C, true, kSlotCap) >= 1;
}

bool reassemble_byte_lanes_supported(int C) { return warp_kernel_serves(C); }

size_t reassemble_map_image_bytes(int C) { return warp_kernel_serves(C) ? warp_image_bytes(C) : 0; }

int compile_reassemble_map(int C, const float* gamma, const float* beta, const int32_t* ptr, const int32_t* src,
                           const float* coef, void* image, cudaStream_t st) {
    if (!warp_kernel_serves(C)) return QLLM_ERR_UNSUPPORTED;
    const WarpImage im = warp_image_at(image, C);
    QLLM_CUDA_TRY(cudaMemsetAsync(im.head, 0, 16, st));
    compile_map_warp_kernel<<<(C + 255) / 256, 256, 0, st>>>(C, gamma, beta, ptr, src, coef, im);
    return after_launch();
}

int reassemble_map_slots(int C, const void* image, cudaStream_t st, int* slots) {
    if (!warp_kernel_serves(C)) return QLLM_ERR_UNSUPPORTED;
    const WarpImage im = warp_image_at(const_cast<void*>(image), C);
    QLLM_CUDA_TRY(cudaMemcpyAsync(slots, im.head, sizeof(int), cudaMemcpyDeviceToHost, st));
    QLLM_CUDA_TRY(cudaStreamSynchronize(st));
    return QLLM_OK;
}

int launch_reassemble_quant(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                            const float* beta, float eps, const int32_t* ptr, const int32_t* src,
                            const float* coef, int bits, const void* map_image, uint8_t* codes, float* a_scale,
                            float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool byte_lanes, int slots_known,
                            bool share_sm) {
    if (!warp_kernel_serves(C) || !gamma) {              // no LayerNorm: the shape-agnostic kernel
        if (byte_lanes && bits == 4) return QLLM_ERR_UNSUPPORTED;
        return launch_reassemble_quant_generic(x, x_dtype, M, C, gamma, beta, eps, ptr, src, coef, bits, codes,
                                               a_scale, a_zero, a_rowsum, st);
    }
    if (!map_image) {
        // direct call: compile the map for this launch into per-stream library scratch
        uint8_t* buf = nullptr;
        int rc = stream_scratch(kScratchMapImage, st, warp_image_bytes(C), &buf);
        if (rc != QLLM_OK) return rc;
        rc = compile_reassemble_map(C, gamma, beta, ptr, src, coef, buf, st);
        if (rc != QLLM_OK) return rc;
        map_image = buf;
        slots_known = -1;
    }
    const WarpImage im = warp_image_at(const_cast<void*>(map_image), C);
    int slot_room = kSlotCap;
    if (slots_known >= 0) slot_room = slots_known > kSlotCap ? 0 : ((slots_known + 3) & ~3);
    const RawMap rm{gamma, ptr, src, coef};
    const bool packed = bits == 4 && !byte_lanes, has_beta = beta != nullptr;
    if (x_dtype == QLLM_BF16) {
        // LLaMA hidden sizes: shape fixed at compile time
#define QLLM_TOKEN_ARGS has_beta, packed, x, M, eps, bits, im, slot_room, rm, codes, a_scale, a_zero, a_rowsum, st, share_sm
        if (M <= device_sm_count()) {                          // one token per CTA: spread it over more warps
            if (C == 4096) return launch_token_variant<16, 8, 8>(QLLM_TOKEN_ARGS);
            if (C == 5120) return launch_token_variant<40, 4, 4>(QLLM_TOKEN_ARGS);
            if (C == 8192) return launch_token_variant<16, 16, 16>(QLLM_TOKEN_ARGS);
        }
        if (C == 4096) return launch_token_variant<QLLM_RQ_4096, QLLM_RQ_4096_G, QLLM_RQ_4096_W>(QLLM_TOKEN_ARGS);
        if (C == 5120) return launch_token_variant<QLLM_RQ_5120, QLLM_RQ_5120_G, QLLM_RQ_5120_W>(QLLM_TOKEN_ARGS);
        if (C == 8192) return launch_token_variant<QLLM_RQ_8192, QLLM_RQ_8192_G, QLLM_RQ_8192_W>(QLLM_TOKEN_ARGS);
#undef QLLM_TOKEN_ARGS
    }
#define QLLM_RQW(XT, B, P) launch_warp<XT, B, P>(x, M, C, eps, bits, im, slot_room, rm, codes, a_scale, a_zero, a_rowsum, st)
    if (x_dtype == QLLM_BF16) {
        if (has_beta) return packed ? QLLM_RQW(__nv_bfloat16, true, true) : QLLM_RQW(__nv_bfloat16, true, false);
        return packed ? QLLM_RQW(__nv_bfloat16, false, true) : QLLM_RQW(__nv_bfloat16, false, false);
    }
    if (has_beta) return packed ? QLLM_RQW(float, true, true) : QLLM_RQW(float, true, false);
    return packed ? QLLM_RQW(float, false, true) : QLLM_RQW(float, false, false);
#undef QLLM_RQW
}

}  // namespace qllm
