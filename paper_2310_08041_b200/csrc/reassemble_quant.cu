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
//   Virtual slots, rows of two entries first (slots 0 .. n2-1), rows of three and more after them
//   (slots n2 .. n2+n34-1), each field an array of its own so that a warp reads them without bank conflicts:
//   p01 uint32[kSlotCap], w0, w1 float[kSlotCap]     pos0 | pos1 << 16 and the two weights, every slot
//   p23 uint32[kOtherCap], w2, w3 float[kOtherCap]   entries 2 and 3 of slot n2 + t (weight 0 where absent)
//   A row longer than kInline entries has zero weights in those fields and is listed in
//   lmeta int4[kLongRows]    {slot, first, n, kind}: kind 1 = entries lent[first .. first+n), kind 0 = CSR entries
//   lent uint2[kLongCap]     {position, weight bits}
//   head int[8]         [0], [3] = pairs / other rows given a slot so far (assign kernel), [1] = entries handed out in
//                       lent, [2] = rows longer than kInline listed so far, [4] = n2, [5] = n34, [6] = rows longer
//                       than kInline (count kernel)
// The slots serve a launch when n2 + n34 <= the row's slot room, n34 <= the room for p23/w2/w3 and all longer
// rows are listed; otherwise the launch walks the CSR arrays.
constexpr int kOtherCap = 1024;
struct WarpImage {
    uint16_t* idx;
    float *wlo, *whi, *blo, *bhi;
    uint32_t* p01;
    float *w0, *w1;
    uint32_t* p23;
    float *w2, *w3;
    int4* lmeta;
    uint2* lent;
    int* head;
};
__host__ __device__ inline size_t warp_image_bytes(int C) {
    return size_t(C) * 10 + size_t(kSlotCap) * 12 + size_t(kOtherCap) * 12 + size_t(kLongRows) * 16 +
           size_t(kLongCap) * 8 + 32;
}
__host__ __device__ inline WarpImage warp_image_at(void* base, int C) {
    WarpImage im;
    uint8_t* b = static_cast<uint8_t*>(base);
    im.idx = reinterpret_cast<uint16_t*>(b);
    im.wlo = reinterpret_cast<float*>(b + size_t(C) * 2);
    im.whi = im.wlo + C / 2;
    im.blo = im.whi + C / 2;
    im.bhi = im.blo + C / 2;
    im.p01 = reinterpret_cast<uint32_t*>(im.bhi + C / 2);
    im.w0 = reinterpret_cast<float*>(im.p01 + kSlotCap);
    im.w1 = im.w0 + kSlotCap;
    im.p23 = reinterpret_cast<uint32_t*>(im.w1 + kSlotCap);
    im.w2 = reinterpret_cast<float*>(im.p23 + kOtherCap);
    im.w3 = im.w2 + kOtherCap;
    im.lmeta = reinterpret_cast<int4*>(im.w3 + kOtherCap);
    im.lent = reinterpret_cast<uint2*>(im.lmeta + kLongRows);
    im.head = reinterpret_cast<int*>(im.lent + kLongCap);
    return im;
}

__device__ __forceinline__ bool slots_fit(const int* head, int slot_room, int other_room) {
    return head[4] + head[5] <= slot_room && head[5] <= other_room && head[6] <= kLongRows;
}

// Pass 1: how many rows have two entries, how many more.  head must be zero at launch.
__global__ void __launch_bounds__(256)
count_rows_kernel(int C, const int32_t* __restrict__ ptr, WarpImage im) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    const int n = __ldg(ptr + c + 1) - __ldg(ptr + c);
    if (n == 2) atomicAdd(im.head + 4, 1);
    else if (n > 2) atomicAdd(im.head + 5, 1);
    if (n > kInline) atomicAdd(im.head + 6, 1);
}

// Pass 2: one thread per output channel writes its record and, for a multi-entry row, its slot.
__global__ void __launch_bounds__(256)
compile_map_warp_kernel(int C, const float* __restrict__ gamma, const float* __restrict__ beta,
                        const int32_t* __restrict__ ptr, const int32_t* __restrict__ src,
                        const float* __restrict__ coef, WarpImage im) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    const int n2 = im.head[4], n34 = im.head[5];
    const bool fits = slots_fit(im.head, kSlotCap, kOtherCap);
    const int j0 = __ldg(ptr + c), n = __ldg(ptr + c + 1) - j0;
    const int s0 = __ldg(src + j0);
    const float c0 = __ldg(coef + j0);
    uint32_t pos = uint32_t(dplane(s0, C));
    float w = c0 * __ldg(gamma + s0);
    float b = beta ? c0 * __ldg(beta + s0) : 0.f;
    if (n > 1) {                                          // merged row
        if (beta)
            for (int j = j0 + 1; j < j0 + n; ++j) b = fmaf(__ldg(coef + j), __ldg(beta + __ldg(src + j)), b);
        if (fits) {
            uint32_t o[kInline] = {0, 0, 0, 0};
            float ww[kInline] = {0.f, 0.f, 0.f, 0.f};
            if (n <= kInline)
                for (int e = 0; e < n; ++e) {
                    const int sj = __ldg(src + j0 + e);
                    o[e] = uint32_t(dplane(sj, C));
                    ww[e] = __ldg(coef + j0 + e) * __ldg(gamma + sj);
                }
            int slot;
            if (n == 2) {
                slot = atomicAdd(im.head, 1);
            } else {
                const int t = atomicAdd(im.head + 3, 1);
                slot = n2 + t;
                im.p23[t] = o[2] | (o[3] << 16);
                im.w2[t] = ww[2];
                im.w3[t] = ww[3];
            }
            im.p01[slot] = o[0] | (o[1] << 16);
            im.w0[slot] = ww[0];
            im.w1[slot] = ww[1];
            if (n > kInline) {
                int first = atomicAdd(im.head + 1, n), kind = 1;
                if (first + n <= kLongCap) {              // entries as (position, weight) pairs for shared memory
                    for (int e = 0; e < n; ++e) {
                        const int sj = __ldg(src + j0 + e);
                        im.lent[first + e] = make_uint2(uint32_t(dplane(sj, C)),
                                                        __float_as_uint(__ldg(coef + j0 + e) * __ldg(gamma + sj)));
                    }
                } else {                                  // walks the CSR arrays at run time
                    first = j0;
                    kind = 0;
                }
                const int li = atomicAdd(im.head + 2, 1);
                if (li < kLongRows) im.lmeta[li] = make_int4(slot, first, n, kind);
            }
            pos = uint32_t(C + slot);
            w = 1.0f;
        }
    }
    im.idx[c] = uint16_t(pos);
    const int g = c >> 3, j = c & 7;
    (j < 4 ? im.wlo : im.whi)[4 * g + (j & 3)] = w;
    (j < 4 ? im.blo : im.bhi)[4 * g + (j & 3)] = b;
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
    const bool slow = !slots_fit(im.head, row_words - C, kOtherCap);   // uniform over the grid
    const int n2 = slow ? 0 : __ldg(im.head + 4);
    const int nslots = slow ? 0 : n2 + __ldg(im.head + 5);
    const int nlong = slow ? 0 : __ldg(im.head + 6);
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
            const uint32_t p = __ldg(im.p01 + vi);
            float e = __ldg(im.w0 + vi) * d[p & 0xFFFFu];
            e = fmaf(__ldg(im.w1 + vi), d[p >> 16], e);
            if (vi >= n2) {
                const uint32_t q = __ldg(im.p23 + vi - n2);
                e = fmaf(__ldg(im.w2 + vi - n2), d[q & 0xFFFFu], e);
                e = fmaf(__ldg(im.w3 + vi - n2), d[q >> 16], e);
            }
            d[C + vi] = e;
        }
        if (nlong > 0) __syncwarp();                           // another lane wrote this slot's record value just above
        for (int k = lane; k < nlong; k += 32) {               // the few rows longer than a record
            const int4 lm = __ldg(im.lmeta + k);
            d[C + lm.x] = lm.w ? pair_row(im.lent, d, lm.y, lm.z) : csr_row(rm, d, C, lm.y, lm.z);
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
// Positions stay 16-bit and slot records are split by field (and by row length) in shared memory: what limits
// the kernel is the number of shared-memory wavefronts per token and the tokens that fit beside the records.
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
                       int row_words, int other_room, int TOK /* tokens in flight per CTA */, RawMap rm,
                       uint8_t* __restrict__ codes, float* __restrict__ a_scale,
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
    uint16_t* s_idx = reinterpret_cast<uint16_t*>(HAS_BETA ? s_bB + C / 2 : s_bA);     // [C] word positions
    float* s_ex = reinterpret_cast<float*>(s_idx + C);                  // [MAXW / G][8 G] exchange words per token slot
    const int slot_room = row_words - C;
    uint32_t* s_p01 = reinterpret_cast<uint32_t*>(s_ex + (MAXW / G) * 8 * G);   // slot records, field by field
    float* s_w0 = reinterpret_cast<float*>(s_p01 + slot_room);
    float* s_w1 = s_w0 + slot_room;
    uint32_t* s_p23 = reinterpret_cast<uint32_t*>(s_w1 + slot_room);
    float* s_w2 = reinterpret_cast<float*>(s_p23 + other_room);
    float* s_w3 = s_w2 + other_room;
    int4* s_lmeta = reinterpret_cast<int4*>(s_w3 + other_room);                 // [kLongRows] rows longer than a record
    uint2* s_lent = reinterpret_cast<uint2*>(s_lmeta + kLongRows);              // [kLongCap] their entries
    float* rows = reinterpret_cast<float*>(s_lent + kLongCap);

    // a kernel launched as this one's programmatic dependent (the decode GEMM) may start its prologue now
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
        auto copy16 = [&](void* dst, const void* src, int n16) {
            for (int i = threadIdx.x; i < n16; i += blockDim.x)
                cp_async16(static_cast<uint4*>(dst) + i, static_cast<const uint4*>(src) + i);
        };
        copy16(s_idx, im.idx, 2 * C / 16);
        copy16(s_p01, im.p01, slot_room / 4);
        copy16(s_w0, im.w0, slot_room / 4);
        copy16(s_w1, im.w1, slot_room / 4);
        copy16(s_p23, im.p23, other_room / 4);
        copy16(s_w2, im.w2, other_room / 4);
        copy16(s_w3, im.w3, other_room / 4);
        copy16(s_lmeta, im.lmeta, kLongRows);
        copy16(s_lent, im.lent, kLongCap / 2);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const bool slow = !slots_fit(im.head, slot_room, other_room);   // uniform over the grid: walk the CSR arrays
    const int n2 = slow ? 0 : __ldg(im.head + 4);          // slots of two-entry rows come first
    const int nslots = slow ? 0 : n2 + __ldg(im.head + 5);
    const int nlong = slow ? 0 : __ldg(im.head + 6);       // rows longer than a slot record
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
            // two-entry rows first, then the rows with entries 2 and 3 (only the warp step that straddles n2 diverges);
            // a longer row's record carries zero weights and is patched afterwards
#pragma unroll 4
            for (int vi = g0; vi < nslots; vi += GS) {
                const uint32_t p = s_p01[vi];
                float e = s_w0[vi] * d[p & 0xFFFFu];
                e = fmaf(s_w1[vi], d[p >> 16], e);
                if (vi >= n2) {
                    const uint32_t q = s_p23[vi - n2];
                    e = fmaf(s_w2[vi - n2], d[q & 0xFFFFu], e);
                    e = fmaf(s_w3[vi - n2], d[q >> 16], e);
                }
                d[C + vi] = e;
            }
            if (nlong > 0) token_sync<G>(barid);           // another lane wrote this slot's record value just above
            for (int k = g0; k < nlong; k += GS) {         // few rows
                const int4 lm = s_lmeta[k];
                d[C + lm.x] = lm.w ? pair_row(s_lent, d, lm.y, lm.z) : csr_row(rm, d, C, lm.y, lm.z);
            }
            token_sync<G>(barid);
        }
        // -- reassembly: one gather per channel; row range
        float v[NPL];
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const int g = g0 + i * GS;
            const uint4 iw = reinterpret_cast<const uint4*>(s_idx)[g];     // 8 word positions
            const float4 wa = reinterpret_cast<const float4*>(s_wA)[g], wb = reinterpret_cast<const float4*>(s_wB)[g];
            float* u = v + 8 * i;
            if (slow) {
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] = csr_channel(rm, d, C, 8 * g + j);
            } else {
            u[0] = wa.x * d[iw.x & 0xFFFFu]; u[1] = wa.y * d[iw.x >> 16];
            u[2] = wa.z * d[iw.y & 0xFFFFu]; u[3] = wa.w * d[iw.y >> 16];
            u[4] = wb.x * d[iw.z & 0xFFFFu]; u[5] = wb.y * d[iw.z >> 16];
            u[6] = wb.z * d[iw.w & 0xFFFFu]; u[7] = wb.w * d[iw.w >> 16];
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
int launch_token(const void* x, int64_t M, float eps, int bits, const WarpImage& im, int slot_room, int other_room,
                 const RawMap& rm,
                 uint8_t* codes, float* a_scale, float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool share_sm) {
    constexpr int C = NPL * 32 * G;
    auto kern = reassemble_quant_token<NPL, G, HAS_BETA, PACKED, MAXW>;
    const int row_words = C + slot_room;
    // weights (+ bias), positions, exchange words, slot records field by field, longer rows
    const int64_t fixed = int64_t(HAS_BETA ? 8 : 4) * C + 2 * C + (MAXW / G) * 8 * G * 4 + int64_t(slot_room) * 12 +
                          int64_t(other_room) * 12 + kLongRows * 16 + kLongCap * 8;
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
    // the fewest rounds that the token slots allow, then the fewest slots that still make those rounds: every
    // round is equally full on every SM (2048 tokens on 148 SMs: two rounds of 7 instead of 8 + 6 on some SMs and
    // 8 + 0 on others), and a slot less leaves its share of shared-memory bandwidth to the others
    const int64_t rounds = (per_cta + tok_fit - 1) / tok_fit;
    const int tok = int((per_cta + rounds - 1) / rounds);
    int W = tok * G;
    if (W < 4) W = 4;                                       // spare warps help copy the records
    const size_t smem = size_t(fixed) + size_t(tok) * row_words * 4;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
    kern<<<grid, 32 * W, smem, st>>>(static_cast<const __nv_bfloat16*>(x), M, eps, bits, im, row_words, other_room, tok, rm,
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
                         const WarpImage& im, int slot_room, int other_room, const RawMap& rm, uint8_t* codes,
                         float* a_scale,
                         float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool share_sm) {
#define QLLM_RQT(B, P) launch_token<NPL, G, B, P, MAXW>(x, M, eps, bits, im, slot_room, other_room, rm, codes, a_scale, a_zero, a_rowsum, st, share_sm)
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
    QLLM_CUDA_TRY(cudaMemsetAsync(im.head, 0, 32, st));
    count_rows_kernel<<<(C + 255) / 256, 256, 0, st>>>(C, ptr, im);
    compile_map_warp_kernel<<<(C + 255) / 256, 256, 0, st>>>(C, gamma, beta, ptr, src, coef, im);
    return after_launch(2);
}

int reassemble_map_slots(int C, const void* image, cudaStream_t st, int* slots) {
    if (!warp_kernel_serves(C)) return QLLM_ERR_UNSUPPORTED;
    const WarpImage im = warp_image_at(const_cast<void*>(image), C);
    int head[8];
    QLLM_CUDA_TRY(cudaMemcpyAsync(head, im.head, sizeof(head), cudaMemcpyDeviceToHost, st));
    QLLM_CUDA_TRY(cudaStreamSynchronize(st));
    // rows with two entries + rows with more, and the latter again in the upper half; -1 (unknown: the launcher
    // then assumes the largest image) when the image's slots cannot serve a launch anyway
    const bool fits = head[4] + head[5] <= kSlotCap && head[5] <= kOtherCap && head[6] <= kLongRows;
    *slots = fits ? ((head[5] << 16) | (head[4] + head[5])) : -1;
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
    // room for slot records and slot values: exact when the caller knows the image's counts, else the largest
    // image's total with a quarter of it for rows of three and more entries (an image beyond the room makes the
    // launch walk the CSR arrays)
    int slot_room = kSlotCap, other_room = kSlotCap / 4;
    if (slots_known >= 0) {
        slot_room = ((slots_known & 0xFFFF) + 3) & ~3;
        other_room = ((slots_known >> 16) + 3) & ~3;
    }
    const RawMap rm{gamma, ptr, src, coef};
    const bool packed = bits == 4 && !byte_lanes, has_beta = beta != nullptr;
    if (x_dtype == QLLM_BF16) {
        // LLaMA hidden sizes: shape fixed at compile time
#define QLLM_TOKEN_ARGS has_beta, packed, x, M, eps, bits, im, slot_room, other_room, rm, codes, a_scale, a_zero, a_rowsum, st, share_sm
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
