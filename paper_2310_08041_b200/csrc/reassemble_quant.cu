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
#include "reassemble_quant_common.cuh"

namespace qllm {

namespace {

constexpr int kMaxWarps = 16;

// position of channel k in a warp's row
__host__ __device__ __forceinline__ int dplane(int k, int C) { return (k & 7) * (C >> 3) + (k >> 3); }

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


}  // namespace

// ---- host entry points -----------------------------------------------------------------------
// The warp kernel serves a channel count when the records (with bias terms) and at least one row with
// the full slot allowance fit into shared memory; other shapes take the shape-agnostic kernel.  bf16 rows
// of the LLaMA hidden sizes take the token kernel (reassemble_quant_token.cu), which has its own image.
static bool warp_kernel_serves(int C) {
    return C % 256 == 0 && C + kSlotCap <= 65535 && warps_that_fit(C, true, kSlotCap) >= 1;
}
static bool token_path(int C, int x_dtype) { return x_dtype == QLLM_BF16 && token_kernel_serves(C); }

bool reassemble_byte_lanes_supported(int C) { return warp_kernel_serves(C); }

// Token path: the image is the token kernel's, followed by the warp kernel's (used when the token kernel cannot
// serve the map: slots beyond its limits, or source channels read by several rows with different coefficients).
size_t reassemble_map_image_bytes(int C, int x_dtype) {
    if (token_path(C, x_dtype)) return token_image_bytes(C) + warp_image_bytes(C);
    return warp_kernel_serves(C) ? warp_image_bytes(C) : 0;
}

static int compile_warp_map(int C, const float* gamma, const float* beta, const int32_t* ptr, const int32_t* src,
                            const float* coef, void* image, cudaStream_t st) {
    const WarpImage im = warp_image_at(image, C);
    QLLM_CUDA_TRY(cudaMemsetAsync(im.head, 0, 32, st));
    count_rows_kernel<<<(C + 255) / 256, 256, 0, st>>>(C, ptr, im);
    compile_map_warp_kernel<<<(C + 255) / 256, 256, 0, st>>>(C, gamma, beta, ptr, src, coef, im);
    return after_launch(2);
}

int compile_reassemble_map(int C, int x_dtype, const float* gamma, const float* beta, const int32_t* ptr,
                           const int32_t* src, const float* coef, void* image, cudaStream_t st) {
    if (token_path(C, x_dtype)) {
        const int rc = compile_token_map(C, gamma, beta, ptr, src, coef, image, st);
        if (rc != QLLM_OK) return rc;
        return compile_warp_map(C, gamma, beta, ptr, src, coef, static_cast<uint8_t*>(image) + token_image_bytes(C), st);
    }
    if (!warp_kernel_serves(C)) return QLLM_ERR_UNSUPPORTED;
    return compile_warp_map(C, gamma, beta, ptr, src, coef, image, st);
}

int reassemble_map_counts(int C, int x_dtype, const void* image, cudaStream_t st, MapCounts* out) {
    if (token_path(C, x_dtype)) return token_map_counts(C, image, st, out);
    if (!warp_kernel_serves(C)) return QLLM_ERR_UNSUPPORTED;
    const WarpImage im = warp_image_at(const_cast<void*>(image), C);
    int head[8];
    QLLM_CUDA_TRY(cudaMemcpyAsync(head, im.head, sizeof(head), cudaMemcpyDeviceToHost, st));
    QLLM_CUDA_TRY(cudaStreamSynchronize(st));
    MapCounts mc;
    mc.known = true;
    mc.slots = head[4] + head[5];
    mc.other = head[5];
    mc.long_rows = head[6];
    mc.long_entries = head[1] <= kLongCap ? head[1] : kLongCap;
    mc.fits = mc.slots <= kSlotCap && mc.other <= kOtherCap && mc.long_rows <= kLongRows;
    *out = mc;
    return QLLM_OK;
}

int launch_reassemble_quant(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                            const float* beta, float eps, const int32_t* ptr, const int32_t* src,
                            const float* coef, int bits, const void* map_image, uint8_t* codes, float* a_scale,
                            float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool byte_lanes, const MapCounts* counts,
                            bool share_sm) {
    if (!warp_kernel_serves(C) || !gamma) {              // no LayerNorm: the shape-agnostic kernel
        if (byte_lanes && bits == 4) return QLLM_ERR_UNSUPPORTED;
        return launch_reassemble_quant_generic(x, x_dtype, M, C, gamma, beta, eps, ptr, src, coef, bits, codes,
                                               a_scale, a_zero, a_rowsum, st);
    }
    MapCounts mc;                                          // unknown unless the caller compiled the image before
    if (map_image && counts) mc = *counts;
    if (token_path(C, x_dtype)) {
        if (!map_image) {
            // direct call: the map is compiled into per-stream library scratch by one launch ahead of the kernel,
            // which first hashes the map, gamma and beta and leaves the image alone when it was made from the
            // same contents (the key sits at the start of the scratch; whatever else writes the scratch resets
            // it); the token kernel serves the image if the image says it can, else the shape-agnostic kernel
            // behind it does
            uint8_t* buf = nullptr;
            int rc = stream_scratch(kScratchMapImage, st, kMapScratchHeader + token_image_bytes(C), &buf);
            if (rc != QLLM_OK) return rc;
            rc = compile_token_map(C, gamma, beta, ptr, src, coef, buf + kMapScratchHeader, st,
                                   reinterpret_cast<uint64_t*>(buf));
            if (rc != QLLM_OK) return rc;
            buf += kMapScratchHeader;
            rc = launch_reassemble_quant_token(x, M, C, gamma, beta, eps, ptr, src, coef, bits, buf, MapCounts(), codes,
                                               a_scale, a_zero, a_rowsum, st, false, share_sm);
            if (rc != QLLM_OK) return rc;
            return launch_reassemble_quant_generic(x, x_dtype, M, C, gamma, beta, eps, ptr, src, coef, bits, codes,
                                                   a_scale, a_zero, a_rowsum, st, token_image_served_flag(C, buf));
        }
        if (mc.known && mc.fits)
            return launch_reassemble_quant_token(x, M, C, gamma, beta, eps, ptr, src, coef, bits, map_image, mc, codes,
                                                 a_scale, a_zero, a_rowsum, st, byte_lanes, share_sm);
        // the token kernel cannot serve this map: the warp kernel with its own image (counts not read back)
        map_image = static_cast<const uint8_t*>(map_image) + token_image_bytes(C);
        mc = MapCounts();
    }
    if (!map_image) {
        // direct call: compile the map for this launch into per-stream library scratch
        uint8_t* buf = nullptr;
        int rc = stream_scratch(kScratchMapImage, st, kMapScratchHeader + warp_image_bytes(C), &buf);
        if (rc != QLLM_OK) return rc;
        QLLM_CUDA_TRY(cudaMemsetAsync(buf, 0, 16, st));     // no token-kernel image is in the scratch any more
        buf += kMapScratchHeader;
        rc = compile_warp_map(C, gamma, beta, ptr, src, coef, buf, st);
        if (rc != QLLM_OK) return rc;
        map_image = buf;
    }
    const WarpImage im = warp_image_at(const_cast<void*>(map_image), C);
    // room for slot records and slot values: exact when the caller knows the image's counts, else the largest
    // image's total (an image beyond the room makes the launch walk the CSR arrays)
    int slot_room = kSlotCap;
    if (mc.known && mc.fits) slot_room = (mc.slots + 3) & ~3;
    const RawMap rm{gamma, ptr, src, coef};
    const bool packed = bits == 4 && !byte_lanes, has_beta = beta != nullptr;
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
