// Fused pre-GEMM kernel: LayerNorm -> channel reassembly -> per-token asymmetric
// quantization (QLLM Eq. 2-4; the fusion the paper leaves as future work, Sec. 6).
//
// HBM-bound: every token row of x is read once and its codes written once.  Design:
//  * persistent CTAs, C / CPT threads each; a thread owns CPT output channels for every
//    token its CTA processes, so the reassembly map is read ONCE per CTA into registers:
//    per channel the first two entries (source offset, coefficient * gamma) and the bias
//    term sum_j coef_j * beta[src_j].  Per token the only shared-memory traffic is the
//    centred row d = x - mean (written once, 4 B / channel) and the gathers from it.
//        x'_c = rstd * sum_j (coef_j gamma[src_j]) d[src_j] + sum_j coef_j beta[src_j]
//    Rows with more than two entries (a channel that absorbed several others) add their
//    tail from the CSR arrays in a short per-thread loop.
//  * 128-bit coalesced loads of the row, next row prefetched into registers.
//  * ownership is by channel pairs (2p, 2p+1), p = t + NT*i, so a thread packs whole bytes
//    of 4-bit codes; lanes 16-31 keep their pairs swapped in registers so that the two
//    gathers of a pair hit different banks across the two half-warps.
//  * three CTA reductions per token (sum, sum of squares, min/max) through shared memory,
//    parity-double-buffered so each costs one barrier.
//  * rounding by the 1.5 * 2^23 magic constant (nearest-even, as cvt.rni), saturating
//    cvt.pack for the clamp and the nibble / byte packing.
// Shapes outside the specialisation (C not a multiple of 32*CPT, C > 8192) take the
// shape-agnostic kernel.

#include <cuda_bf16.h>

#include <mutex>
#include <vector>

#include "common.h"
#include "device_utils.cuh"

namespace qllm {

namespace {

constexpr int kVirt = 2048;                    // virtual slots (rows with more than one entry)
constexpr int kVirtEntries = 4;                // entries a virtual-slot record can hold
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23
constexpr int kMagicBits = 0x4B400000;

// Position of channel k in the shared-memory row: even channels in the first half, odd channels in the
// second, so that the gathers of the even (odd) channels of consecutive pairs walk consecutive banks.
__device__ __forceinline__ int dpos(int k, int C) { return (k >> 1) + (k & 1) * (C >> 1); }

template <typename XT> struct RowLoad;
template <> struct RowLoad<__nv_bfloat16> { static constexpr int PER_CHUNK = 8; };
template <> struct RowLoad<float> { static constexpr int PER_CHUNK = 4; };

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

// Sum over the CTA of one value per warp already stored in red[0..nw4) (zero padded to a
// multiple of four).  Same order in every thread, so all threads hold identical bits.
__device__ __forceinline__ float sum_of(const float* red, int nw4) {
    float s = 0.f;
    for (int w = 0; w < nw4; w += 4) {
        const float4 q = *reinterpret_cast<const float4*>(red + w);
        s += (q.x + q.y) + (q.z + q.w);
    }
    return s;
}

// Compiled form of the reassembly map for one thread layout (CPT channels per thread, NT threads):
//   rec[slot * NT + t] = {byte offset into d, weight, bias, flags}  flags bit 0: the row takes the
//                        per-thread CSR fallback (entries 1.. are added from the raw map)
//   vrec[2 vi], [2 vi + 1] = virtual slot vi: {offsets 0|1, offsets 2|3, w0, w1}, {w2, w3, n, 0}
//   head[0] = virtual slots handed out (a counter; readers clamp it to kVirt)
// Built by compile_map_kernel and loaded by the main kernel with coalesced 128-bit loads; the layer
// object builds it once, direct calls build it per call.
struct MapImage {
    uint4* rec;
    uint4* vrec;
    int* head;
};
__host__ __device__ inline size_t map_image_bytes(int cpt, int nt) {
    return size_t(cpt) * nt * 16 + size_t(kVirt) * 32 + 16;
}
__host__ __device__ inline MapImage map_image_at(void* base, int cpt, int nt) {
    MapImage im;
    im.rec = static_cast<uint4*>(base);
    im.vrec = im.rec + size_t(cpt) * nt;
    im.head = reinterpret_cast<int*>(im.vrec + 2 * size_t(kVirt));
    return im;
}

// One warp per CTA so that the dependent load rounds of all NT threads run on many SMs at once.
// im.head[0] must be zero at launch.
template <int CPT>
__global__ void __launch_bounds__(32)
compile_map_kernel(int C, int NT, const float* __restrict__ gamma, const float* __restrict__ beta,
                   const int32_t* __restrict__ ptr, const int32_t* __restrict__ src,
                   const float* __restrict__ coef, MapImage im) {
    const int t = blockIdx.x * 32 + threadIdx.x;
    int j0[CPT], len[CPT];
#pragma unroll
    for (int slot = 0; slot < CPT; ++slot) {
        const int c = 2 * (t + NT * (slot >> 1)) + (slot & 1);
        j0[slot] = __ldg(ptr + c);
        len[slot] = __ldg(ptr + c + 1) - j0[slot];
    }
    int s0[CPT];
    float c0[CPT];
#pragma unroll
    for (int slot = 0; slot < CPT; ++slot) {
        s0[slot] = __ldg(src + j0[slot]);
        c0[slot] = __ldg(coef + j0[slot]);
    }
#pragma unroll
    for (int slot = 0; slot < CPT; ++slot) {
        uint32_t off = uint32_t(dpos(s0[slot], C) * 4);
        float w = c0[slot] * __ldg(gamma + s0[slot]);
        float b = beta ? c0[slot] * __ldg(beta + s0[slot]) : 0.f;
        uint32_t flags = 0;
        const int n = len[slot];
        if (n > 1) {                                  // merged row (short loops, minority of rows)
            if (beta)
                for (int j = j0[slot] + 1; j < j0[slot] + n; ++j)
                    b = fmaf(__ldg(coef + j), __ldg(beta + __ldg(src + j)), b);
            const int vi = n <= kVirtEntries ? atomicAdd(im.head, 1) : kVirt;
            if (vi < kVirt) {
                uint32_t o[kVirtEntries] = {0, 0, 0, 0};
                float ww[kVirtEntries] = {0.f, 0.f, 0.f, 0.f};
                for (int e = 0; e < n; ++e) {
                    const int sj = __ldg(src + j0[slot] + e);
                    o[e] = uint32_t(dpos(sj, C) * 4);
                    ww[e] = __ldg(coef + j0[slot] + e) * __ldg(gamma + sj);
                }
                im.vrec[2 * vi] = make_uint4(o[0] | (o[1] << 16), o[2] | (o[3] << 16), __float_as_uint(ww[0]),
                                             __float_as_uint(ww[1]));
                im.vrec[2 * vi + 1] = make_uint4(__float_as_uint(ww[2]), __float_as_uint(ww[3]), uint32_t(n), 0u);
                off = uint32_t((C + vi) * 4);
                w = 1.0f;
            } else {
                flags = 1;                            // first entry in registers, the rest from the CSR
            }
        }
        im.rec[slot * NT + t] = make_uint4(off, __float_as_uint(w), __float_as_uint(b), flags);
    }
}

template <int CPT, int NTT, typename XT, bool HAS_BETA, bool FOURBIT>
__global__ void __launch_bounds__(NTT ? NTT : 512, (NTT && NTT <= 256) ? 3 : 1)
reassemble_quant_fast(const XT* __restrict__ x, int64_t M, int C, const float* __restrict__ gamma,
                      float eps, const int32_t* __restrict__ ptr, const int32_t* __restrict__ src,
                      const float* __restrict__ coef, int bits, MapImage im,
                      uint8_t* __restrict__ codes, float* __restrict__ a_scale, float* __restrict__ a_zero,
                      int32_t* __restrict__ a_rowsum) {
    constexpr int PER = RowLoad<XT>::PER_CHUNK;
    constexpr int NCH = CPT / PER;               // 16-byte chunks of the row per thread
    constexpr int NP = CPT / 2;                  // channel pairs per thread
    extern __shared__ __align__(16) uint8_t smem_bytes[];
    float* red = reinterpret_cast<float*>(smem_bytes);         // [2][4][32] per-warp partials
    int* redi = reinterpret_cast<int*>(red + 2 * 4 * 32);      // [2][32] code-sum partials
    float* d = reinterpret_cast<float*>(redi + 2 * 32);        // [C + kVirt] centred row + virtual slots

    const int t = threadIdx.x, NT = NTT ? NTT : int(blockDim.x), lane = t & 31, warp = t >> 5;
    const int nw = NT >> 5, nw4 = (nw + 3) & ~3;
    const float invC = 1.0f / float(C);
    const float qmax = float((1 << bits) - 1);
    const float inv_qmax = 1.0f / qmax;

    // ---- compiled map -> registers (once per CTA, coalesced) -----------------------------
    uint32_t off[CPT];
    float wgt[CPT], bias[HAS_BETA ? CPT : 1];
    uint32_t fallback = 0;                       // bit per slot: the row continues in the raw CSR
#pragma unroll
    for (int slot = 0; slot < CPT; ++slot) {
        const uint4 r = __ldg(im.rec + slot * NT + t);
        off[slot] = r.x;
        wgt[slot] = __uint_as_float(r.y);
        if (HAS_BETA) bias[slot] = __uint_as_float(r.z);
        fallback |= (r.w & 1u) << slot;
    }
    const int nvirt = min(__ldg(im.head), kVirt);
    for (int i = t; i < 2 * 4 * 32 + 2 * 32; i += NT) red[i] = 0.f;   // zero bit pattern for redi too
    const char* dbytes = reinterpret_cast<const char*>(d);

    // ---- token loop ---------------------------------------------------------------------
    uint4 raw[NCH];
    int64_t m = blockIdx.x;
    if (m < M) {
#pragma unroll
        for (int j = 0; j < NCH; ++j)
            raw[j] = *reinterpret_cast<const uint4*>(x + m * C + PER * (t + NT * j));
    }
    __syncthreads();
    int par = 0;
    int64_t m_prev = -1;
    for (; m < M; m += gridDim.x, par ^= 1) {
        float* rsum = red + par * 128;
        float* rsq = rsum + 32;
        float* rlo = rsum + 64;
        float* rhi = rsum + 96;
        // -- row to fp32, mean
        float xv[CPT];
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            if constexpr (PER == 8) {
                const uint32_t w[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    xv[8 * j + 2 * k] = __uint_as_float(w[k] << 16);
                    xv[8 * j + 2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
                }
            } else {
                xv[4 * j] = __uint_as_float(raw[j].x); xv[4 * j + 1] = __uint_as_float(raw[j].y);
                xv[4 * j + 2] = __uint_as_float(raw[j].z); xv[4 * j + 3] = __uint_as_float(raw[j].w);
            }
        }
        const int64_t m_next = m + gridDim.x;
        if (m_next < M) {
#pragma unroll
            for (int j = 0; j < NCH; ++j)
                raw[j] = *reinterpret_cast<const uint4*>(x + m_next * C + PER * (t + NT * j));
        }
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < CPT; ++i) s += xv[i];
        s = warp_sum(s);
        if (lane == 0) rsum[warp] = s;
        __syncthreads();                                               // S1
        const float mean = sum_of(rsum, nw4) * invC;
        if (t == 0 && m_prev >= 0 && a_rowsum) {                       // code sum of the previous token
            const int* ri = redi + (par ^ 1) * 32;
            int tot = 0;
            for (int w = 0; w < nw; ++w) tot += ri[w];
            a_rowsum[m_prev] = tot;
        }
        // -- centred row to shared memory, variance
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < CPT; ++i) {
            xv[i] -= mean;
            sq = fmaf(xv[i], xv[i], sq);
        }
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            // channels PER*u .. PER*u + PER-1: even ones to d[PER/2 * u ..], odd ones to d[C/2 + PER/2 * u ..]
            const int u = t + NT * j;
            float* ev = d + (PER / 2) * u;
            float* od = ev + (C >> 1);
            if constexpr (PER == 8) {
                *reinterpret_cast<float4*>(ev) = make_float4(xv[8 * j], xv[8 * j + 2], xv[8 * j + 4], xv[8 * j + 6]);
                *reinterpret_cast<float4*>(od) = make_float4(xv[8 * j + 1], xv[8 * j + 3], xv[8 * j + 5], xv[8 * j + 7]);
            } else {
                *reinterpret_cast<float2*>(ev) = make_float2(xv[4 * j], xv[4 * j + 2]);
                *reinterpret_cast<float2*>(od) = make_float2(xv[4 * j + 1], xv[4 * j + 3]);
            }
        }
        sq = warp_sum(sq);
        if (lane == 0) rsq[warp] = sq;
        __syncthreads();                                               // S2: d visible
        const float var = sum_of(rsq, nw4) * invC;
        const float rstd = rsqrtf(var + eps);        // a common factor of the whole row: its last-bit
                                                     // error rescales alpha with the row, codes unchanged
        // -- merged rows: one thread per row sums its entries into the row's virtual slot
        if (nvirt > 0) {                             // uniform over the CTA
            for (int vi = t; vi < nvirt; vi += NT) {
                const uint4 r0 = __ldg(im.vrec + 2 * vi), r1 = __ldg(im.vrec + 2 * vi + 1);
                float e = __uint_as_float(r0.z) * *reinterpret_cast<const float*>(dbytes + (r0.x & 0xFFFFu));
                e = fmaf(__uint_as_float(r0.w), *reinterpret_cast<const float*>(dbytes + (r0.x >> 16)), e);
                if (r1.z > 2u) {
                    e = fmaf(__uint_as_float(r1.x), *reinterpret_cast<const float*>(dbytes + (r0.y & 0xFFFFu)), e);
                    if (r1.z > 3u)
                        e = fmaf(__uint_as_float(r1.y), *reinterpret_cast<const float*>(dbytes + (r0.y >> 16)), e);
                }
                d[C + vi] = e;
            }
            __syncthreads();                                           // S2b
        }
        // -- reassembly: one gather per channel with the register-resident map
        float v[CPT];
#pragma unroll
        for (int slot = 0; slot < CPT; ++slot)
            v[slot] = wgt[slot] * *reinterpret_cast<const float*>(dbytes + off[slot]);
        if (fallback) {                                                // rows beyond the virtual slots (rare)
            for (uint32_t fb = fallback; fb; fb &= fb - 1) {
                const int slot = __ffs(int(fb)) - 1;
                const int c = 2 * (t + NT * (slot >> 1)) + (slot & 1);
                float e = 0.f;
                for (int j = ptr[c] + 1; j < ptr[c + 1]; ++j) {
                    const int sj = src[j];
                    e = fmaf(coef[j] * gamma[sj], d[dpos(sj, C)], e);
                }
#pragma unroll
                for (int q = 0; q < CPT; ++q)
                    if (q == slot) v[q] += e;
            }
        }
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int slot = 0; slot < CPT; slot += 2) {
            v[slot] = HAS_BETA ? fmaf(rstd, v[slot], bias[slot]) : rstd * v[slot];
            v[slot + 1] = HAS_BETA ? fmaf(rstd, v[slot + 1], bias[slot + 1]) : rstd * v[slot + 1];
            lo = min3(lo, v[slot], v[slot + 1]);
            hi = max3(hi, v[slot], v[slot + 1]);
        }
        lo = redux_min(lo);
        hi = redux_max(hi);
        if (lane == 0) { rlo[warp] = lo; rhi[warp] = hi; }
        __syncthreads();                                               // S3
        for (int w = 0; w < nw4; w += 4) {          // padding holds 0: restored below from real warps
            const float4 a = *reinterpret_cast<const float4*>(rlo + w);
            const float4 b = *reinterpret_cast<const float4*>(rhi + w);
            if (w + 3 < nw) {
                lo = min3(min3(lo, a.x, a.y), a.z, a.w);
                hi = max3(max3(hi, b.x, b.y), b.z, b.w);
            } else {
                lo = fminf(lo, a.x); hi = fmaxf(hi, b.x);
                if (w + 1 < nw) { lo = fminf(lo, a.y); hi = fmaxf(hi, b.y); }
                if (w + 2 < nw) { lo = fminf(lo, a.z); hi = fmaxf(hi, b.z); }
            }
        }
        // -- Eq. 2
        float alpha = (hi - lo) * inv_qmax;
        if (!(hi > lo)) alpha = lo != 0.f ? fabsf(lo) : 1.f;
        const float inv = __frcp_rn(alpha);
        const float zero = -rintf(lo * inv);
        const bool big = fmaxf(fabsf(lo), fabsf(hi)) * inv >= 2097152.f || fabsf(zero) >= 2097152.f;
        const int zadd = int(zero) - kMagicBits;
        int n[CPT];
        if (!big) {
#pragma unroll
            for (int slot = 0; slot < CPT; ++slot)
                n[slot] = __float_as_int(fmaf(v[slot], inv, kMagic)) + zadd;
        } else {
#pragma unroll
            for (int slot = 0; slot < CPT; ++slot) {
                const float q = fminf(fmaxf(rintf(v[slot] * inv) + zero, 0.f), qmax);
                n[slot] = int(q);
            }
        }
        int csum = 0;
        if (FOURBIT) {
            // one byte per pair: low nibble = even channel
            uint32_t w[NP / 4];
#pragma unroll
            for (int g = 0; g < NP / 4; ++g) {
                uint32_t p = 0;
#pragma unroll
                for (int i = 3; i >= 0; --i) p = pack_sat_u4(n[2 * (4 * g + i) + 1], n[2 * (4 * g + i)], p);
                w[g] = p;
                const uint32_t nib = (p & 0x0F0F0F0Fu) + ((p >> 4) & 0x0F0F0F0Fu);
                csum = int(__dp4a(nib, 0x01010101u, uint32_t(csum)));
            }
            uint8_t* out = codes + m * (C / 2) + t;
#pragma unroll
            for (int i = 0; i < NP; ++i) out[NT * i] = uint8_t(w[i >> 2] >> (8 * (i & 3)));
        } else {
            const int top = int(qmax);
            uint16_t* out = reinterpret_cast<uint16_t*>(codes + m * C) + t;
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const int e = n[2 * i], o = n[2 * i + 1];
                const uint32_t p = pack_sat_u8(min(o, top), min(e, top), 0);
                out[NT * i] = uint16_t(p);
                csum += int(p & 0xFFu) + int(p >> 8);
            }
        }
        if (t == 0) { a_scale[m] = alpha; a_zero[m] = zero; }
        csum = __reduce_add_sync(0xffffffffu, csum);
        if (lane == 0) redi[par * 32 + warp] = csum;
        m_prev = m;
    }
    __syncthreads();
    if (t == 0 && m_prev >= 0 && a_rowsum) {
        const int* ri = redi + (par ^ 1) * 32;
        int tot = 0;
        for (int w = 0; w < nw; ++w) tot += ri[w];
        a_rowsum[m_prev] = tot;
    }
}

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            n = 148;
    }
    return n;
}

template <int CPT, int NTT, typename XT, bool HAS_BETA, bool FOURBIT>
int launch_main(const void* x, int64_t M, int C, const float* gamma, float eps, const int32_t* ptr,
                const int32_t* src, const float* coef, int bits, const MapImage& im, uint8_t* codes,
                float* a_scale, float* a_zero, int32_t* a_rowsum, cudaStream_t st) {
    auto kern = reassemble_quant_fast<CPT, NTT, XT, HAS_BETA, FOURBIT>;
    const int nt = C / CPT;
    const size_t smem = size_t(C + kVirt) * 4 + (2 * 4 * 32 + 2 * 32) * 4;
    if (smem > 48 * 1024)
        QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    int per_sm = 0;
    QLLM_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, nt, smem));
    if (per_sm < 1) per_sm = 1;
    const int grid = int(std::min<int64_t>(M, int64_t(sm_count()) * per_sm));
    kern<<<grid, nt, smem, st>>>(static_cast<const XT*>(x), M, C, gamma, eps, ptr, src, coef, bits, im, codes,
                                 a_scale, a_zero, a_rowsum);
    return after_launch();
}

template <int CPT, int NTT, typename XT>
int launch_layout(const void* x, int64_t M, int C, const float* gamma, bool has_beta, float eps,
                  const int32_t* ptr, const int32_t* src, const float* coef, int bits, bool packed,
                  const MapImage& im, uint8_t* codes, float* a_scale, float* a_zero, int32_t* a_rowsum,
                  cudaStream_t st) {
#define QLLM_MAIN(B, F) launch_main<CPT, NTT, XT, B, F>(x, M, C, gamma, eps, ptr, src, coef, bits, im, codes, a_scale, a_zero, a_rowsum, st)
    // run-time thread counts keep one variant per bit packing (the bias registers are always present)
    if (NTT == 0 || has_beta) return packed ? QLLM_MAIN(true, true) : QLLM_MAIN(true, false);
    return packed ? QLLM_MAIN(false, true) : QLLM_MAIN(false, false);
#undef QLLM_MAIN
}

// Thread layout of the specialised kernel for a channel count: channels per thread (0 = none).
int layout_cpt(int C) {
    if (C % 512 == 0 && C <= 8192) return 16;
    if (C % 256 == 0 && C <= 4096) return 8;
    return 0;
}

}  // namespace

bool reassemble_byte_lanes_supported(int C) { return layout_cpt(C) != 0; }

size_t reassemble_map_image_bytes(int C) {
    const int cpt = layout_cpt(C);
    return cpt ? map_image_bytes(cpt, C / cpt) : 0;
}

int compile_reassemble_map(int C, const float* gamma, const float* beta, const int32_t* ptr, const int32_t* src,
                           const float* coef, void* image, cudaStream_t st) {
    const int cpt = layout_cpt(C);
    if (!cpt) return QLLM_ERR_UNSUPPORTED;
    const int nt = C / cpt;
    const MapImage im = map_image_at(image, cpt, nt);
    QLLM_CUDA_TRY(cudaMemsetAsync(im.head, 0, 16, st));
    if (cpt == 16) compile_map_kernel<16><<<nt / 32, 32, 0, st>>>(C, nt, gamma, beta, ptr, src, coef, im);
    else compile_map_kernel<8><<<nt / 32, 32, 0, st>>>(C, nt, gamma, beta, ptr, src, coef, im);
    return after_launch();
}

int launch_reassemble_quant(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                            const float* beta, float eps, const int32_t* ptr, const int32_t* src,
                            const float* coef, int bits, const void* map_image, uint8_t* codes, float* a_scale,
                            float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool byte_lanes) {
    const int cpt = layout_cpt(C);
    if (!cpt && byte_lanes && bits == 4) return QLLM_ERR_UNSUPPORTED;
    const bool packed = bits == 4 && !byte_lanes;
    if (!cpt)
        return launch_reassemble_quant_generic(x, x_dtype, M, C, gamma, beta, eps, ptr, src, coef, bits, codes,
                                               a_scale, a_zero, a_rowsum, st);
    const int nt = C / cpt;
    if (!map_image) {
        // direct call: compile the map for this launch into per-stream library scratch
        uint8_t* buf = nullptr;
        int rc = stream_scratch(kScratchMapImage, st, map_image_bytes(cpt, nt), &buf);
        if (rc != QLLM_OK) return rc;
        rc = compile_reassemble_map(C, gamma, beta, ptr, src, coef, buf, st);
        if (rc != QLLM_OK) return rc;
        map_image = buf;
    }
    const MapImage im = map_image_at(const_cast<void*>(map_image), cpt, nt);
    const bool bf = x_dtype == QLLM_BF16, hb = beta != nullptr;
#define QLLM_RQ_ARGS x, M, C, gamma, hb, eps, ptr, src, coef, bits, packed, im, codes, a_scale, a_zero, a_rowsum, st
    // LLaMA hidden sizes get compile-time thread counts (immediate offsets, unrolled reductions)
    if (bf && C == 4096) return launch_layout<16, 256, __nv_bfloat16>(QLLM_RQ_ARGS);
    if (bf && C == 5120) return launch_layout<16, 320, __nv_bfloat16>(QLLM_RQ_ARGS);
    if (bf && C == 8192) return launch_layout<16, 512, __nv_bfloat16>(QLLM_RQ_ARGS);
    if (cpt == 16)
        return bf ? launch_layout<16, 0, __nv_bfloat16>(QLLM_RQ_ARGS) : launch_layout<16, 0, float>(QLLM_RQ_ARGS);
    return bf ? launch_layout<8, 0, __nv_bfloat16>(QLLM_RQ_ARGS) : launch_layout<8, 0, float>(QLLM_RQ_ARGS);
#undef QLLM_RQ_ARGS
}

}  // namespace qllm
