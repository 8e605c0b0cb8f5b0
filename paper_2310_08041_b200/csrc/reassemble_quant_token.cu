// Fused pre-GEMM kernel for bf16 rows of LLaMA hidden sizes (4096, 5120, 8192 channels):
// LayerNorm -> channel reassembly -> per-token asymmetric quantization (QLLM Eq. 2-4; the fusion
// the paper leaves as future work, Sec. 6).
//
// HBM roofline: a token row is read from DRAM once and its codes are written once.  In practice the kernel is
// bound by issue slots (~18 instructions per channel) and by the shared-memory data pipe (the gathers of a real map
// hit ~3 banks twice), so the design keeps both low and keeps several tokens in flight per SM.  Design:
//  * G warps own a token from load to store (a lane owns NPL = C / (32 G) channels, 8 consecutive ones per
//    step); the per-token reductions are warp shuffles plus a G-warp named barrier.  One CTA per SM holds as
//    many tokens as registers and shared memory allow; tokens are dealt round-robin.
//  * Sum and sum of squares of the row come from the tensor cores (the registers of the 16-byte loads are a
//    bf16 operand as they are).  A row whose mean dominates its spread takes a second, centred pass.
//  * The work is done on the SOURCE side: a channel k of the normalised row is used by one output row of the
//    map only (or by the T sub-channels of a disassembled channel, Eq. 3, which all take x_k / T), so
//    y_k = ws_k (x_k - mean) [* rstd + bs_k with beta], ws_k = coef * gamma_k, is computed where x_k was loaded,
//    stored once as fp32, and the row's range is taken there too (members of merged sets, Eq. 4, excluded by a
//    per-lane bit mask).  Rows with several entries become "virtual slots": once per token a lane sums their
//    members into a slot appended to the row and folds the sum into the range.  Every output channel is then
//    ONE gather that feeds the quantizer directly: besides the loaded row only the gather addresses stay in
//    registers across phases.  A map in which a source channel is read by rows with different coefficients
//    cannot be served this way: the compiled image says so and the launch does nothing (see the launcher).
//  * Layout of the row: channel k sits at word ((k >> 2) & 1) * C/2 + (k >> 3) * 4 + (k & 3) (two planes of
//    4-channel quads), so the two 16-byte stores of a step are conflict-free; a lane visits its 8 output
//    channels in an order rotated by lane / 8, which spreads the gathers of order-preserving stretches of the map
//    over the banks.  The packed output word is rotated back with one funnel shift.
//  * The next row of the token slot is asked into L2 one token ahead; rstd is folded into the quantization
//    scale; rounding by the 1.5 * 2^23 constant; clamp and packing by saturating cvt.pack (nibbles) or by byte
//    permutes and a clamp inside the word (one code per byte).

#include <cuda_bf16.h>

#include "common.h"
#include "device_utils.cuh"
#include "reassemble_quant_common.cuh"
#include "token_image.cuh"

namespace qllm {

namespace {

__device__ __forceinline__ void put_source(const TokImage& im, int k, float w, float b) {
    (((k & 7) < 4) ? im.wsA : im.wsB)[4 * (k >> 3) + (k & 3)] = w;
    (((k & 7) < 4) ? im.bsA : im.bsB)[4 * (k >> 3) + (k & 3)] = b;
}

// 64-bit finaliser of the splitmix64 generator (Steele, Lea, Flood 2014): every input bit reaches every output bit
__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
// Content key of everything a compiled image depends on: the sum over all elements of mix64(array, index, bits),
// plus the sizes.  Order-independent, so every thread adds up a strided share.  Never 0 (0 marks "no image").
__device__ uint64_t map_content_key(int C, const float* gamma, const float* beta, const int32_t* ptr,
                                    const int32_t* src, const float* coef, uint64_t* red) {
    const int nnz = __ldg(ptr + C);
    uint64_t h = 0;
    auto add = [&](uint64_t array, int i, uint32_t bits) { h += mix64((array << 56) ^ (uint64_t(uint32_t(i)) << 32) ^ bits); };
    for (int i = threadIdx.x; i <= C; i += blockDim.x) add(1, i, uint32_t(__ldg(ptr + i)));
    for (int i = threadIdx.x; i < nnz; i += blockDim.x) {
        add(2, i, uint32_t(__ldg(src + i)));
        add(3, i, __float_as_uint(__ldg(coef + i)));
    }
    for (int i = threadIdx.x; i < C; i += blockDim.x) {
        add(4, i, __float_as_uint(__ldg(gamma + i)));
        if (beta) add(5, i, __float_as_uint(__ldg(beta + i)));
    }
    for (int o = 16; o > 0; o >>= 1) h += __shfl_xor_sync(0xffffffffu, h, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = h;
    __syncthreads();
    h = mix64((uint64_t(uint32_t(C)) << 32) ^ uint32_t(nnz) ^ (beta ? 1ull << 63 : 0ull));
    for (int w = 0; w < int(blockDim.x >> 5); ++w) h += red[w];
    return h ? h : 1;
}

// One CTA compiles the whole map: a counting pass, then one thread per output channel writes its record, the
// weights of the sources it reads and, for a multi-entry row, its slot.
// key (may be null): where the content key of the image's inputs is kept beside an image that lives in library
// scratch.  A call whose inputs hash to the key already there finds its image in place and compiles nothing.
__global__ void __launch_bounds__(1024)
compile_map_token_kernel(int C, const float* __restrict__ gamma, const float* __restrict__ beta,
                         const int32_t* __restrict__ ptr, const int32_t* __restrict__ src,
                         const float* __restrict__ coef, TokImage im, uint64_t* key) {
    __shared__ int cnt[8];
    __shared__ uint64_t red[32];
    constexpr uint32_t kUnread = 0xFFFFFFFFu;
    uint64_t content = 0;
    if (key) {
        content = map_content_key(C, gamma, beta, ptr, src, coef, red);
        if (*key == content) return;                          // the same value for every thread
        __syncthreads();
        if (threadIdx.x == 0) *key = 0;                       // no valid image while this one is being written
    }
    if (threadIdx.x < 8) cnt[threadIdx.x] = 0;
    for (int i = threadIdx.x; i < C / 32; i += blockDim.x) im.member[i] = 0u;
    for (int k = threadIdx.x; k < C; k += blockDim.x) { im.tag[k] = kUnread; im.nmulti[k] = 0; }
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const int n = __ldg(ptr + c + 1) - __ldg(ptr + c);
        if (n == 2) atomicAdd(cnt + 4, 1);
        else if (n > 2) atomicAdd(cnt + 5, 1);
        if (n > kTokInline) atomicAdd(cnt + 6, 1);
    }
    __syncthreads();
    const int n2 = cnt[4], n34 = cnt[5];
    const bool fits = n2 + n34 <= kSlotCap && n34 <= kTokOtherCap && cnt[6] <= kLongRows;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const int j0 = __ldg(ptr + c), n = __ldg(ptr + c + 1) - j0;
        const int s0 = __ldg(src + j0);
        uint32_t off = uint32_t(4 * qpos(s0, C));
        if (n == 1) {
            // the only reader of channel s0, or one of the T sub-channels that all read it with the same coef
            const float c0 = __ldg(coef + j0);
            put_source(im, s0, c0 * __ldg(gamma + s0), beta ? c0 * __ldg(beta + s0) : 0.f);
            const uint32_t seen = atomicCAS(im.tag + s0, kUnread, __float_as_uint(c0));
            if ((seen != kUnread && seen != __float_as_uint(c0)) || __float_as_uint(c0) == kUnread) cnt[7] = 1;
        } else {                                              // merged row: its members keep gamma, beta; the slot has coef
            uint32_t o[kTokInline] = {0, 0, 0, 0, 0, 0, 0, 0};
            float cc[kTokInline] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            for (int e = 0; e < n; ++e) {
                const int sj = __ldg(src + j0 + e);
                put_source(im, sj, __ldg(gamma + sj), beta ? __ldg(beta + sj) : 0.f);
                atomicOr(im.member + (sj >> 5), 1u << (sj & 31));
                if (atomicAdd(im.nmulti + sj, 1) > 0) cnt[7] = 1;         // read by a second multi-entry row
                if (e < kTokInline) { o[e] = uint32_t(4 * qpos(sj, C)); cc[e] = __ldg(coef + j0 + e); }
            }
            if (fits) {
                int slot, li = 0;
                if (n == 2) {
                    slot = atomicAdd(cnt, 1);
                } else if (n <= kTokInline) {
                    const int t = atomicAdd(cnt + 3, 1);
                    slot = n2 + t;
                    for (int h = 0; h < 3; ++h)
                        im.rec23[3 * t + h] = make_uint4(o[2 * h + 2] | (o[2 * h + 3] << 16), __float_as_uint(cc[2 * h + 2]),
                                                         __float_as_uint(cc[2 * h + 3]), 0u);
                } else {                                      // the longer rows take the last slots
                    li = atomicAdd(cnt + 2, 1);
                    slot = n2 + n34 - cnt[6] + li;
                }
                im.rec01[slot] = make_uint4(o[0] | (o[1] << 16), __float_as_uint(cc[0]), __float_as_uint(cc[1]), 0u);
                if (n > kTokInline) {
                    int first = atomicAdd(cnt + 1, n), kind = 1;
                    if (first + n <= kLongCap) {              // entries as (position, coef) pairs for shared memory
                        for (int e = 0; e < n; ++e)
                            im.lent[first + e] = make_uint2(uint32_t(qpos(__ldg(src + j0 + e), C)),
                                                            __float_as_uint(__ldg(coef + j0 + e)));
                    } else {                                  // walks the CSR arrays at run time
                        first = j0;
                        kind = 0;
                    }
                    if (li < kLongRows) im.lmeta[li] = make_int4(slot, first, n, kind);
                }
                off = uint32_t(4 * (C + slot));
            }
        }
        const int g = c >> 3, r = (g & 31) >> 3, t = ((c & 7) - r) & 7;     // record slot of channel c
        im.idx[8 * g + t] = uint16_t(off);
    }
    __syncthreads();
    for (int k = threadIdx.x; k < C; k += blockDim.x) {
        const bool single = im.tag[k] != kUnread, multi = im.nmulti[k] > 0;
        if (single && multi) cnt[7] = 1;                      // read with a coefficient of its own and as a member
        if (!single && !multi) {                              // read by nobody: out of the range, finite
            put_source(im, k, 0.f, 0.f);
            atomicOr(im.member + (k >> 5), 1u << (k & 31));
        }
    }
    __syncthreads();
    if (threadIdx.x < 8) im.head[threadIdx.x] = threadIdx.x == 7 ? int(fits && cnt[7] == 0) : cnt[threadIdx.x];
    if (key && threadIdx.x == 0) { __threadfence(); *key = content; }
}

// Output channel c from the stored row y by its CSR row: y[src] for a single entry (the coefficient is in y
// already), sum coef_j y[src_j] for a merged row.  Out of line: it serves only maps that do not fit the slots.
__device__ __noinline__ float csr_channel(const RawMap& rm, const float* d, int C, int c) {
    const int j0 = __ldg(rm.ptr + c), n = __ldg(rm.ptr + c + 1) - j0;
    if (n == 1) return d[qpos(__ldg(rm.src + j0), C)];
    float e = 0.f;
    for (int j = j0; j < j0 + n; ++j) e = fmaf(__ldg(rm.coef + j), d[qpos(__ldg(rm.src + j), C)], e);
    return e;
}
__device__ __forceinline__ float csr_entries(const RawMap& rm, const float* d, int C, int j0, int n) {
    float e = 0.f;
    for (int j = j0; j < j0 + n; ++j) e = fmaf(__ldg(rm.coef + j), d[qpos(__ldg(rm.src + j), C)], e);
    return e;
}
// sum of a longer row's entries kept as (position, coef) pairs
__device__ __forceinline__ float pair_row(const uint2* ent, const float* d, int first, int n) {
    float e = 0.f;
    for (int k = 0; k < n; ++k) {
        const uint2 pw = ent[first + k];
        e = fmaf(__uint_as_float(pw.y), d[pw.x], e);
    }
    return e;
}

template <int G>
__device__ __forceinline__ void token_sync(int barid) {
    asm volatile("bar.sync %0, %1;" ::"r"(barid), "n"(32 * G) : "memory");
}

// Shared memory through 32-bit window addresses: one register per pointer, offsets fold into the instruction.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ float lds_f32(uint32_t a) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(a));
    return v;
}
template <int OFF>
__device__ __forceinline__ uint4 lds_u4(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4 + %5];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a), "n"(OFF));
    return v;
}
template <int OFF>
__device__ __forceinline__ float4 lds_f4(uint32_t a) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4 + %5];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a), "n"(OFF));
    return v;
}
template <int OFF>
__device__ __forceinline__ void sts_f4(uint32_t a, float x, float y, float z, float w) {
    asm volatile("st.shared.v4.f32 [%0 + %1], {%2, %3, %4, %5};" ::"r"(a), "n"(OFF), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
// D += A (16 x 16 bf16, row-major fragment a[0..3]) * B (16 x 8 bf16, fragment b0, b1), fp32 accumulators
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ldg_u4_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void sts_f32(uint32_t a, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v) : "memory");
}
__device__ __forceinline__ void sts_f2(uint32_t a, float x, float y) {
    asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(a), "f"(x), "f"(y) : "memory");
}
__device__ __forceinline__ uint4 lds_u4_at(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ float2 lds_f2_at(uint32_t a) {
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ float4 lds_f4_at(uint32_t a) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts_f4_at(uint32_t a, float x, float y, float z, float w) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}

// Shared memory of a CTA, in bytes, before the token rows.
__host__ __device__ inline int tok_fixed_bytes(int C, bool has_beta, int max_tok, int G, int slot_room, int other_room,
                                               int long_rows, int long_ent) {
    return (has_beta ? 8 : 4) * C + max_tok * 8 * G * 4 + slot_room * 16 + other_room * 48 + long_rows * 16 +
           long_ent * 8;
}

struct TokRooms {
    int slot, other, long_rows, long_ent;      // multiples of 4
};

template <int C, int G, bool HAS_BETA, bool PACKED, int MAXW>
__global__ void __launch_bounds__(32 * MAXW, 1)
reassemble_quant_token(const __nv_bfloat16* __restrict__ x, int64_t M, float eps, int bits, TokImage im, TokRooms rooms,
                       int TOK /* tokens in flight per CTA */, RawMap rm, uint8_t* __restrict__ codes,
                       float* __restrict__ a_scale, float* __restrict__ a_zero, int32_t* __restrict__ a_rowsum) {
    constexpr int NPL = C / (32 * G);                      // channels per lane
    constexpr int NIT = NPL / 8;                           // steps of 8 channels per lane
    constexpr int GS = 32 * G;                             // groups per step over the token's lanes
    constexpr int MAXTOK = MAXW / G;
    static_assert(NPL % 8 == 0 && NPL * 32 * G == C && NIT <= 8, "a lane owns up to 8 whole groups of 8 channels");
    extern __shared__ __align__(16) uint8_t smem_bytes[];
    float* s_ws = reinterpret_cast<float*>(smem_bytes);    // wsA | wsB (| bsA | bsB with beta), [C/8][4] each
    float* s_ex = s_ws + (HAS_BETA ? 2 : 1) * C;           // [MAXTOK][8 G] exchange words per token slot
    uint4* s_rec01 = reinterpret_cast<uint4*>(s_ex + MAXTOK * 8 * G);       // slot records
    uint4* s_rec23 = s_rec01 + rooms.slot;
    int4* s_lmeta = reinterpret_cast<int4*>(s_rec23 + 3 * rooms.other);     // rows longer than the records
    uint2* s_lent = reinterpret_cast<uint2*>(s_lmeta + rooms.long_rows);    // their entries
    float* rows = reinterpret_cast<float*>(s_lent + rooms.long_ent);
    const int row_words = C + rooms.slot;

    // a kernel launched as this one's programmatic dependent (the decode GEMM) may start its prologue now
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // The map's image says whether this kernel can serve it; if not the launch does nothing (the caller has
    // arranged for the shape-agnostic kernel to run instead).  Uniform over the grid.
    if (__ldg(im.head + 7) == 0) return;
    const int lane = threadIdx.x & 31;
    const int warp = __shfl_sync(0xffffffffu, int(threadIdx.x >> 5), 0);   // warp-uniform for the compiler
    const int tslot = warp / G, wsub = warp % G;
    const int g0 = wsub * 32 + lane;                       // this lane's group in step 0
    const int stride = int(gridDim.x) * TOK;               // token indices fit an int (M is checked by the launcher)
    int m = int(blockIdx.x) * TOK + tslot;
    const int Mi = int(M);
    const bool active = tslot < TOK && m < Mi;

    // first row of this token slot: towards L2 before anything else
    const uint4* xr = reinterpret_cast<const uint4*>(x + int64_t(active ? m : 0) * C) + g0;
    if (active) {
#pragma unroll
        for (int i = 0; i < NIT; i += 2)                   // even lanes ask for step i, odd lanes for step i + 1:
            if (i + (lane & 1) < NIT) prefetch_l2(xr + (i + (lane & 1)) * GS);   // every 128-byte line is touched
    }
    {   // slot records (and bias terms) -> shared memory, asynchronously
        auto copy16 = [&](void* dst, const void* src, int n16) {
            for (int i = threadIdx.x; i < n16; i += blockDim.x)
                cp_async16(static_cast<uint4*>(dst) + i, static_cast<const uint4*>(src) + i);
        };
        copy16(s_ws, im.wsA, (HAS_BETA ? 8 : 4) * C / 16);  // wsA | wsB | bsA | bsB back to back
        copy16(s_rec01, im.rec01, rooms.slot);
        copy16(s_rec23, im.rec23, 3 * rooms.other);
        copy16(s_lmeta, im.lmeta, rooms.long_rows);
        copy16(s_lent, im.lent, rooms.long_ent / 2);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    const int n2 = __ldg(im.head + 4);                     // slots of two-entry rows come first
    const int nslots = n2 + __ldg(im.head + 5);
    const int nlong = __ldg(im.head + 6);                  // rows longer than the slot records, last slots
    if (!active) {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        return;
    }
    const int barid = 1 + tslot;
    const float* d = rows + size_t(tslot) * row_words;     // generic view, for the rare longer rows only
    const uint32_t d_sa = smem_addr(d);
    const uint32_t rec01_sa = smem_addr(s_rec01), rec23_sa = smem_addr(s_rec23);
    const uint32_t dq_sa = d_sa + g0 * 16;                 // this lane's quads of the row, step 0
    const uint32_t ws_sa = smem_addr(s_ws) + g0 * 16;      // this lane's source weights (and bias terms), step 0
    // This lane's gathers, for the whole launch: their addresses in shared memory, and which of its source
    // channels stay out of the range.
    uint32_t ridx[NPL];
    uint32_t mreg[(NIT + 3) / 4];
    {
#pragma unroll
        for (int k = 0; k < (NIT + 3) / 4; ++k) mreg[k] = 0u;
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const int g = g0 + i * GS;
            const uint4 iw = __ldg(reinterpret_cast<const uint4*>(im.idx) + g);
            const uint32_t pw[4] = {iw.x, iw.y, iw.z, iw.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                ridx[8 * i + 2 * k] = d_sa + (pw[k] & 0xFFFFu);
                ridx[8 * i + 2 * k + 1] = d_sa + (pw[k] >> 16);
            }
            mreg[i / 4] |= ((__ldg(im.member + (g >> 2)) >> (8 * (g & 3))) & 0xFFu) << (8 * (i & 3));

        }
    }
    // exchange words of the token slot: [0, 2G) sums, [2G, 4G) range, [4G, 5G) code sums, [5G, 6G) centred squares
    const uint32_t ex_sa = smem_addr(s_ex + tslot * 8 * G);
    constexpr uint32_t kExR = 2 * G * 4, kExS = 4 * G * 4, kExQ = 5 * G * 4;
    const int rot = lane >> 3;                             // this lane's records are rotated by rot channels
    constexpr float invC = 1.0f / float(C);
    const float qmax = float((1 << bits) - 1);
    const float inv_qmax = 1.0f / qmax;
    const int top = int(qmax);
    const float qnan = __int_as_float(0x7FFFFFFF);
    uint8_t* crow = codes + int64_t(m) * (PACKED ? C / 2 : C) + (PACKED ? 4 : 8) * g0;   // this lane's words of the codes
    const int64_t crow_step = int64_t(stride) * (PACKED ? C / 2 : C);
    const int64_t xrow_step = int64_t(stride) * (C / 8);   // in 16-byte units
    int m_prev = -1;
    asm volatile("cp.async.wait_group 0;" ::: "memory");   // the records have landed (the first row is on its way)
    __syncthreads();

    for (; m < Mi; m += stride, crow += crow_step) {
        uint4 raw[NIT];                                    // the row: in L2 by now, asked for a token ago
#pragma unroll
        for (int i = 0; i < NIT; ++i) raw[i] = ldg_u4_stream(xr + i * GS);
        if (m + stride < Mi) {                             // and the next row of this token slot towards L2
            xr += xrow_step;
#pragma unroll
            for (int i = 0; i < NIT; i += 2)
                if (i + (lane & 1) < NIT) prefetch_l2(xr + (i + (lane & 1)) * GS);
        }
        // -- sum and sum of squares on the tensor cores: the four registers of a step are a 16 x 16 bf16 operand
        // whatever the order of its elements; times a matrix of ones it gives sums, times its own two halves
        // transposed it gives sums of squares on the diagonals (products exact, accumulation in fp32)
        float as[4] = {0.f, 0.f, 0.f, 0.f}, aq0[4] = {0.f, 0.f, 0.f, 0.f}, aq1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
            mma_bf16(as, w, 0x3F803F80u, 0x3F803F80u);
            mma_bf16(aq0, w, w[0], w[2]);
            mma_bf16(aq1, w, w[1], w[3]);
        }
        {   // every column of the ones product holds the row sums (each lane quartet repeats them); the squares sit
            // where row == column: rows 0..7 in the first product, 8..15 in the second.  Both sums in one
            // butterfly: the lower half-warp collects s, the upper ss.
            const float s = 0.25f * (as[0] + as[2]);
            const float ss = ((lane & 3) == (lane >> 3)) ? ((lane & 4) ? aq0[1] + aq1[3] : aq0[0] + aq1[2]) : 0.f;
            const bool up = lane & 16;
            float t = (up ? ss : s) + __shfl_xor_sync(0xffffffffu, up ? s : ss, 16);
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if ((lane & 15) == 0) sts_f32(ex_sa + 8 * wsub + (lane >> 4) * 4, t);
        }
        token_sync<G>(barid);                              // nobody reads the row of the token before any more
        float S = 0.f, SS = 0.f;
        if (G % 2 == 0 && G <= 8) {
#pragma unroll
            for (int w = 0; w < G; w += 2) {
                const float4 t = lds_f4_at(ex_sa + 8 * w);
                S += t.x + t.z;
                SS += t.y + t.w;
            }
        } else {
            const float2 t = lane < G ? lds_f2_at(ex_sa + 8 * lane) : make_float2(0.f, 0.f);
            S = warp_sum(t.x);
            SS = warp_sum(t.y);
        }
        const float mean = S * invC;
        float var = fmaf(-mean, mean, SS * invC);
        if (!(mean * mean <= 4.0f * var)) {
            // the mean dominates the spread (or the row is constant): E[x^2] - mean^2 has lost its digits;
            // take the centred sum of squares instead (same branch in all lanes of the token)
            float q = 0.f;
#pragma unroll
            for (int i = 0; i < NIT; ++i) {
                const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float e0 = __uint_as_float(w[k] << 16) - mean, e1 = __uint_as_float(w[k] & 0xFFFF0000u) - mean;
                    q = fmaf(e0, e0, q);
                    q = fmaf(e1, e1, q);
                }
            }
            q = warp_sum(q);
            if (lane == 0) sts_f32(ex_sa + kExQ + 4 * wsub, q);
            token_sync<G>(barid);
            float Q = 0.f;
            for (int w = 0; w < G; ++w) Q += lds_f32(ex_sa + kExQ + 4 * w);
            var = Q * invC;
        }
        const float rstd = rsqrtf(var + eps);              // without beta a common factor of the whole row: its
                                                           // last-bit error rescales alpha, codes unchanged
        if (m_prev >= 0 && a_rowsum && warp % G == 0 && lane == 0) {   // code sum of the token before this one
            int tot = 0;
#pragma unroll
            for (int w = 0; w < G; ++w) tot += __float_as_int(lds_f32(ex_sa + kExS + 4 * w));
            a_rowsum[m_prev] = tot;
        }
        // -- source side: y_k = ws_k (x_k - mean) [* rstd + bs_k] to shared memory, range of the channels that are
        // outputs by themselves
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
            const float4 wa = lds_f4_at(ws_sa + i * GS * 16), wb = lds_f4_at(ws_sa + i * GS * 16 + C * 2);
            const float ws[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
            float y[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                y[2 * k] = __uint_as_float(w[k] << 16) - mean;
                y[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u) - mean;
            }
            if (HAS_BETA) {
                const float4 ba = lds_f4_at(ws_sa + i * GS * 16 + C * 4), bb = lds_f4_at(ws_sa + i * GS * 16 + C * 6);
                const float bs[8] = {ba.x, ba.y, ba.z, ba.w, bb.x, bb.y, bb.z, bb.w};
#pragma unroll
                for (int j = 0; j < 8; ++j) y[j] = fmaf(rstd * ws[j], y[j], bs[j]);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) y[j] *= ws[j];
            }
            const uint32_t mb = mreg[i / 4] >> (8 * (i & 3));  // bit j: channel j of this step is no output by itself
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const float ya = (mb & (1u << j)) ? qnan : y[j], yb = (mb & (2u << j)) ? qnan : y[j + 1];
                lo = min3(lo, ya, yb);                     // a NaN operand is ignored
                hi = max3(hi, ya, yb);
            }
            sts_f4_at(dq_sa + i * GS * 16, y[0], y[1], y[2], y[3]);
            sts_f4_at(dq_sa + i * GS * 16 + C * 2, y[4], y[5], y[6], y[7]);
        }
        // -- merged rows (Eq. 4): a lane per row sums the members into the row's virtual slot
        if (nslots > 0) {
            token_sync<G>(barid);                          // the row is complete
            // two-entry rows: a lane's records first, then their gathers, so that the loads are in flight together
            constexpr int SMAX = 4;
            for (int b0 = 0; b0 < n2; b0 += SMAX * GS) {
                uint4 r[SMAX];
                float a[SMAX], b[SMAX];
#pragma unroll
                for (int k = 0; k < SMAX; ++k)
                    if (b0 + k * GS < n2) r[k] = lds_u4_at(rec01_sa + 16 * min(b0 + k * GS + g0, n2 - 1));   // uniform over the token
#pragma unroll
                for (int k = 0; k < SMAX; ++k)
                    if (b0 + k * GS < n2) {
                        a[k] = lds_f32(d_sa + (r[k].x & 0xFFFFu));
                        b[k] = lds_f32(d_sa + (r[k].x >> 16));
                    }
#pragma unroll
                for (int k = 0; k < SMAX; ++k)
                    if (b0 + k * GS + g0 < n2) {
                        const float e = fmaf(__uint_as_float(r[k].z), b[k], __uint_as_float(r[k].y) * a[k]);
                        sts_f32(d_sa + 4 * (C + b0 + k * GS + g0), e);
                        lo = fminf(lo, e);
                        hi = fmaxf(hi, e);
                    }
            }
            // rows of three to eight entries (records and gathers in flight together), then longer rows, if any
            const int n38 = nslots - n2 - nlong;
            for (int vj = g0; vj < n38; vj += GS) {
                uint4 r[4];
                r[0] = lds_u4_at(rec01_sa + 16 * (n2 + vj));
#pragma unroll
                for (int h = 0; h < 3; ++h) r[h + 1] = lds_u4_at(rec23_sa + 16 * (3 * vj + h));
                float a[8];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    a[2 * h] = lds_f32(d_sa + (r[h].x & 0xFFFFu));
                    a[2 * h + 1] = lds_f32(d_sa + (r[h].x >> 16));
                }
                float e = __uint_as_float(r[0].y) * a[0];
                e = fmaf(__uint_as_float(r[0].z), a[1], e);
#pragma unroll
                for (int h = 1; h < 4; ++h) {
                    e = fmaf(__uint_as_float(r[h].y), a[2 * h], e);
                    e = fmaf(__uint_as_float(r[h].z), a[2 * h + 1], e);
                }
                sts_f32(d_sa + 4 * (C + n2 + vj), e);
                lo = fminf(lo, e);
                hi = fmaxf(hi, e);
            }
            for (int k = g0; k < nlong; k += GS) {
                const int4 lm = s_lmeta[k];
                const float e = lm.w ? pair_row(s_lent, d, lm.y, lm.z) : csr_entries(rm, d, C, lm.y, lm.z);
                sts_f32(d_sa + 4 * (C + lm.x), e);
                lo = fminf(lo, e);
                hi = fmaxf(hi, e);
            }
        }
        if (!HAS_BETA) { lo *= rstd; hi *= rstd; }         // rstd > 0: scaling commutes with min / max
        lo = redux_min(lo);
        hi = redux_max(hi);
        if (lane == 0) sts_f2(ex_sa + kExR + 8 * wsub, lo, hi);
        token_sync<G>(barid);                              // row and slots complete, range parts in place
        if (G % 2 == 0 && G <= 8) {
#pragma unroll
            for (int w = 0; w < G; w += 2) {
                const float4 t = lds_f4_at(ex_sa + kExR + 8 * w);
                lo = fminf(lo, fminf(t.x, t.z));
                hi = fmaxf(hi, fmaxf(t.y, t.w));
            }
        } else {
            const float2 t = lane < G ? lds_f2_at(ex_sa + kExR + 8 * lane) : make_float2(INFINITY, -INFINITY);
            lo = redux_min(t.x);
            hi = redux_max(t.y);
        }
        // -- Eq. 2
        float alpha = (hi - lo) * inv_qmax;
        if (!(hi > lo)) alpha = lo != 0.f ? fabsf(lo) : 1.f;
        const float inv = __frcp_rn(alpha);
        const float zero = -rintf(lo * inv);
        const bool big = fmaxf(fabsf(lo), fabsf(hi)) * inv >= 2097152.f || fabsf(zero) >= 2097152.f;
        const float sc = HAS_BETA ? inv : rstd * inv;      // without beta the row holds x' / rstd
        const int zadd = int(zero) - kMagicBits;
        const float magicz = kMagic + zero;                // exact while |zero| < 2^21 (else big)
        const int sh_over = bits == 4 ? 4 : 6;             // the bit above qmax's
        // -- reassembly (Eq. 3, 4): one gather per output channel, straight into the quantizer
        int csum = 0;
#pragma unroll
        for (int i = 0; i < NIT; ++i) {
            float u[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) u[j] = lds_f32(ridx[8 * i + j]);
            int n[8];
            if (!PACKED && !big && bits < 8) {
                // one code per byte, qmax = 15 or 63: the rounding constant carries the zero-point, so the low byte of
                // each float is the code modulo 256; a code is -1 .. qmax + 1 before the clamp, and the bit above
                // qmax's is set exactly for the two values the clamp changes (-1 -> 0, qmax + 1 -> qmax)
                uint32_t f[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) f[j] = __float_as_uint(fmaf(u[j], sc, magicz));
                uint32_t p0 = __byte_perm(__byte_perm(f[0], f[1], 0x0040), __byte_perm(f[2], f[3], 0x0040), 0x5410);
                uint32_t p1 = __byte_perm(__byte_perm(f[4], f[5], 0x0040), __byte_perm(f[6], f[7], 0x0040), 0x5410);
                const uint32_t lowm = 0x01010101u * uint32_t(top);
                p0 = (p0 & lowm) ^ (((p0 >> sh_over) & 0x01010101u) * uint32_t(top));
                p1 = (p1 & lowm) ^ (((p1 >> sh_over) & 0x01010101u) * uint32_t(top));
                csum = int(__dp4a(p0, 0x01010101u, uint32_t(csum)));
                csum = int(__dp4a(p1, 0x01010101u, uint32_t(csum)));
                const uint32_t q0 = __funnelshift_l(p1, p0, 8 * rot), q1 = __funnelshift_l(p0, p1, 8 * rot);
                *reinterpret_cast<uint2*>(crow + i * GS * 8) = make_uint2(q0, q1);
                continue;
            }
            if (!big) {
#pragma unroll
                for (int j = 0; j < 8; ++j) n[j] = __float_as_int(fmaf(u[j], sc, kMagic)) + zadd;
            } else {                                       // quotients beyond the range of the rounding constant
#pragma unroll
                for (int j = 0; j < 8; ++j) n[j] = int(fminf(fmaxf(rintf(u[j] * sc) + zero, 0.f), qmax));
            }
            if (PACKED) {
                // record slot t is channel (t + rot) & 7: pack in record order, rotate the nibbles into place
                uint32_t p = 0;
#pragma unroll
                for (int k = 3; k >= 0; --k) p = pack_sat_u4(n[2 * k + 1], n[2 * k], p);
                const uint32_t nib = (p & 0x0F0F0F0Fu) + ((p >> 4) & 0x0F0F0F0Fu);
                csum = int(__dp4a(nib, 0x01010101u, uint32_t(csum)));
                p = __funnelshift_l(p, p, 4 * rot);
                *reinterpret_cast<uint32_t*>(crow + i * GS * 4) = p;
            } else {
                uint32_t p0 = pack_sat_u8(min(n[3], top), min(n[2], top), 0u);
                p0 = pack_sat_u8(min(n[1], top), min(n[0], top), p0);
                uint32_t p1 = pack_sat_u8(min(n[7], top), min(n[6], top), 0u);
                p1 = pack_sat_u8(min(n[5], top), min(n[4], top), p1);
                csum = int(__dp4a(p0, 0x01010101u, uint32_t(csum)));
                csum = int(__dp4a(p1, 0x01010101u, uint32_t(csum)));
                // byte t of p1:p0 is channel (t + rot) & 7, rot < 4: rotate the 64-bit word left by rot bytes
                const uint32_t q0 = __funnelshift_l(p1, p0, 8 * rot), q1 = __funnelshift_l(p0, p1, 8 * rot);
                *reinterpret_cast<uint2*>(crow + i * GS * 8) = make_uint2(q0, q1);
            }
        }
        csum = __reduce_add_sync(0xffffffffu, csum);
        // the partial code sums are added up after the next barrier of this token slot (the next token's first, or
        // the one behind the loop): the barrier just passed orders these writes behind the reads of the sums before
        if (lane == 0) {
            sts_f32(ex_sa + kExS + 4 * wsub, __int_as_float(csum));
            if (wsub == 0) {
                a_scale[m] = alpha;
                a_zero[m] = zero;
            }
        }
        m_prev = m;
    }
    token_sync<G>(barid);
    if (a_rowsum && wsub == 0 && lane == 0) {
        int tot = 0;
#pragma unroll
        for (int w = 0; w < G; ++w) tot += __float_as_int(lds_f32(ex_sa + kExS + 4 * w));
        a_rowsum[m_prev] = tot;
    }
}

template <int C, int G, bool HAS_BETA, bool PACKED, int MAXW>
int launch_token(const void* x, int64_t M, float eps, int bits, const TokImage& im, const TokRooms& rooms,
                 const RawMap& rm, uint8_t* codes, float* a_scale, float* a_zero, int32_t* a_rowsum, cudaStream_t st,
                 bool share_sm) {
    auto kern = reassemble_quant_token<C, G, HAS_BETA, PACKED, MAXW>;
    constexpr int MAXTOK = MAXW / G;
    const int row_words = C + rooms.slot;
    const int fixed = tok_fixed_bytes(C, HAS_BETA, MAXTOK, G, rooms.slot, rooms.other, rooms.long_rows, rooms.long_ent);
    int tok_fit = int((kSmemBudget - fixed) / (int64_t(row_words) * 4));
    if (tok_fit > MAXTOK) tok_fit = MAXTOK;
    if (share_sm) {
        // leave a fifth of the register file free: the layer expands its 4-bit weights for the coming GEMM
        // on a second stream meanwhile, and that bandwidth-bound kernel needs room on every SM to keep
        // enough loads in flight
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
    // round is equally full on every SM
    const int64_t rounds = (per_cta + tok_fit - 1) / tok_fit;
    const int tok = int((per_cta + rounds - 1) / rounds);
    const int W = tok * G;
    const size_t smem = size_t(fixed) + size_t(tok) * row_words * 4;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
    // no more of the SM's array than the launch uses: what is left is L1, where the few spilled registers live
    const int carve = int((smem + 1024) * 100 / (228 * 1024)) + 1;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, carve > 100 ? 100 : carve));
    kern<<<grid, 32 * W, smem, st>>>(static_cast<const __nv_bfloat16*>(x), M, eps, bits, im, rooms, tok, rm, codes,
                                     a_scale, a_zero, a_rowsum);
    return after_launch();
}

template <int C, int G, int MAXW>
int launch_token_variant(bool has_beta, bool packed, const void* x, int64_t M, float eps, int bits,
                         const TokImage& im, const TokRooms& rooms, const RawMap& rm, uint8_t* codes, float* a_scale,
                         float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool share_sm) {
#define QLLM_RQT(B, P) launch_token<C, G, B, P, MAXW>(x, M, eps, bits, im, rooms, rm, codes, a_scale, a_zero, a_rowsum, st, share_sm)
    if (has_beta) return packed ? QLLM_RQT(true, true) : QLLM_RQT(true, false);
    return packed ? QLLM_RQT(false, true) : QLLM_RQT(false, false);
#undef QLLM_RQT
}

}  // namespace

bool token_kernel_serves(int C) { return C == 4096 || C == 5120 || C == 8192; }

size_t token_image_bytes(int C) { return token_kernel_serves(C) ? (tok_image_bytes_impl(C) + 15) / 16 * 16 : 0; }

int compile_token_map(int C, const float* gamma, const float* beta, const int32_t* ptr, const int32_t* src,
                      const float* coef, void* image, cudaStream_t st, uint64_t* key) {
    if (!token_kernel_serves(C)) return QLLM_ERR_UNSUPPORTED;
    compile_map_token_kernel<<<1, 1024, 0, st>>>(C, gamma, beta, ptr, src, coef, tok_image_at(image, C), key);
    return after_launch();
}

const int* token_image_served_flag(int C, const void* image) { return tok_image_at(const_cast<void*>(image), C).head + 7; }

int token_map_counts(int C, const void* image, cudaStream_t st, MapCounts* out) {
    if (!token_kernel_serves(C)) return QLLM_ERR_UNSUPPORTED;
    const TokImage im = tok_image_at(const_cast<void*>(image), C);
    int head[8];
    QLLM_CUDA_TRY(cudaMemcpyAsync(head, im.head, sizeof(head), cudaMemcpyDeviceToHost, st));
    QLLM_CUDA_TRY(cudaStreamSynchronize(st));
    MapCounts mc;
    mc.known = true;
    mc.slots = head[4] + head[5];
    mc.other = head[5];
    mc.long_rows = head[6];
    mc.long_entries = head[1] <= kLongCap ? head[1] : kLongCap;
    mc.fits = head[7] != 0;                                // the slots fit and the map is one this kernel can serve
    *out = mc;
    return QLLM_OK;
}

// The caller has checked that the image can serve the launch (counts known), or launches the shape-agnostic
// kernel behind this one with the image's flag (counts unknown: the kernel itself looks at the flag).
int launch_reassemble_quant_token(const void* x, int64_t M, int C, const float* gamma, const float* beta, float eps,
                                  const int32_t* ptr, const int32_t* src, const float* coef, int bits,
                                  const void* image, const MapCounts& mc, uint8_t* codes, float* a_scale,
                                  float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool byte_lanes, bool share_sm) {
    if ((mc.known && !mc.fits) || M > 0x7FFFFFFF) return QLLM_ERR_UNSUPPORTED;
    const TokImage im = tok_image_at(const_cast<void*>(image), C);
    // room for slot records and slot values: exact when the caller knows the image's counts, else the largest image's
    TokRooms rooms{kSlotCap, kTokOtherCap, kLongRows, kLongCap};   // whatever an image that serves can hold
    if (mc.known) {
        auto up4 = [](int v) { return (v + 3) & ~3; };
        rooms = TokRooms{up4(mc.slots), up4(mc.other), up4(mc.long_rows), up4(mc.long_entries)};
    }
    const RawMap rm{gamma, ptr, src, coef};
    const bool packed = bits == 4 && !byte_lanes, has_beta = beta != nullptr;
#define QLLM_TOKEN_ARGS has_beta, packed, x, M, eps, bits, im, rooms, rm, codes, a_scale, a_zero, a_rowsum, st, share_sm
    if (M <= device_sm_count()) {                          // one token per CTA: spread it over more warps
        if (C == 4096) return launch_token_variant<4096, 16, 16>(QLLM_TOKEN_ARGS);
        if (C == 5120) return launch_token_variant<5120, 20, 20>(QLLM_TOKEN_ARGS);
        if (C == 8192) return launch_token_variant<8192, 16, 16>(QLLM_TOKEN_ARGS);
    }
    if (C == 4096) return launch_token_variant<4096, 4, 20>(QLLM_TOKEN_ARGS);
    if (C == 5120) return launch_token_variant<5120, 5, 20>(QLLM_TOKEN_ARGS);
    if (C == 8192) return launch_token_variant<8192, 8, 24>(QLLM_TOKEN_ARGS);
#undef QLLM_TOKEN_ARGS
    return QLLM_ERR_UNSUPPORTED;
}


}  // namespace qllm
