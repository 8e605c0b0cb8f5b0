// The compiled reassembly map of the kernels that work on the source side of the map (QLLM Eq. 3, 4): layout of
// the image in device memory and of a token's row in shared memory.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "reassemble_quant_common.cuh"

namespace qllm {

// word position of source channel k in a token's row
__host__ __device__ __forceinline__ int qpos(int k, int C) {
    return ((k >> 2) & 1) * (C >> 1) + ((k >> 3) << 2) + (k & 3);
}

// Compiled map for this kernel: one allocation, in this order.
//   wsA, wsB  float[C/8][4]  source weights of channels 8g .. 8g+3 / 8g+4 .. 8g+7: coef * gamma_k of the one map
//                            entry that reads channel k (gamma_k alone for a member of a merged set)
//   bsA, bsB  the same for coef * beta_k (zero without beta)
//   idx       uint16[C]      byte offset in the row of the output channel's source, or of its slot
//                            (4 * (C + slot)); record slot t of group g is channel 8g + ((t + r) & 7), r = (g & 31) >> 3
//   member    uint32[C/32]   bit k: source channel k is a member of a merged set (not an output by itself), or
//                            is not read at all
//   Virtual slots, rows of two entries first (slots 0 .. n2-1), then rows of three to eight, longer rows last:
//   rec01 uint4[kSlotCap]      {byte offsets off0 | off1 << 16, coef 0, coef 1, 0}
//   rec23 uint4[kTokOtherCap][3]  {off2 | off3 << 16, coef 2, coef 3, 0}, then entries 4, 5 and 6, 7 of slot n2 + t
//                              (coef 0 where absent)
//   A row longer than kTokInline entries is listed in
//   lmeta int4[kLongRows]    {slot, first, n, kind}: kind 1 = entries lent[first .. first+n), kind 0 = CSR entries
//   lent uint2[kLongCap]     {word position, coef bits}
//   head int[8]              [0], [3] = pairs / other rows given a slot, [1] = entries handed out in lent,
//                            [2] = rows longer than kTokInline listed, [4] = n2, [5] = rows of three and more,
//                            [6] = rows longer than kTokInline, [7] = 1 when this kernel can serve the map:
//                            the slots fit and every source channel is read either by single-entry rows that
//                            all carry one coefficient, or by exactly one multi-entry row
//   tag       uint32[C], nmulti int[C]   scratch of the compilation (coefficient seen / multi-entry readers)
constexpr int kTokInline = 8;                  // entries held inside a slot's records
constexpr int kTokOtherCap = 512;              // rows of three and more entries an image can describe
struct TokImage {
    float *wsA, *wsB, *bsA, *bsB;
    uint16_t* idx;
    uint32_t* member;
    uint4* rec01;
    uint4* rec23;
    int4* lmeta;
    uint2* lent;
    int* head;
    uint32_t* tag;
    int* nmulti;
};
__host__ __device__ inline size_t tok_image_bytes_impl(int C) {
    return size_t(C) * 10 + size_t(C) / 8 + size_t(kSlotCap) * 16 + size_t(kTokOtherCap) * 48 + size_t(kLongRows) * 16 +
           size_t(kLongCap) * 8 + 32 + size_t(C) * 8;
}
__host__ __device__ inline TokImage tok_image_at(void* base, int C) {
    TokImage im;
    im.wsA = static_cast<float*>(base);
    im.wsB = im.wsA + C / 2;
    im.bsA = im.wsB + C / 2;
    im.bsB = im.bsA + C / 2;
    im.idx = reinterpret_cast<uint16_t*>(im.bsB + C / 2);
    im.member = reinterpret_cast<uint32_t*>(im.idx + C);
    im.rec01 = reinterpret_cast<uint4*>(im.member + C / 32);
    im.rec23 = im.rec01 + kSlotCap;
    im.lmeta = reinterpret_cast<int4*>(im.rec23 + 3 * kTokOtherCap);
    im.lent = reinterpret_cast<uint2*>(im.lmeta + kLongRows);
    im.head = reinterpret_cast<int*>(im.lent + kLongCap);
    im.tag = reinterpret_cast<uint32_t*>(im.head + 8);
    im.nmulti = reinterpret_cast<int*>(im.tag + C);
    return im;
}

}  // namespace qllm
