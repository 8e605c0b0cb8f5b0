// Device helpers and limits shared by the fused pre-GEMM kernels (LayerNorm -> reassembly ->
// per-token quantization, QLLM Eq. 2-4): rounding constant, 3-input min/max, saturating packs,
// the limits of a compiled map image, and the counts a compiled image reports to the launcher.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace qllm {

constexpr int kSlotCap = 2048;                 // virtual slots an image can describe
constexpr int kOtherCap = 1024;                // of which rows with three and more entries
constexpr int kInline = 4;                     // entries held inside a slot record
constexpr int kLongCap = 512;                  // entries of longer rows kept as (position, weight) pairs
constexpr int kLongRows = 256;                 // longer rows listed by slot
constexpr int kSmemBudget = 227 * 1024;
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23: adding it rounds to nearest-even integer
constexpr int kMagicBits = 0x4B400000;

// What a compiled image holds, as the launcher needs it to size shared memory: slots = rows with several
// entries, other = those with three and more, long_rows = those longer than a slot record, long_entries =
// entries kept for them.  known = false: the launcher assumes the largest image.
struct MapCounts {
    int slots = 0, other = 0, long_rows = 0, long_entries = 0;
    bool known = false;
    bool fits = false;                         // the slots can serve a launch (else it walks the CSR arrays)
};

struct RawMap {
    const float* gamma;
    const int32_t* ptr;
    const int32_t* src;
    const float* coef;
};

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

}  // namespace qllm
