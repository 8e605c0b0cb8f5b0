// Decode-sized integer GEMM (M <= 16 tokens): a weight-streaming kernel.  The weight codes
// (N*K/2 bytes for 4-bit) are read from HBM exactly once with 128-bit streaming loads; the few
// token rows are expanded to byte codes in shared memory once per CTA and reused by every
// weight row.  The kernel is HBM-bound, so the contraction runs on the warp-level integer MMA
// (m16n8k32, u8 x u8 -> s32): tokens are the 16-row operand, eight output channels of weights
// are the 8-column operand, and a 32-bit register of packed nibbles becomes the two operand
// registers with one mask and one shift+mask.  Plain dp4a would need ~2 M integer instructions
// per 8 weight codes and turn ALU-bound at M = 8..16; tcgen05 tiles (128 rows) would be 8x
// padding at these M.
//
// Work split: one task = 8 consecutive output channels over the whole K (no split-K, so no
// scratch and no atomics).  One CTA per SM; the number of warps per CTA is chosen on the host
// so that tasks fill whole waves.  K order inside a task is permuted (each thread walks its own
// 16-byte column of the row); both operands follow the same order, so every sum is exact.

#include <cuda_bf16.h>

#include "common.h"
#include "epilogue.cuh"

namespace qllm {

namespace {

constexpr int kMaxWarps = 24;

__device__ __forceinline__ void mma_u8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                       uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Token codes -> shared memory, K bytes per token (+ pad).  When the weights are packed
// nibbles (WP) every group of 8 codes is stored as (even codes, odd codes), the order in which
// a packed weight word splits into its two operand registers; otherwise natural order.
template <bool WP>
__device__ void fill_tokens(uint8_t* As, int stride, const uint8_t* __restrict__ a, int M, int K, int a_bits,
                            int rows) {
    const int groups = K / 8;
    const int total = rows * groups;
    constexpr int U = 4;                          // independent loads in flight per thread
    for (int base = threadIdx.x; base < total; base += U * blockDim.x) {
        uint2 v[U];
        int r[U], g8[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = base + u * blockDim.x;
            r[u] = idx / groups;
            g8[u] = idx - r[u] * groups;
            v[u] = make_uint2(0, 0);
            if (idx < total && r[u] < M) {
                if (a_bits == 4) v[u].x = __ldg(reinterpret_cast<const uint32_t*>(a + size_t(r[u]) * (K / 2) + g8[u] * 4));
                else v[u] = __ldg(reinterpret_cast<const uint2*>(a + size_t(r[u]) * K + g8[u] * 8));
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (base + u * blockDim.x >= total) break;
            uint32_t e, o;
            if (a_bits == 4) {
                const uint32_t lo = v[u].x & 0x0F0F0F0Fu, hi = (v[u].x >> 4) & 0x0F0F0F0Fu;
                if (WP) { e = lo; o = hi; }
                else { e = __byte_perm(lo, hi, 0x5140); o = __byte_perm(lo, hi, 0x7362); }
            } else {
                if (WP) { e = __byte_perm(v[u].x, v[u].y, 0x6420); o = __byte_perm(v[u].x, v[u].y, 0x7531); }
                else { e = v[u].x; o = v[u].y; }
            }
            *reinterpret_cast<uint2*>(As + r[u] * stride + g8[u] * 8) = make_uint2(e, o);
        }
    }
}

template <bool WP, bool M16>
__global__ void __launch_bounds__(32 * kMaxWarps, 1)
qgemm_decode_kernel(const uint8_t* __restrict__ a, const uint8_t* __restrict__ w, int M, int N, int K,
                    int a_bits, EpilogueArgs ep, int tasks) {
    extern __shared__ __align__(16) uint8_t As[];
    constexpr int PAD = WP ? 16 : 64;             // keeps the 16-byte fragment loads conflict-free
    constexpr int UN = 4;                         // iterations per register buffer (2 buffers in flight)
    const int stride = K + PAD;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = lane >> 2, tig = lane & 3;
    const int row_bytes = WP ? K / 2 : K;
    const int iters = row_bytes / 64;             // 4 threads x 16 bytes of a row per iteration
    const uint8_t* a_lo = As + g * stride;        // token g
    const uint8_t* a_hi = As + (g + 8) * stride;  // token g + 8 (M16 only)

    auto row_ptr = [&](int task) {
        const int n_ld = min(task * 8 + g, N - 1);   // rows past N re-read the last row; never stored
        return reinterpret_cast<const uint4*>(w + size_t(n_ld) * row_bytes) + tig;
    };
    auto load_block = [&](uint4 (&buf)[UN], const uint4* wp, int it0) {
#pragma unroll
        for (int u = 0; u < UN; ++u)
            buf[u] = (it0 + u < iters) ? __ldcs(wp + 4 * (it0 + u)) : make_uint4(0, 0, 0, 0);
    };

    // The kernel is launched as a programmatic dependent of the kernel before it (the pre-GEMM kernel that writes
    // the tokens): until that kernel is complete (griddepcontrol.wait) it only asks for its first weight rows to
    // be brought into L2 -- harmless whoever wrote them -- so the launch latency and the first trip to HBM pass
    // under the previous kernel.
    int task = blockIdx.x * nwarps + warp;
    if (task < tasks) {
        const int n_first = min(task * 8, N - 1), n_rows = min(8, N - n_first);
        const char* base = reinterpret_cast<const char*>(w + size_t(n_first) * row_bytes);
        for (int o = lane * 128; o < n_rows * row_bytes; o += 32 * 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(base + o));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // first weights are requested before the token rows are expanded: the stream starts at once
    uint4 cur[UN], nxt[UN];
    const uint4* wp = nullptr;
    if (task < tasks) { wp = row_ptr(task); load_block(cur, wp, 0); }
    fill_tokens<WP>(As, stride, a, M, K, a_bits, M16 ? 16 : 8);
    __syncthreads();

    // One step of the stream: UN x 16 bytes of this thread's weight column against the matching token
    // fragments.  Loads past the end of the row return zeros, so a step needs no bounds test: zero weights
    // add nothing (the token fragments then come from the slack behind the last row).  Two accumulator sets
    // halve the chain of dependent MMAs.
    auto step = [&](const uint4 (&buf)[UN], int it0, int (&c0)[4], int (&c1)[4]) {
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int it = it0 + u;
            const uint4 wv = buf[u];
            if (WP) {
                // 32 codes of this thread's column: words s = 0..3, each -> (even, odd) registers
                const int aoff = (16 * it + 4 * tig) * 8;
                const uint4 A0 = *reinterpret_cast<const uint4*>(a_lo + aoff);
                const uint4 A1 = *reinterpret_cast<const uint4*>(a_lo + aoff + 16);
                uint4 B0 = make_uint4(0, 0, 0, 0), B1 = B0;
                if (M16) {
                    B0 = *reinterpret_cast<const uint4*>(a_hi + aoff);
                    B1 = *reinterpret_cast<const uint4*>(a_hi + aoff + 16);
                }
                mma_u8(c0, A0.x, B0.x, A0.y, B0.y, wv.x & 0x0F0F0F0Fu, (wv.x >> 4) & 0x0F0F0F0Fu);
                mma_u8(c1, A0.z, B0.z, A0.w, B0.w, wv.y & 0x0F0F0F0Fu, (wv.y >> 4) & 0x0F0F0F0Fu);
                mma_u8(c0, A1.x, B1.x, A1.y, B1.y, wv.z & 0x0F0F0F0Fu, (wv.z >> 4) & 0x0F0F0F0Fu);
                mma_u8(c1, A1.z, B1.z, A1.w, B1.w, wv.w & 0x0F0F0F0Fu, (wv.w >> 4) & 0x0F0F0F0Fu);
            } else {
                // 16 byte codes of this thread's column: two k32 steps
                const int aoff = (4 * it + tig) * 16;
                const uint4 A0 = *reinterpret_cast<const uint4*>(a_lo + aoff);
                uint4 B0 = make_uint4(0, 0, 0, 0);
                if (M16) B0 = *reinterpret_cast<const uint4*>(a_hi + aoff);
                mma_u8(c0, A0.x, B0.x, A0.y, B0.y, wv.x, wv.y);
                mma_u8(c1, A0.z, B0.z, A0.w, B0.w, wv.z, wv.w);
            }
        }
    };

    for (; task < tasks; task += gridDim.x * nwarps) {
        const int n_base = task * 8;
        int c[4] = {0, 0, 0, 0}, c2[4] = {0, 0, 0, 0};
        for (int it0 = 0; it0 < iters; it0 += 2 * UN) {
            load_block(nxt, wp, it0 + UN);        // zeros past the end of the row
            step(cur, it0, c, c2);
            load_block(cur, wp, it0 + 2 * UN);
            step(nxt, it0 + UN, c, c2);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) c[q] += c2[q];
        // next task's first block (if any) while this task's results are written
        const int next_task = task + gridDim.x * nwarps;
        if (next_task < tasks) { wp = row_ptr(next_task); load_block(cur, wp, 0); }
        // c[0], c[1]: token g, channels n_base + 2 tig, + 1;  c[2], c[3]: token g + 8
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int m = g + 8 * h;
            if (m >= M) continue;
            RowTerm rt{0.f, 0, 0};
            if (!ep.raw_acc) rt = make_row_term(ep.a_scale, ep.a_zero, ep.a_rowsum, m);
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int n = n_base + 2 * tig + e;
                if (n >= N) continue;
                const int acc = c[2 * h + e];
                const size_t o = size_t(m) * N + n;
                if (ep.raw_acc) {
                    static_cast<int32_t*>(ep.out)[o] = acc;
                } else {
                    const ColTerm ct = make_col_term(ep.w_scale, ep.w_zero, ep.w_colsum, ep.bias, K, n);
                    const float f = dequant(acc, rt, ct);
                    if (ep.out_dtype == QLLM_F32) static_cast<float*>(ep.out)[o] = f;
                    else static_cast<__nv_bfloat16*>(ep.out)[o] = __float2bfloat16_rn(f);
                }
            }
        }
    }
}

// Warps per CTA (one CTA per SM) that waste the fewest warp-slots in the last wave.
int pick_warps(int tasks, int sms) {
    int best = kMaxWarps;
    double best_eff = 0.0;
    for (int wpc = kMaxWarps; wpc >= 8; --wpc) {
        const int64_t slots = int64_t(sms) * wpc;
        const int64_t waves = (tasks + slots - 1) / slots;
        const double eff = double(tasks) / double(waves * slots);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = wpc; }
    }
    return best;
}

template <bool WP, bool M16>
int launch(const uint8_t* a, const uint8_t* w, int M, int N, int K, int a_bits, const EpilogueArgs& ep,
           cudaStream_t st) {
    auto kern = qgemm_decode_kernel<WP, M16>;
    // + slack: the last steps of a row may read token fragments up to 8 iterations (1 KB) past the last row
    const size_t smem = size_t(M16 ? 16 : 8) * size_t(K + (WP ? 16 : 64)) + 1024;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    const int tasks = (N + 7) / 8;
    const int sms = device_sm_count();
    const int grid = std::min(sms, tasks);
    const int wpc = tasks <= sms * 8 ? 8 : pick_warps(tasks, sms);
    QLLM_CUDA_TRY(launch_dependent(kern, dim3(grid), dim3(32 * wpc), smem, st, a, w, M, N, K, a_bits, ep, tasks));
    return after_launch();
}

}  // namespace

bool qgemm_decode_supported(int64_t M, int N, int K, int a_bits, int w_bits) {
    (void)a_bits; (void)w_bits;
    if (M < 1 || M > 16 || N < 1 || K % 128 != 0) return false;
    return size_t(16) * size_t(K + 64) + 1024 <= 200 * 1024;
}

int launch_qgemm_decode(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, int a_bits, int w_bits,
                        const EpilogueArgs& ep, cudaStream_t st) {
    const bool wp = w_bits == 4, m16 = M > 8;
    if (wp) return m16 ? launch<true, true>(a, w, int(M), N, K, a_bits, ep, st)
                       : launch<true, false>(a, w, int(M), N, K, a_bits, ep, st);
    return m16 ? launch<false, true>(a, w, int(M), N, K, a_bits, ep, st)
               : launch<false, false>(a, w, int(M), N, K, a_bits, ep, st);
}

}  // namespace qllm
