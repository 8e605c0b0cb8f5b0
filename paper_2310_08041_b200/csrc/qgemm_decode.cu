// Decode-sized integer GEMM (M <= 16 tokens): a weight-streaming kernel.  The weight codes
// (N*K/2 bytes for 4-bit) are read from HBM exactly once with 128-bit streaming loads; the few
// token rows are expanded to byte codes in shared memory once per CTA and reused by every
// weight row.  The kernel is HBM-bound, so the contraction runs on the warp-level integer MMA
// (m16n8k32, u8 x u8 -> s32): sixteen output channels of weights are the 16-row operand (a 32-bit
// register of packed nibbles becomes two operand registers with one mask and one shift+mask),
// eight tokens are the 8-column operand read from shared memory; tokens 8..15 take a second MMA
// on the same weight registers.  Up to eight tokens this is half the MMAs of the opposite
// assignment (tokens as the 16-row operand), and the integer MMA pipe, not HBM, is what that
// assignment ran into.  Plain dp4a would need ~2 M integer instructions per 8 weight codes and
// turn ALU-bound at M = 8..16; tcgen05 tiles (128 rows) would be 8x padding at these M.
//
// Work split: one task = 16 consecutive output channels; the two warps of a pair take one half
// of K each and join their exact integer sums through shared memory (no global scratch, no
// atomics).  One CTA per SM; the number of warp pairs per CTA is chosen on the host so that tasks
// fill whole waves.  K order inside a task is permuted (each thread walks its own 16-byte column
// of two rows); both operands follow the same order, so every sum is exact.

#include <cuda_bf16.h>

#include "common.h"
#include "epilogue.cuh"

namespace qllm {

namespace {

constexpr int kMaxWarps = 20;

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
// A thread moves 16 bytes of a token row per item and has all its loads in flight before the
// first use: the fill is one trip to memory, not one per item.
template <bool WP>
__device__ void fill_tokens(uint8_t* As, int stride, const uint8_t* __restrict__ a, int M, int K, int a_bits,
                            int rows) {
    const int per_row = (a_bits == 4 ? K / 2 : K) / 16;    // 16-byte items of a token row
    const int total = rows * per_row;
    constexpr int U = 4;                                   // independent loads in flight per thread
    for (int base = threadIdx.x; base < total; base += U * blockDim.x) {
        uint4 v[U];
        int r[U], c[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = base + u * blockDim.x;
            r[u] = idx / per_row;
            c[u] = idx - r[u] * per_row;
            v[u] = make_uint4(0, 0, 0, 0);
            if (idx < total && r[u] < M)
                v[u] = __ldg(reinterpret_cast<const uint4*>(a + size_t(r[u]) * per_row * 16) + c[u]);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (base + u * blockDim.x >= total) break;
            if (a_bits == 4) {
                // 32 codes -> four (even, odd) groups = 32 bytes
                const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                uint32_t o[8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t lo = w[k] & 0x0F0F0F0Fu, hi = (w[k] >> 4) & 0x0F0F0F0Fu;
                    if (WP) { o[2 * k] = lo; o[2 * k + 1] = hi; }
                    else { o[2 * k] = __byte_perm(lo, hi, 0x5140); o[2 * k + 1] = __byte_perm(lo, hi, 0x7362); }
                }
                uint4* dst = reinterpret_cast<uint4*>(As + r[u] * stride + c[u] * 32);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            } else {
                // 16 byte codes = two groups of 8
                uint4 o = v[u];
                if (WP) {
                    o.x = __byte_perm(v[u].x, v[u].y, 0x6420); o.y = __byte_perm(v[u].x, v[u].y, 0x7531);
                    o.z = __byte_perm(v[u].z, v[u].w, 0x6420); o.w = __byte_perm(v[u].z, v[u].w, 0x7531);
                }
                *reinterpret_cast<uint4*>(As + r[u] * stride + c[u] * 16) = o;
            }
        }
    }
}

template <bool WP, bool M16>
__global__ void __launch_bounds__(32 * kMaxWarps, 1)
qgemm_decode_kernel(const uint8_t* __restrict__ a, const uint8_t* __restrict__ w, int M, int N, int K,
                    int a_bits, EpilogueArgs ep, int tasks) {
    extern __shared__ __align__(16) uint8_t As[];
    constexpr int PAD = WP ? 16 : 64;             // keeps the 16-byte fragment loads conflict-free
    constexpr int UN = 2;                         // iterations per register buffer (3 buffers in flight)
    constexpr int NT = M16 ? 16 : 8;              // token rows held in shared memory
    const int stride = K + PAD;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = lane >> 2, tig = lane & 3;
    const int row_bytes = WP ? K / 2 : K;
    const int iters = row_bytes / 64;             // 4 threads x 16 bytes of a row per iteration
    // the two warps of a pair stream the two halves of K for the same 16 output channels
    const int khalf = warp & 1, pair = warp >> 1, npairs = nwarps >> 1;
    const int half_it = (iters + 1) >> 1;
    const int it_begin = khalf * half_it, it_end = khalf ? iters : half_it;
    const uint8_t* t_lo = As + g * stride;        // token g
    const uint8_t* t_hi = As + (g + 8) * stride;  // token g + 8 (M16 only)
    int* xch = reinterpret_cast<int*>(As + size_t(NT) * stride + 1024) + (pair * 32 + lane) * 8;

    // thread (g, tig) reads column tig of weight rows n_base + g and n_base + g + 8
    auto row_ptr = [&](int task, int h) {
        const int n_ld = min(task * 16 + g + 8 * h, N - 1);   // rows past N re-read the last row; never stored
        return reinterpret_cast<const uint4*>(w + size_t(n_ld) * row_bytes) + tig;
    };
    auto load_block = [&](uint4 (&b0)[UN], uint4 (&b1)[UN], const uint4* w0, const uint4* w1, int it0) {
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const bool in = it0 + u < it_end;
            b0[u] = in ? __ldcs(w0 + 4 * (it0 + u)) : make_uint4(0, 0, 0, 0);
            b1[u] = in ? __ldcs(w1 + 4 * (it0 + u)) : make_uint4(0, 0, 0, 0);
        }
    };

    // The kernel is launched as a programmatic dependent of the kernel before it (the pre-GEMM kernel that writes
    // the tokens): until that kernel is complete (griddepcontrol.wait) it only asks for the weight rows of its
    // first task to be brought into L2 -- harmless whoever wrote them -- so the launch latency and the first trip
    // to HBM pass under the previous kernel.  (Requesting register blocks as well before the wait delayed that
    // kernel's own loads and made the step longer; without the L2 requests the step is 1.7 us longer.)
    int task = blockIdx.x * npairs + pair;
    if (task < tasks) {
        const int n_first = min(task * 16, N - 1), n_rows = min(16, N - n_first);
        const char* base = reinterpret_cast<const char*>(w + size_t(n_first) * row_bytes);
        // each warp of the pair asks for its own half of every row
        const int hb = half_it * 64, h0 = khalf * hb, h1 = min(row_bytes, h0 + hb);
        for (int r = 0; r < n_rows; ++r)
            for (int o = h0 + lane * 128; o < h1; o += 32 * 128)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(base + size_t(r) * row_bytes + o));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // first weights are requested before the token rows are expanded: the stream starts at once
    uint4 p0[UN], q0[UN], p1[UN], q1[UN], p2[UN], q2[UN];
    const uint4 *w0 = nullptr, *w1 = nullptr;
    if (task < tasks) {
        w0 = row_ptr(task, 0);
        w1 = row_ptr(task, 1);
        load_block(p0, q0, w0, w1, it_begin);
        load_block(p1, q1, w0, w1, it_begin + UN);
        load_block(p2, q2, w0, w1, it_begin + 2 * UN);
    }
    fill_tokens<WP>(As, stride, a, M, K, a_bits, NT);
    __syncthreads();

    // One step of the stream: UN x 16 bytes of this thread's column of two weight rows against the matching
    // token fragments.  The weights are the 16-row operand (a register of packed nibbles splits into its
    // operand registers with one mask and one shift+mask), eight tokens the 8-column operand; tokens 8..15
    // reuse the weight registers in a second MMA.  Loads past the end of the warp's K range return zeros, so a
    // step needs no bounds test: zero weights add nothing (the token fragments then come from the next rows or
    // the slack behind the last one).  With eight tokens two accumulator sets halve the chain of dependent MMAs.
    auto step = [&](const uint4 (&b0)[UN], const uint4 (&b1)[UN], int it0, int (&c0)[4], int (&c1)[4]) {
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int it = it0 + u;
            const uint4 p = b0[u], q = b1[u];
            if (WP) {
                // 32 codes of this thread's column: words s = 0..3, each -> (even, odd) registers
                const int aoff = (16 * it + 4 * tig) * 8;
                const uint4 T0 = *reinterpret_cast<const uint4*>(t_lo + aoff);
                const uint4 T1 = *reinterpret_cast<const uint4*>(t_lo + aoff + 16);
                constexpr uint32_t F = 0x0F0F0F0Fu;
                mma_u8(c0, p.x & F, q.x & F, (p.x >> 4) & F, (q.x >> 4) & F, T0.x, T0.y);
                mma_u8(M16 ? c0 : c1, p.y & F, q.y & F, (p.y >> 4) & F, (q.y >> 4) & F, T0.z, T0.w);
                mma_u8(c0, p.z & F, q.z & F, (p.z >> 4) & F, (q.z >> 4) & F, T1.x, T1.y);
                mma_u8(M16 ? c0 : c1, p.w & F, q.w & F, (p.w >> 4) & F, (q.w >> 4) & F, T1.z, T1.w);
                if (M16) {
                    const uint4 U0 = *reinterpret_cast<const uint4*>(t_hi + aoff);
                    const uint4 U1 = *reinterpret_cast<const uint4*>(t_hi + aoff + 16);
                    mma_u8(c1, p.x & F, q.x & F, (p.x >> 4) & F, (q.x >> 4) & F, U0.x, U0.y);
                    mma_u8(c1, p.y & F, q.y & F, (p.y >> 4) & F, (q.y >> 4) & F, U0.z, U0.w);
                    mma_u8(c1, p.z & F, q.z & F, (p.z >> 4) & F, (q.z >> 4) & F, U1.x, U1.y);
                    mma_u8(c1, p.w & F, q.w & F, (p.w >> 4) & F, (q.w >> 4) & F, U1.z, U1.w);
                }
            } else {
                // 16 byte codes of this thread's column: two k32 steps
                const int aoff = (4 * it + tig) * 16;
                const uint4 T0 = *reinterpret_cast<const uint4*>(t_lo + aoff);
                mma_u8(c0, p.x, q.x, p.y, q.y, T0.x, T0.y);
                mma_u8(M16 ? c0 : c1, p.z, q.z, p.w, q.w, T0.z, T0.w);
                if (M16) {
                    const uint4 U0 = *reinterpret_cast<const uint4*>(t_hi + aoff);
                    mma_u8(c1, p.x, q.x, p.y, q.y, U0.x, U0.y);
                    mma_u8(c1, p.z, q.z, p.w, q.w, U0.z, U0.w);
                }
            }
        }
    };

    for (; task < tasks; task += gridDim.x * npairs) {
        const int n_base = task * 16;
        // M16: c = tokens 0..7, c2 = tokens 8..15; else two partial sums of tokens 0..7
        int c[4] = {0, 0, 0, 0}, c2[4] = {0, 0, 0, 0};
        // column terms of the epilogue travel while the weights stream
        ColTerm ct[2] = {{0.f, 0, 0, 0.f}, {0.f, 0, 0, 0.f}};
        if (!khalf && !ep.raw_acc) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int n = n_base + g + 8 * h;
                if (n < N) ct[h] = make_col_term(ep.w_scale, ep.w_zero, ep.w_colsum, ep.bias, K, n);
            }
        }
        // three register blocks in flight
        for (int it0 = it_begin; it0 < it_end; it0 += 3 * UN) {
            step(p0, q0, it0, c, c2);
            if (it0 + 3 * UN < it_end) load_block(p0, q0, w0, w1, it0 + 3 * UN);
            if (it0 + UN < it_end) {
                step(p1, q1, it0 + UN, c, c2);
                if (it0 + 4 * UN < it_end) load_block(p1, q1, w0, w1, it0 + 4 * UN);
            }
            if (it0 + 2 * UN < it_end) {
                step(p2, q2, it0 + 2 * UN, c, c2);
                if (it0 + 5 * UN < it_end) load_block(p2, q2, w0, w1, it0 + 5 * UN);
            }
        }
        if (!M16) {
#pragma unroll
            for (int q = 0; q < 4; ++q) c[q] += c2[q];
        }
        // next task's first blocks (if any) while this task's results are written
        const int next_task = task + gridDim.x * npairs;
        if (next_task < tasks) {
            w0 = row_ptr(next_task, 0);
            w1 = row_ptr(next_task, 1);
            load_block(p0, q0, w0, w1, it_begin);
            load_block(p1, q1, w0, w1, it_begin + UN);
            load_block(p2, q2, w0, w1, it_begin + 2 * UN);
        }
        // the second half of K joins the first through shared memory (integer sums: exact in any order)
        const int barid = 1 + pair;
        if (khalf) {
            *reinterpret_cast<int4*>(xch) = make_int4(c[0], c[1], c[2], c[3]);
            if (M16) *reinterpret_cast<int4*>(xch + 4) = make_int4(c2[0], c2[1], c2[2], c2[3]);
        }
        asm volatile("bar.sync %0, 64;" ::"r"(barid) : "memory");
        if (!khalf) {
            const int4 o0 = *reinterpret_cast<const int4*>(xch);
            c[0] += o0.x; c[1] += o0.y; c[2] += o0.z; c[3] += o0.w;
            if (M16) {
                const int4 o1 = *reinterpret_cast<const int4*>(xch + 4);
                c2[0] += o1.x; c2[1] += o1.y; c2[2] += o1.z; c2[3] += o1.w;
            }
        }
        asm volatile("bar.sync %0, 64;" ::"r"(barid) : "memory");   // the words are rewritten by the next task
        if (khalf) continue;
        // c[0], c[1]: channel n_base + g, tokens 2 tig, + 1;  c[2], c[3]: channel n_base + g + 8;  c2: tokens + 8
#pragma unroll
        for (int t = 0; t < (M16 ? 4 : 2); ++t) {
            const int m = 2 * tig + (t & 1) + 8 * (t >> 1);
            if (m >= M) continue;
            RowTerm rt{0.f, 0, 0};
            if (!ep.raw_acc) rt = make_row_term(ep.a_scale, ep.a_zero, ep.a_rowsum, m);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int n = n_base + g + 8 * h;
                if (n >= N) continue;
                const int acc = (t >> 1) ? c2[2 * h + (t & 1)] : c[2 * h + (t & 1)];
                const size_t o = size_t(m) * N + n;
                if (ep.raw_acc) {
                    static_cast<int32_t*>(ep.out)[o] = acc;
                } else {
                    const float f = dequant(acc, rt, ct[h]);
                    if (ep.out_dtype == QLLM_F32) static_cast<float*>(ep.out)[o] = f;
                    else static_cast<__nv_bfloat16*>(ep.out)[o] = __float2bfloat16_rn(f);
                }
            }
        }
    }
}

// Warp pairs per CTA (one CTA per SM) that waste the fewest pair-slots in the last wave.
int pick_pairs(int tasks, int sms) {
    int best = kMaxWarps / 2;
    double best_eff = 0.0;
    for (int ppc = kMaxWarps / 2; ppc >= 4; --ppc) {
        const int64_t slots = int64_t(sms) * ppc;
        const int64_t waves = (tasks + slots - 1) / slots;
        const double eff = double(tasks) / double(waves * slots);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = ppc; }
    }
    return best;
}

template <bool WP, bool M16>
int launch(const uint8_t* a, const uint8_t* w, int M, int N, int K, int a_bits, const EpilogueArgs& ep,
           cudaStream_t st) {
    auto kern = qgemm_decode_kernel<WP, M16>;
    const int tasks = (N + 15) / 16;
    const int sms = device_sm_count();
    const int grid = std::min(sms, tasks);
    const int ppc = tasks <= sms * 4 ? 4 : pick_pairs(tasks, sms);
    // + slack: the last steps of a row may read token fragments up to 8 iterations (1 KB) past the last row;
    // + 1 KB per warp pair for the partial sums of the second half of K
    const size_t smem = size_t(M16 ? 16 : 8) * size_t(K + (WP ? 16 : 64)) + 1024 + size_t(ppc) * 1024;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    QLLM_CUDA_TRY(launch_dependent(kern, dim3(grid), dim3(64 * ppc), smem, st, a, w, M, N, K, a_bits, ep, tasks));
    return after_launch();
}

}  // namespace

bool qgemm_decode_supported(int64_t M, int N, int K, int a_bits, int w_bits) {
    (void)a_bits; (void)w_bits;
    if (M < 1 || M > 16 || N < 1 || K % 128 != 0) return false;
    return size_t(16) * size_t(K + 64) + 1024 + (kMaxWarps / 2) * 1024 <= 200 * 1024;
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
