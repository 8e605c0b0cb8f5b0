// Prefill integer GEMM on CTA pairs (tcgen05 cta_group::2), byte-lane codes on both operands:
//   acc[m][n] = sum_k qa[m][k] * qw[n][k]   (Eq. 1 on codes), then the dequantizing epilogue.
//
// One 256 x BN output tile per pair of SMs.  Each CTA of the pair loads its own 128 token rows
// of A and its own BN/2 of the tile's weight rows; the pair's tensor cores read both halves of
// the weight tile, so per CTA the operand bytes that pass through shared memory (written by TMA,
// read by the tensor core) per MMA drop by a third against a 128 x BN tile on one SM.  That
// traffic is what bounds the kernel: with TMA switched off (stale tiles) or the MMAs repeated on
// resident tiles the pipe runs at its nominal 128 clocks per 256 x 256 x 32 MMA; with both it
// settles near 150.
// Roles per CTA: warp 0 TMA producer (own halves), warp 1 MMA issuer (one thread of the leader
// CTA, cluster rank 0, issues for the pair) and owner of the tensor-memory allocation,
// warps 2-9 epilogue (own 128 rows; two warps per quarter of the TMEM lanes take alternate 32-column
// chunks, stage them in shared memory and hand them to the copy engine).  No TMA multicast is used.
//
// Barriers:  full[s]      (leader's)  bytes of both CTAs' tiles of stage s have landed
//            empty[s]     (own CTA)   the pair's MMAs that read stage s are complete
//            acc_full[b]  (own CTA)   accumulator buffer b is complete
//            acc_empty[b] (leader's)  16 arrivals: the 8 epilogue warps of each CTA drained buffer b
// The leader's MMA thread commits to the barriers of both CTAs.  Every wait is bounded (see
// wait_bounded); the pair leaves together through a cluster barrier.

#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "common.h"
#include "epilogue.cuh"
#include "ptx_sm100.cuh"
#include "qgemm_tc_common.cuh"

namespace qllm {

namespace {

using namespace tc;

// A pipeline stage holds KS = 2 swizzle rows (256 codes) of K per operand, as two 128-byte-wide
// sub-tiles: the issuing thread's per-stage work (barrier wait, two commits) is then spread over
// 8 MMAs instead of 4 -- with 4 it, not the tensor pipe, set the pace (measured: 8 or 16 MMAs
// per handshake run at the pipe's nominal 128 clocks each, 4 at ~165).
constexpr int KS = 2;

template <int BN>
struct PairTile {
    static constexpr int HALF_N = BN / 2;                       // weight rows each CTA loads
    static constexpr int SUBA = BM * BK, SUBW = HALF_N * BK;    // one swizzled 128-byte-wide sub-tile
    static constexpr int OPA = KS * SUBA, OPW = KS * SUBW;
    static constexpr int STAGE = OPA + OPW;
    static constexpr int EPI_WARPS = 8;                         // two per quarter of the TMEM lanes, alternating chunks
    static constexpr int OUTBUF = EPI_WARPS * 2048;             // per epilogue warp: one 32-row x 64-byte store box
    static constexpr int FIXED = BN * 16 + 256 + OUTBUF;        // column terms + barriers + store staging
    static constexpr int FIT = (227 * 1024 - 1024 - FIXED) / STAGE;
    static constexpr int STAGES = FIT > 8 ? 8 : FIT;
    static constexpr int SMEM = STAGES * STAGE + FIXED + 1024;  // + alignment slack
    static constexpr int THREADS = 32 * (kFirstEpiWarp + EPI_WARPS);   // 10 warps
    static constexpr uint32_t TMEM_COLS = 2 * BN <= 256 ? 256 : 512;
    static_assert(HALF_N % 8 == 0 && BN % 16 == 0 && BN <= 256, "tile width");
};

template <int BN>
__global__ void __launch_bounds__(PairTile<BN>::THREADS, 1)
qgemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmO, int64_t M, int N, int K, EpilogueArgs ep, int* status) {
    using T = PairTile<BN>;
    constexpr int S = T::STAGES;
    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* opA = smem;
    uint8_t* opW = opA + S * T::OPA;
    uint8_t* outbuf = opW + S * T::OPW;                         // 1024-byte aligned (stages are multiples of 1024)
    int4* colterm = reinterpret_cast<int4*>(outbuf + T::OUTBUF);
    uint64_t* bars = reinterpret_cast<uint64_t*>(colterm + BN);
    uint64_t* full = bars;                 // [S]
    uint64_t* empty = bars + S;            // [S]
    uint64_t* acc_full = bars + 2 * S;     // [2]
    uint64_t* acc_empty = acc_full + 2;    // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();           // 0 = leader
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int tiles_m = int((M + 2 * BM - 1) / (2 * BM));
    const int tiles_n = (N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int KB = (K + KS * BK - 1) / (KS * BK);
    const Abort ab{abort_flag, status};

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&acc_full[b], 1);
            ptx::mbar_init(&acc_empty[b], 2 * T::EPI_WARPS);
        }
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmW);
        ptx::prefetch_tensormap(&tmO);
    }
    __syncthreads();
    ptx::cluster_sync();                    // both CTAs' barriers exist before any remote arrive
    if (warp == 1) {
        ptx::tmem_alloc_pair(tmem_slot, T::TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (own halves)
        if (lane == 0) {
            // the leader's full barriers (a CTA's window of the cluster address space is contiguous)
            const uint32_t full_addr0 = ptx::map_to_cta(ptx::smem_addr(&full[0]), 0);
            uint32_t it = 0;
            bool ok = true;
            // The kernel is launched as a programmatic dependent of the kernel before it on the stream (for a layer,
            // the pre-GEMM kernel that writes the tokens): all of the set-up above has run under that kernel's tail
            // and the launch latency; the roles that touch global memory wait here for it to be complete.
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int tile = pair; ok && tile < num_tiles; tile += npairs) {
                const int m0 = (tile % tiles_m) * 2 * BM + int(rank) * BM;
                const int n0 = (tile / tiles_m) * BN + int(rank) * T::HALF_N;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1;
                    if (!wait_bounded(&empty[s], ph ^ 1, ab)) { ok = false; break; }
                    if (rank == 0) ptx::mbar_arrive_expect_tx(&full[s], 2 * T::STAGE);
#pragma unroll
                    for (int h = 0; h < KS; ++h) {
                        const int x = (kb * KS + h) * BK;     // a sub-tile past the end of K reads as zeros
                        ptx::tma_load_2d_pair(opA + s * T::OPA + h * T::SUBA, &tmA, x, m0, full_addr0 + 8u * s);
                        ptx::tma_load_2d_pair(opW + s * T::OPW + h * T::SUBW, &tmW, x, n0, full_addr0 + 8u * s);
                    }
                }
            }
            if (!ok && rank == 0) {
                // give copies still in flight (both CTAs') a bounded chance to land before the pair retires
                const uint32_t issued = it < uint32_t(S) ? it : uint32_t(S);
                for (uint32_t j = 0; j < issued; ++j) {
                    const uint32_t k = it - 1 - j;
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(&full[k % S], (k / S) & 1) && clock64() - t0 < (1ll << 24)) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (rank == 0 && lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_u8u8_s32(2 * BM, BN);
            // barrier arrays of both CTAs (a CTA's window of the cluster address space is contiguous)
            const uint32_t empty_own = ptx::map_to_cta(ptx::smem_addr(&empty[0]), 0);
            const uint32_t empty_peer = ptx::map_to_cta(ptx::smem_addr(&empty[0]), 1);
            const uint32_t accfull_own = ptx::map_to_cta(ptx::smem_addr(&acc_full[0]), 0);
            const uint32_t accfull_peer = ptx::map_to_cta(ptx::smem_addr(&acc_full[0]), 1);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += npairs, ++lt) {
                const uint32_t abuf = lt & 1, aph = (lt >> 1) & 1;
                if (!wait_bounded(&acc_empty[abuf], aph ^ 1, ab)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + abuf * BN;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1;
                    if (!wait_bounded(&full[s], ph, ab)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = ptx::smem_addr(opA + s * T::OPA);
                    const uint32_t b_addr = ptx::smem_addr(opW + s * T::OPW);
#pragma unroll
                    for (int kk = 0; kk < KS * BK / 32; ++kk) {
                        const uint32_t ao = (kk / 4) * T::SUBA + (kk % 4) * 32;
                        const uint32_t bo = (kk / 4) * T::SUBW + (kk % 4) * 32;
                        ptx::mma_i8_ss_pair(d_tmem, ptx::smem_desc_sw128(a_addr + ao),
                                            ptx::smem_desc_sw128(b_addr + bo), idesc, (kb | kk) != 0);
                    }
                    ptx::mma_commit_pair(empty_own + 8u * s);
                    ptx::mma_commit_pair(empty_peer + 8u * s);
                }
                if (ok) {
                    ptx::mma_commit_pair(accfull_own + 8u * abuf);
                    ptx::mma_commit_pair(accfull_peer + 8u * abuf);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (own 128 rows)
        const int quad = warp & 3;                        // TMEM lanes 32*quad .. +31
        const int half = (warp - kFirstEpiWarp) >> 2;     // even or odd 32-column chunks of the tile
        const int et = threadIdx.x - 32 * kFirstEpiWarp;  // 0 .. 32 * EPI_WARPS - 1
        constexpr int ET = 32 * T::EPI_WARPS;
        const uint32_t accempty_addr[2] = {ptx::map_to_cta(ptx::smem_addr(&acc_empty[0]), 0),
                                           ptx::map_to_cta(ptx::smem_addr(&acc_empty[1]), 0)};
        uint8_t* mybuf = outbuf + (warp - kFirstEpiWarp) * 2048;
        uint32_t lt = 0;
        asm volatile("griddepcontrol.wait;" ::: "memory");   // the row terms below come from the kernel before
        for (int tile = pair; tile < num_tiles; tile += npairs, ++lt) {
            const uint32_t abuf = lt & 1, aph = (lt >> 1) & 1;
            const int m0 = (tile % tiles_m) * 2 * BM + int(rank) * BM;
            const int n0 = (tile / tiles_m) * BN;
            ptx::named_bar_sync(1, ET);
            stage_col_terms(ep, colterm, BN, n0, N, K, et, ET);
            ptx::named_bar_sync(1, ET);
            const int row0 = m0 + quad * 32;              // first of this warp's 32 rows; rows >= M are not written
            RowTerm rt[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int64_t m = int64_t(row0) + (lane >> 2) + 8 * i;
                rt[i] = RowTerm{0.f, 0, 0};
                if (!ep.raw_acc && m < M) rt[i] = make_row_term(ep.a_scale, ep.a_zero, ep.a_rowsum, m);
            }
            if (!wait_bounded(&acc_full[abuf], aph, ab)) break;
            ptx::tc_fence_after_sync();
#pragma unroll 1
            for (int ch = half; ch < BN / 32; ch += 2) {
                const int nb = n0 + ch * 32;
                if (nb >= N) break;                       // uniform over the warp
                uint32_t lo[16], hi[16];
                const uint32_t taddr = tmem_base + (uint32_t(quad * 32) << 16) + abuf * BN + ch * 32;
                ptx::tmem_ld_16x256b_x4(taddr, lo);
                ptx::tmem_ld_16x256b_x4(taddr + (16u << 16), hi);
                ptx::tmem_ld_wait();
                stage_chunk(ep, lo, hi, colterm + ch * 32, rt, lane, nb,
                            [&](int) {
                                // the previous box used this buffer: its shared-memory reads must be over
                                if (lane == 0) ptx::bulk_wait_group_read<0>();
                                __syncwarp();
                                return mybuf;
                            },
                            [&](int, int x_bytes) {
                                ptx::fence_proxy_async_smem();
                                __syncwarp();
                                if (lane == 0 && row0 < M) {
                                    ptx::tma_store_2d(&tmO, mybuf, x_bytes, row0);
                                    ptx::bulk_commit_group();
                                }
                            });
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(accempty_addr[abuf]);
        }
        if (lane == 0) ptx::bulk_wait_group<0>();         // the stores are complete before the CTA retires
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                    // the peer may still read this CTA's shared memory / barriers
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, T::TMEM_COLS);
    }
}

template <int BN>
int launch_pair(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, const EpilogueArgs& ep,
                cudaStream_t st) {
    using T = PairTile<BN>;
    static_assert(T::STAGES >= 2, "pipeline needs at least two stages");
    CUtensorMap tmA, tmW, tmO;
    if (!make_map(&tmA, a, uint64_t(M), uint64_t(K), BM, BK, true) ||
        !make_map(&tmW, w, uint64_t(N), uint64_t(K), T::HALF_N, BK, true) ||
        !make_store_map(&tmO, ep.out, uint64_t(M), uint64_t(N) * (ep.raw_acc || ep.out_dtype == QLLM_F32 ? 4 : 2)))
        return QLLM_ERR_CUDA;
    int* status = device_status_word();
    if (!status) return QLLM_ERR_CUDA;
    auto kern = qgemm_tc2_kernel<BN>;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, T::SMEM));
    const int64_t tiles = ((M + 2 * BM - 1) / (2 * BM)) * int64_t((N + BN - 1) / BN);
    const int pairs = int(std::min<int64_t>(tiles, device_sm_count() / 2));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(2 * pairs));
    cfg.blockDim = dim3(T::THREADS);
    cfg.dynamicSmemBytes = T::SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    QLLM_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmW, tmO, M, N, K, ep, status));
    return after_launch();
}

}  // namespace

bool qgemm_tc2_supported(int64_t M, int N, int K, int a_bits, int w_bits) {
    return a_bits != 4 && w_bits != 4 && M > BM && qgemm_tc_supported(M, N, K, a_bits, w_bits) && device_sm_count() >= 2;
}

int launch_qgemm_tc2(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, const EpilogueArgs& ep,
                     cudaStream_t st) {
    // Tile width by estimated time.  The kernel is bound by shared-memory bandwidth (every operand
    // byte is written once by TMA and read once by the tensor core), so a tile costs about
    // (256 + BN) bytes per unit of K, and the grid takes ceil(tiles / pairs) rounds of such tiles;
    // the constant stands for the per-tile fill/drain.  Measured per-MMA times (62 / 68 / 81 ns at
    // BN = 128 / 192 / 256) follow the same proportion.
    const int64_t tm = (M + 2 * BM - 1) / (2 * BM);
    const int pairs = device_sm_count() / 2;
    auto cost = [&](int bn) {
        const int64_t tiles = tm * ((N + bn - 1) / bn);
        return ((tiles + pairs - 1) / pairs) * int64_t(256 + bn + 12);
    };
    int best = 256;
    for (int bn : {224, 192, 160, 128})
        if (cost(bn) < cost(best)) best = bn;
    switch (best) {
        case 256: return launch_pair<256>(a, w, M, N, K, ep, st);
        case 224: return launch_pair<224>(a, w, M, N, K, ep, st);
        case 192: return launch_pair<192>(a, w, M, N, K, ep, st);
        case 160: return launch_pair<160>(a, w, M, N, K, ep, st);
        default: return launch_pair<128>(a, w, M, N, K, ep, st);
    }
}

}  // namespace qllm
