// Prefill integer GEMM on the 5th-generation tensor cores (tcgen05, kind::i8) with the
// dequantizing epilogue:   acc[m][n] = sum_k qa[m][k] * qw[n][k]   (Eq. 1 on codes).
//
// One persistent CTA per SM walks 128 x BN output tiles.  Warp roles:
//   warp 0      TMA producer: tiles of both operands, BK = 128 codes of K per stage
//   warp 1      MMA issuer (one thread) and owner of the tensor-memory allocation
//   warps 2-5   epilogue: TMEM -> registers -> dequantize -> global (one TMEM lane quadrant each)
//   warps 6-13  (4-bit operands only) unpack nibbles to bytes in shared memory
// Operands reach the tensor core K-major with the 128-byte swizzle.  Byte-lane codes (6/8 bit)
// are written in that form by TMA itself; packed 4-bit codes land in a plain staging tile and
// the unpack warps expand them.  Both operands put the even nibbles of each 32-code chunk in
// one 16-byte unit and the odd nibbles in the next, so the expansion is a mask and a shift and
// the dot product over K is unchanged (same permutation on both sides).
// Accumulators live in tensor memory, double-buffered so that the epilogue of tile i overlaps
// the MMAs of tile i+1.  Every mbarrier wait is bounded: on expiry the kernel raises the
// library's device status word, all roles leave their loops, TMEM is freed, and the kernel ends.

#include <cuda.h>
#include <cuda_bf16.h>

#include "common.h"
#include "epilogue.cuh"
#include "ptx_sm100.cuh"
#include "qgemm_tc_common.cuh"

namespace qllm {

namespace {

using namespace tc;

template <int BN, bool AP, bool WP>
struct Tile {
    static constexpr int OPA = BM * BK, OPW = BN * BK;                  // swizzled byte tiles
    static constexpr int RAWA = AP ? BM * BK / 2 : 0, RAWW = WP ? BN * BK / 2 : 0;
    static constexpr int STAGE = OPA + OPW + RAWA + RAWW;
    static constexpr int FIXED = BN * 16 + 256;                          // column terms + barriers
    static constexpr int STAGES = (227 * 1024 - 1024 - FIXED) / STAGE > 6 ? 6 : (227 * 1024 - 1024 - FIXED) / STAGE;
    static constexpr int SMEM = STAGES * STAGE + FIXED + 1024;           // + alignment slack
    static constexpr int THREADS = (AP || WP) ? 32 * (kFirstUnpackWarp + kUnpackWarps) : 32 * kFirstUnpackWarp;
    static constexpr int OP_ARRIVALS = ((AP || WP) ? kUnpackWarps : 0) + ((!AP || !WP) ? 1 : 0);
    static constexpr uint32_t TMEM_COLS = 2 * BN <= 32 ? 32 : (2 * BN <= 64 ? 64 : (2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512)));
};

template <int BN, bool AP, bool WP>
__global__ void __launch_bounds__(Tile<BN, AP, WP>::THREADS, 1)
qgemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                int64_t M, int N, int K, EpilogueArgs ep, int* status, uint32_t opa_tx, int early_w) {
    using T = Tile<BN, AP, WP>;
    constexpr int S = T::STAGES;
    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* opA = smem;
    uint8_t* opW = opA + S * T::OPA;
    uint8_t* rawA = opW + S * T::OPW;
    uint8_t* rawW = rawA + S * T::RAWA;
    int4* colterm = reinterpret_cast<int4*>(rawW + S * T::RAWW);
    uint64_t* bars = reinterpret_cast<uint64_t*>(colterm + BN);
    uint64_t* full_raw = bars;             // [S] TMA -> unpack warps
    uint64_t* full_op = bars + S;          // [S] operands ready for the MMA
    uint64_t* empty = bars + 2 * S;        // [S] MMAs that read the stage have completed
    uint64_t* acc_full = bars + 3 * S;     // [2]
    uint64_t* acc_empty = acc_full + 2;    // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = int((M + BM - 1) / BM);
    const int tiles_n = (N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int KB = (K + BK - 1) / BK;
    const Abort ab{abort_flag, status};

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(&full_raw[s], 1);
            ptx::mbar_init(&full_op[s], T::OP_ARRIVALS);
            ptx::mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&acc_full[b], 1);
            ptx::mbar_init(&acc_empty[b], 4);
        }
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmW);
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, T::TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // The kernel is launched as a programmatic dependent of the kernel before it on the stream (for a layer, the
    // pre-GEMM kernel that writes the tokens): everything above touched no global memory and has run under that
    // kernel and the launch latency.  Every role that touches global memory waits for that kernel to be complete
    // (griddepcontrol.wait) before it does; with early_w (the caller vouches that no kernel before this one on the
    // stream writes the weights: a layer's own weights) the producer first asks for the weight tiles of its first
    // stages, so that they travel while the tokens are still being written.

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0, pre = 0;
            bool ok = true;
            if (early_w && int(blockIdx.x) < num_tiles) {
                // the first stages of the first tile: barriers armed for both operands, weight copies on their way
                const int n0 = (int(blockIdx.x) / tiles_m) * BN;
                pre = uint32_t(KB < S ? KB : S);
                for (uint32_t kb = 0; kb < pre; ++kb) {
                    if (AP || WP) ptx::mbar_arrive_expect_tx(&full_raw[kb], T::RAWA + T::RAWW);
                    if (!AP || !WP) ptx::mbar_arrive_expect_tx(&full_op[kb], (AP ? 0 : opa_tx) + (WP ? 0 : T::OPW));
                    if (WP) ptx::tma_load_2d(rawW + kb * T::RAWW, &tmW, int(kb) * (BK / 2), n0, &full_raw[kb]);
                    else    ptx::tma_load_2d(opW + kb * T::OPW, &tmW, int(kb) * BK, n0, &full_op[kb]);
                }
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1;
                    if (it >= pre) {
                        if (!wait_bounded(&empty[s], ph ^ 1, ab)) { ok = false; break; }
                        if (AP || WP) ptx::mbar_arrive_expect_tx(&full_raw[s], T::RAWA + T::RAWW);
                        if (!AP || !WP) ptx::mbar_arrive_expect_tx(&full_op[s], (AP ? 0 : opa_tx) + (WP ? 0 : T::OPW));
                    }
                    if (AP) ptx::tma_load_2d(rawA + s * T::RAWA, &tmA, kb * (BK / 2), m0, &full_raw[s]);
                    else    ptx::tma_load_2d(opA + s * T::OPA, &tmA, kb * BK, m0, &full_op[s]);
                    if (it >= pre) {
                        if (WP) ptx::tma_load_2d(rawW + s * T::RAWW, &tmW, kb * (BK / 2), n0, &full_raw[s]);
                        else    ptx::tma_load_2d(opW + s * T::OPW, &tmW, kb * BK, n0, &full_op[s]);
                    }
                }
            }
            if (!ok) {
                // give copies still in flight a bounded chance to land before the CTA retires
                const uint32_t issued = it < uint32_t(S) ? it : uint32_t(S);
                for (uint32_t j = 0; j < issued; ++j) {
                    const uint32_t k = it - 1 - j;
                    uint64_t* b = (AP || WP) ? &full_raw[k % S] : &full_op[k % S];
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(b, (k / S) & 1) && clock64() - t0 < (1ll << 24)) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_u8u8_s32(BM, BN);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++lt) {
                const uint32_t abuf = lt & 1, aph = (lt >> 1) & 1;
                if (!wait_bounded(&acc_empty[abuf], aph ^ 1, ab)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + abuf * BN;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1;
                    if (!wait_bounded(&full_op[s], ph, ab)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = ptx::smem_addr(opA + s * T::OPA);
                    const uint32_t b_addr = ptx::smem_addr(opW + s * T::OPW);
#pragma unroll
                    for (int kk = 0; kk < BK / 32; ++kk)
                        ptx::mma_i8_ss(d_tmem, ptx::smem_desc_sw128(a_addr + kk * 32),
                                       ptx::smem_desc_sw128(b_addr + kk * 32), idesc, (kb | kk) != 0);
                    ptx::mma_commit(&empty[s]);
                }
                if (ok) ptx::mma_commit(&acc_full[abuf]);
            }
        }
    } else if (warp < kFirstUnpackWarp) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;                        // TMEM lanes 32*quad .. +31
        const int et = threadIdx.x - 32 * kFirstEpiWarp;  // 0..127
        uint32_t lt = 0;
        asm volatile("griddepcontrol.wait;" ::: "memory");   // the row terms below come from the kernel before
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++lt) {
            const uint32_t abuf = lt & 1, aph = (lt >> 1) & 1;
            const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
            ptx::named_bar_sync(1, 128);
            stage_col_terms(ep, colterm, BN, n0, N, K, et, 128);
            ptx::named_bar_sync(1, 128);
            const int64_t m = int64_t(m0) + quad * 32 + lane;
            RowTerm rt{0.f, 0, 0};
            if (!ep.raw_acc && m < M) rt = make_row_term(ep.a_scale, ep.a_zero, ep.a_rowsum, m);
            if (!wait_bounded(&acc_full[abuf], aph, ab)) break;
            ptx::tc_fence_after_sync();
#pragma unroll 1
            for (int ch = 0; ch < BN / 32; ++ch) {
                const int nb = n0 + ch * 32;
                if (nb >= N) break;                       // uniform over the CTA
                uint32_t r[32];
                ptx::tmem_ld_32x32b_x32(tmem_base + (uint32_t(quad * 32) << 16) + abuf * BN + ch * 32, r);
                ptx::tmem_ld_wait();
                if (m < M) store_chunk(ep, r, colterm + ch * 32, rt, m, N, nb);
                __syncwarp();   // reconverge before the next warp-wide TMEM load
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&acc_empty[abuf]);
        }
    } else {
        // ------------------------------------------------------------------ unpack (4-bit operands)
        if (AP || WP) {
            const int t = threadIdx.x - 32 * kFirstUnpackWarp;
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1;
                    if (!wait_bounded(&full_raw[s], ph, ab)) { ok = false; break; }
                    if (AP) unpack_tile<BM, AP && WP>(rawA + s * T::RAWA, opA + s * T::OPA, t);
                    if (WP) unpack_tile<BN, AP && WP>(rawW + s * T::RAWW, opW + s * T::OPW, t);
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&full_op[s]);
                }
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, T::TMEM_COLS);
    }
}

template <int BN, bool AP, bool WP>
int launch(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, const EpilogueArgs& ep, cudaStream_t st,
           bool early_w) {
    using T = Tile<BN, AP, WP>;
    static_assert(T::STAGES >= 2, "pipeline needs at least two stages");
    CUtensorMap tmA, tmW;
    // Byte-lane tokens: the box covers only the rows that exist (32 or 64 of the tile's 128 when there are no
    // more tokens).  The rest of the operand tile keeps whatever shared memory held; it only reaches accumulator
    // rows that are never stored.  Fewer bytes cross shared memory per stage, and a tensor of fewer than 32
    // rows under a 128-row box measured 5.5 us slower per call than one of 32.
    const uint32_t a_rows = AP ? BM : (M <= 32 ? 32 : (M <= 64 ? 64 : BM));
    const bool okA = AP ? make_map(&tmA, a, uint64_t(M), uint64_t(K / 2), BM, BK / 2, false)
                        : make_map(&tmA, a, uint64_t(M), uint64_t(K), a_rows, BK, true);
    const bool okW = WP ? make_map(&tmW, w, uint64_t(N), uint64_t(K / 2), BN, BK / 2, false)
                        : make_map(&tmW, w, uint64_t(N), uint64_t(K), BN, BK, true);
    if (!okA || !okW) return QLLM_ERR_CUDA;
    int* status = device_status_word();
    if (!status) return QLLM_ERR_CUDA;
    auto kern = qgemm_tc_kernel<BN, AP, WP>;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, T::SMEM));
    const int64_t tiles = ((M + BM - 1) / BM) * int64_t((N + BN - 1) / BN);
    const int grid = int(std::min<int64_t>(tiles, device_sm_count()));
    QLLM_CUDA_TRY(launch_dependent(kern, dim3(grid), dim3(T::THREADS), T::SMEM, st, tmA, tmW, M, N, K, ep, status,
                                   uint32_t(a_rows * BK), early_w ? 1 : 0));
    return after_launch();
}

}  // namespace

bool qgemm_tc_supported(int64_t M, int N, int K, int a_bits, int w_bits) {
    (void)a_bits; (void)w_bits;
    return M >= 1 && M < (int64_t(1) << 31) - BM && K % 32 == 0 && N % 8 == 0 && encode_fn() != nullptr;
}

int launch_qgemm_tc(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, int a_bits, int w_bits,
                    const EpilogueArgs& ep, cudaStream_t st, bool weights_static) {
    const bool ap = a_bits == 4, wp = w_bits == 4;
    if (!ap && !wp && qgemm_tc2_supported(M, N, K, a_bits, w_bits)) return launch_qgemm_tc2(a, w, M, N, K, ep, st);
    // Tile width by estimated time: rounds of tiles over the SMs x what one tile costs per unit of K.  Byte-lane
    // operands cost their TMA bytes; a packed operand costs its rows again in the unpack warps, the 128 token
    // rows in every tile, so few tokens with packed weights want narrow tiles that reach every SM.
    const int64_t tm = (M + BM - 1) / BM;
    const int sms = device_sm_count();
    auto cost = [&](int bn) {
        const int64_t tiles = tm * ((N + bn - 1) / bn);
        return ((tiles + sms - 1) / sms) * int64_t((ap ? 2 * BM : BM / 2) + (wp ? 2 * bn : bn / 2) + 24);
    };
    int best = 256;
    for (int bn : {192, 160, 128, 96, 64})
        if (cost(bn) < cost(best)) best = bn;
#define QLLM_TC(BN_, AP_, WP_) launch<BN_, AP_, WP_>(a, w, M, N, K, ep, st, weights_static)
#define QLLM_TC_BN(AP_, WP_) \
    (best == 256 ? QLLM_TC(256, AP_, WP_) : best == 192 ? QLLM_TC(192, AP_, WP_) : best == 160 ? QLLM_TC(160, AP_, WP_) : \
     best == 128 ? QLLM_TC(128, AP_, WP_) : best == 96 ? QLLM_TC(96, AP_, WP_) : QLLM_TC(64, AP_, WP_))
    if (ap && wp) return QLLM_TC_BN(true, true);
    if (!ap && !wp) return QLLM_TC_BN(false, false);
    if (ap) return QLLM_TC_BN(true, false);
    return QLLM_TC_BN(false, true);
#undef QLLM_TC_BN
#undef QLLM_TC
}

}  // namespace qllm
