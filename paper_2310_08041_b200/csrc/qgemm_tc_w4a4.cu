// W4A4 prefill GEMM, tcgen05 kind::i8, packed operands loaded straight to registers.
//
// The 4-bit path of the TMA-staged kernel is bound by the shared-memory pipe: per K-block the packed
// tile is written by TMA, read back by the unpack warps, written again as bytes and read by the MMA.
// Here the load warps fetch the packed nibbles from global memory (L2-resident after the first tile
// row) directly into registers with 128-bit loads and write only the swizzled byte tiles: a third of
// the shared-memory traffic and the TMA hop of the stage latency disappear, and the freed staging
// space gives a fourth pipeline stage.
//   warp 0       MMA issuer (one thread) + tensor-memory allocation
//   warps 1-4    epilogue (TMEM lane quadrant = warp & 3)
//   warps 5-20   load + unpack, in four groups of four warps; group g owns pipeline stage g and the
//                K-blocks it = g, g+4, ...: a group's chain (wait for the stage, expand, proxy fence,
//                arrive, request its next K-block) has four K-block times to complete, and the four
//                groups overlap, so neither the load latency nor the fence sits on the MMA's path
// 128 x 256 tiles, BK = 128 codes, 4 stages of (16 KB A + 32 KB W), accumulators double-buffered in
// 512 TMEM columns.  Both operands use the even/odd-nibble permutation of K (see unpack_tile).

#include <cuda.h>
#include <cuda_bf16.h>

#include "common.h"
#include "epilogue.cuh"
#include "ptx_sm100.cuh"
#include "qgemm_tc_common.cuh"

namespace qllm {

namespace {

using namespace tc;

constexpr int BN = 256;
constexpr int OPA = BM * BK, OPW = BN * BK;
constexpr int STAGE = OPA + OPW;                  // 48 KB
constexpr int S = 4;
constexpr int FIXED = BN * 16 + 256;
constexpr int SMEM = S * STAGE + FIXED + 1024;
constexpr int kEpi0 = 1, kLoad0 = 5, kLoadWarps = 16;
constexpr int kGroups = S;                                // one group of load warps per pipeline stage
constexpr int kGroupWarps = kLoadWarps / kGroups;         // 4 warps = 128 threads per group
constexpr int THREADS = 32 * (kLoad0 + kLoadWarps);
constexpr int CHUNKS_A = BM * 4 / (32 * kGroupWarps);     // 4 per thread
constexpr int CHUNKS_W = BN * 4 / (32 * kGroupWarps);     // 8 per thread
constexpr int ROWS_PER_PASS = 8 * kGroupWarps;            // rows covered by one chunk index over a group
constexpr int CH = CHUNKS_A + CHUNKS_W;

struct Cursor { int tile; int kb; };

// 32 packed codes -> even nibbles to 16-byte unit 2j, odd nibbles to unit 2j+1 of row r (128B swizzle)
__device__ __forceinline__ void expand_store(const uint4 w, uint8_t* tile, int r, int j) {
    uint4 lo, hi;
    lo.x = w.x & 0x0F0F0F0Fu; hi.x = (w.x >> 4) & 0x0F0F0F0Fu;
    lo.y = w.y & 0x0F0F0F0Fu; hi.y = (w.y >> 4) & 0x0F0F0F0Fu;
    lo.z = w.z & 0x0F0F0F0Fu; hi.z = (w.z >> 4) & 0x0F0F0F0Fu;
    lo.w = w.w & 0x0F0F0F0Fu; hi.w = (w.w >> 4) & 0x0F0F0F0Fu;
    uint8_t* row = tile + r * 128;
    const int sw = r & 7;
    *reinterpret_cast<uint4*>(row + (((2 * j) ^ sw) << 4)) = lo;
    *reinterpret_cast<uint4*>(row + (((2 * j + 1) ^ sw) << 4)) = hi;
}

__global__ void __launch_bounds__(THREADS, 1)
qgemm_tc_w4a4_kernel(const uint8_t* __restrict__ a, const uint8_t* __restrict__ w, int64_t M, int N, int K,
                     EpilogueArgs ep, int* status) {
    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* opA = smem;
    uint8_t* opW = opA + S * OPA;
    int4* colterm = reinterpret_cast<int4*>(opW + S * OPW);
    uint64_t* bars = reinterpret_cast<uint64_t*>(colterm + BN);
    uint64_t* full_op = bars;              // [S] 4 arrivals: the warps of the stage's load group
    uint64_t* empty = bars + S;            // [S] MMAs that read the stage have completed
    uint64_t* acc_full = bars + 2 * S;     // [2]
    uint64_t* acc_empty = acc_full + 2;    // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = int((M + BM - 1) / BM);
    const int tiles_n = (N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int KB = (K + BK - 1) / BK;
    const int row_bytes = K / 2;
    const Abort ab{abort_flag, status};

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(&full_op[s], kGroupWarps);
            ptx::mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&acc_full[b], 1);
            ptx::mbar_init(&acc_empty[b], 4);
        }
        *abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
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
                    if (!wait_bounded(&full_op[s], (it / S) & 1, ab)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = ptx::smem_addr(opA + s * OPA);
                    const uint32_t b_addr = ptx::smem_addr(opW + s * OPW);
#pragma unroll
                    for (int kk = 0; kk < BK / 32; ++kk)
                        ptx::mma_i8_ss(d_tmem, ptx::smem_desc_sw128(a_addr + kk * 32),
                                       ptx::smem_desc_sw128(b_addr + kk * 32), idesc, (kb | kk) != 0);
                    ptx::mma_commit(&empty[s]);
                }
                if (ok) ptx::mma_commit(&acc_full[abuf]);
            }
        }
    } else if (warp < kLoad0) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;
        const int et = threadIdx.x - 32 * kEpi0;
        uint32_t lt = 0;
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
                if (nb >= N) break;
                uint32_t r[32];
                ptx::tmem_ld_32x32b_x32(tmem_base + (uint32_t(quad * 32) << 16) + abuf * BN + ch * 32, r);
                ptx::tmem_ld_wait();
                if (m < M) store_chunk(ep, r, colterm + ch * 32, rt, m, N, nb);
                __syncwarp();
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&acc_empty[abuf]);
        }
    } else {
        // ------------------------------------------------------------------ load + unpack
        const int group = (warp - kLoad0) / kGroupWarps;                 // = pipeline stage it serves
        const int t = threadIdx.x - 32 * (kLoad0 + group * kGroupWarps);  // 0..127 within the group
        const int rA = t >> 2, j = t & 3;                 // chunk (row, 16-byte column) within a pass of rows
        auto issue = [&](uint4 (&buf)[CH], const Cursor& c) {
            if (c.tile >= num_tiles) return;
            const int m0 = (c.tile % tiles_m) * BM, n0 = (c.tile / tiles_m) * BN;
            const int col = c.kb * (BK / 2) + j * 16;
            const bool col_ok = col < row_bytes;
#pragma unroll
            for (int i = 0; i < CHUNKS_A; ++i) {
                const int64_t row = int64_t(m0) + rA + ROWS_PER_PASS * i;
                buf[i] = (col_ok && row < M) ? __ldcg(reinterpret_cast<const uint4*>(a + row * row_bytes + col))
                                             : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int i = 0; i < CHUNKS_W; ++i) {
                const int row = n0 + rA + ROWS_PER_PASS * i;
                buf[CHUNKS_A + i] = (col_ok && row < N)
                                        ? __ldcg(reinterpret_cast<const uint4*>(w + int64_t(row) * row_bytes + col))
                                        : make_uint4(0, 0, 0, 0);
            }
        };
        auto advance = [&](Cursor& c) {                   // this group's next K-block: kGroups further on
            c.kb += kGroups;
            while (c.kb >= KB && c.tile < num_tiles) { c.kb -= KB; c.tile += gridDim.x; }
        };
        int my_tiles = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) ++my_tiles;
        const uint32_t total = uint32_t(my_tiles) * uint32_t(KB);
        Cursor lc{int(blockIdx.x), group - kGroups};
        advance(lc);                                      // -> K-block `group` of the first tile (or beyond)
        uint4 buf[CH];
        issue(buf, lc);
        const int s = group;
        uint32_t round = 0;
        for (uint32_t it = uint32_t(group); it < total; it += kGroups, ++round) {
            if (!wait_bounded(&empty[s], (round & 1) ^ 1, ab)) break;
#pragma unroll
            for (int i = 0; i < CHUNKS_A; ++i) expand_store(buf[i], opA + s * OPA, rA + ROWS_PER_PASS * i, j);
#pragma unroll
            for (int i = 0; i < CHUNKS_W; ++i) expand_store(buf[CHUNKS_A + i], opW + s * OPW, rA + ROWS_PER_PASS * i, j);
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&full_op[s]);
            advance(lc);
            issue(buf, lc);
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

int launch_qgemm_tc_w4a4(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, const EpilogueArgs& ep,
                         cudaStream_t st) {
    int* status = device_status_word();
    if (!status) return QLLM_ERR_CUDA;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(qgemm_tc_w4a4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM));
    const int64_t tiles = ((M + BM - 1) / BM) * int64_t((N + BN - 1) / BN);
    const int grid = int(std::min<int64_t>(tiles, sm_count()));
    qgemm_tc_w4a4_kernel<<<grid, THREADS, SMEM, st>>>(a, w, M, N, K, ep, status);
    return after_launch();
}

}  // namespace qllm
