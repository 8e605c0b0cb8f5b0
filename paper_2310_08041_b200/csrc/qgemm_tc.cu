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

namespace qllm {

namespace {

constexpr int BM = 128;              // tile rows (tokens) = MMA M
constexpr int BK = 128;              // codes of K per pipeline stage = one 128-byte swizzle row
constexpr int kUnpackWarps = 8;
constexpr int kFirstEpiWarp = 2, kFirstUnpackWarp = 6;
constexpr long long kWaitCycles = 1ll << 32;   // ~2 s at 2 GHz

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

struct Abort {
    volatile int* flag;     // shared: some role gave up
    int* status;            // global status word of the library
};

__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity, const Abort& ab) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 1;; ++i) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 0) {
            if (*ab.flag) return false;
            if (clock64() - t0 > kWaitCycles) {
                *ab.flag = 1;
                atomicExch(ab.status, QLLM_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// Expand a ROWS x 64-byte tile of packed nibbles into a ROWS x 128-byte swizzled byte tile.
// 16-byte chunk j of row r (codes 32j .. 32j+31) fills units 2j and 2j+1 of the row, each unit
// stored at position unit ^ (r & 7).  PAIRED (both operands 4-bit): even nibbles to unit 2j,
// odd nibbles to unit 2j+1 -- a permutation of K shared by both operands.  Otherwise (the other
// operand holds byte codes in natural order) the nibbles are interleaved back into K order.
template <int ROWS, bool PAIRED>
__device__ __forceinline__ void unpack_tile(const uint8_t* __restrict__ raw, uint8_t* __restrict__ op, int t) {
    constexpr int PER_THREAD = ROWS * 4 / (32 * kUnpackWarps);
    static_assert(PER_THREAD * 32 * kUnpackWarps == ROWS * 4, "tile rows must split evenly over the unpack threads");
#pragma unroll
    for (int i = 0; i < PER_THREAD; ++i) {
        const int q = t + i * 32 * kUnpackWarps;
        const int r = q >> 2, j = q & 3;
        const uint4 w = *reinterpret_cast<const uint4*>(raw + q * 16);
        uint4 lo, hi;
        lo.x = w.x & 0x0F0F0F0Fu; hi.x = (w.x >> 4) & 0x0F0F0F0Fu;
        lo.y = w.y & 0x0F0F0F0Fu; hi.y = (w.y >> 4) & 0x0F0F0F0Fu;
        lo.z = w.z & 0x0F0F0F0Fu; hi.z = (w.z >> 4) & 0x0F0F0F0Fu;
        lo.w = w.w & 0x0F0F0F0Fu; hi.w = (w.w >> 4) & 0x0F0F0F0Fu;
        uint4 u0 = lo, u1 = hi;
        if (!PAIRED) {
            u0.x = __byte_perm(lo.x, hi.x, 0x5140); u0.y = __byte_perm(lo.x, hi.x, 0x7362);
            u0.z = __byte_perm(lo.y, hi.y, 0x5140); u0.w = __byte_perm(lo.y, hi.y, 0x7362);
            u1.x = __byte_perm(lo.z, hi.z, 0x5140); u1.y = __byte_perm(lo.z, hi.z, 0x7362);
            u1.z = __byte_perm(lo.w, hi.w, 0x5140); u1.w = __byte_perm(lo.w, hi.w, 0x7362);
        }
        uint8_t* row = op + r * 128;
        const int sw = r & 7;
        *reinterpret_cast<uint4*>(row + (((2 * j) ^ sw) << 4)) = u0;
        *reinterpret_cast<uint4*>(row + (((2 * j + 1) ^ sw) << 4)) = u1;
    }
}

template <int BN, bool AP, bool WP>
__global__ void __launch_bounds__(Tile<BN, AP, WP>::THREADS, 1)
qgemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                int64_t M, int N, int K, EpilogueArgs ep, int* status) {
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

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
                for (int kb = 0; kb < KB; ++kb, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1;
                    if (!wait_bounded(&empty[s], ph ^ 1, ab)) { ok = false; break; }
                    if (AP || WP) ptx::mbar_arrive_expect_tx(&full_raw[s], T::RAWA + T::RAWW);
                    if (!AP || !WP) ptx::mbar_arrive_expect_tx(&full_op[s], (AP ? 0 : T::OPA) + (WP ? 0 : T::OPW));
                    if (AP) ptx::tma_load_2d(rawA + s * T::RAWA, &tmA, kb * (BK / 2), m0, &full_raw[s]);
                    else    ptx::tma_load_2d(opA + s * T::OPA, &tmA, kb * BK, m0, &full_op[s]);
                    if (WP) ptx::tma_load_2d(rawW + s * T::RAWW, &tmW, kb * (BK / 2), n0, &full_raw[s]);
                    else    ptx::tma_load_2d(opW + s * T::OPW, &tmW, kb * BK, n0, &full_op[s]);
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
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++lt) {
            const uint32_t abuf = lt & 1, aph = (lt >> 1) & 1;
            const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
            ptx::named_bar_sync(1, 128);
            if (!ep.raw_acc) {
                for (int c = et; c < BN; c += 128) {
                    const int n = n0 + c;
                    int4 v = make_int4(0, 0, 0, 0);
                    if (n < N) {
                        const ColTerm ct = make_col_term(ep.w_scale, ep.w_zero, ep.w_colsum, ep.bias, K, n);
                        v = make_int4(__float_as_int(ct.scale), ct.zero, ct.corr, __float_as_int(ct.bias));
                    }
                    colterm[c] = v;
                }
            }
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
                if (m < M) {
                if (ep.raw_acc) {
                    int32_t* o = static_cast<int32_t*>(ep.out) + m * N + nb;
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        if (nb + 4 * v < N)
                            *reinterpret_cast<int4*>(o + 4 * v) = make_int4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                } else {
                    float f[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const int4 ct = colterm[ch * 32 + c];
                        const int I = int(r[c]) - ct.y * rt.rowsum - rt.zero * ct.z;
                        f[c] = fmaf(rt.scale * __int_as_float(ct.x), float(I), __int_as_float(ct.w));
                    }
                    if (ep.out_dtype == QLLM_F32) {
                        float* o = static_cast<float*>(ep.out) + m * N + nb;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (nb + 4 * v < N)
                                *reinterpret_cast<float4*>(o + 4 * v) = make_float4(f[4 * v], f[4 * v + 1], f[4 * v + 2], f[4 * v + 3]);
                    } else {
                        __nv_bfloat16* o = static_cast<__nv_bfloat16*>(ep.out) + m * N + nb;
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            if (nb + 8 * v < N) {
                                uint4 pk;
                                __nv_bfloat162 h0 = __floats2bfloat162_rn(f[8 * v], f[8 * v + 1]);
                                __nv_bfloat162 h1 = __floats2bfloat162_rn(f[8 * v + 2], f[8 * v + 3]);
                                __nv_bfloat162 h2 = __floats2bfloat162_rn(f[8 * v + 4], f[8 * v + 5]);
                                __nv_bfloat162 h3 = __floats2bfloat162_rn(f[8 * v + 6], f[8 * v + 7]);
                                pk.x = *reinterpret_cast<uint32_t*>(&h0); pk.y = *reinterpret_cast<uint32_t*>(&h1);
                                pk.z = *reinterpret_cast<uint32_t*>(&h2); pk.w = *reinterpret_cast<uint32_t*>(&h3);
                                *reinterpret_cast<uint4*>(o + 8 * v) = pk;
                            }
                    }
                }
                }
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

// ---- host side ----------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// uint8 matrix [rows][row_bytes]; box = box_rows x box_bytes; out-of-range parts read as zero.
bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t row_bytes, uint32_t box_rows,
              uint32_t box_bytes, bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {box_bytes, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
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

template <int BN, bool AP, bool WP>
int launch(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, const EpilogueArgs& ep, cudaStream_t st) {
    using T = Tile<BN, AP, WP>;
    static_assert(T::STAGES >= 2, "pipeline needs at least two stages");
    CUtensorMap tmA, tmW;
    const bool okA = AP ? make_map(&tmA, a, uint64_t(M), uint64_t(K / 2), BM, BK / 2, false)
                        : make_map(&tmA, a, uint64_t(M), uint64_t(K), BM, BK, true);
    const bool okW = WP ? make_map(&tmW, w, uint64_t(N), uint64_t(K / 2), BN, BK / 2, false)
                        : make_map(&tmW, w, uint64_t(N), uint64_t(K), BN, BK, true);
    if (!okA || !okW) return QLLM_ERR_CUDA;
    int* status = device_status_word();
    if (!status) return QLLM_ERR_CUDA;
    auto kern = qgemm_tc_kernel<BN, AP, WP>;
    QLLM_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, T::SMEM));
    const int64_t tiles = ((M + BM - 1) / BM) * int64_t((N + BN - 1) / BN);
    const int grid = int(std::min<int64_t>(tiles, sm_count()));
    kern<<<grid, T::THREADS, T::SMEM, st>>>(tmA, tmW, M, N, K, ep, status);
    return after_launch();
}

}  // namespace

bool qgemm_tc_supported(int64_t M, int N, int K, int a_bits, int w_bits) {
    (void)a_bits; (void)w_bits;
    return M >= 1 && M < (int64_t(1) << 31) - BM && K % 32 == 0 && N % 8 == 0 && encode_fn() != nullptr;
}

int launch_qgemm_tc(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, int a_bits, int w_bits,
                    const EpilogueArgs& ep, cudaStream_t st) {
    const bool ap = a_bits == 4, wp = w_bits == 4;
    if (ap && wp) return launch<256, true, true>(a, w, M, N, K, ep, st);
    if (!ap && !wp) return launch<256, false, false>(a, w, M, N, K, ep, st);
    if (ap) return launch<256, true, false>(a, w, M, N, K, ep, st);
    return launch<256, false, true>(a, w, M, N, K, ep, st);
}

}  // namespace qllm
