// Shared host-side plumbing of the library: error bookkeeping, launch counter,
// argument-check helpers.  No kernel code lives here.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <utility>

#include "../../include/qllm.h"

namespace qllm {

extern thread_local int g_last_cuda_error;
extern std::atomic<int64_t> g_launch_count;

inline int cuda_fail(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return QLLM_ERR_CUDA;
}

// Records a launch and turns a launch-time error into a status.
inline int after_launch(int n_launches = 1) {
    g_launch_count.fetch_add(n_launches, std::memory_order_relaxed);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
    return QLLM_OK;
}

#define QLLM_CUDA_TRY(expr)                                   \
    do {                                                      \
        cudaError_t _e = (expr);                              \
        if (_e != cudaSuccess) return ::qllm::cuda_fail(_e);  \
    } while (0)

// Launches kern as a programmatic dependent of the kernel launched just before it on the stream: its CTAs may
// start once that kernel's CTAs have executed griddepcontrol.launch_dependents (or ended), and whatever it does
// before its own griddepcontrol.wait overlaps that kernel's tail and the launch latency.  Before the wait it may
// only touch what no earlier kernel on the stream writes or reads-then-expects-unchanged (prefetches qualify).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool bits_ok(int b) { return b == 4 || b == 6 || b == 8; }
inline bool dtype_ok(int d) { return d == QLLM_F32 || d == QLLM_BF16; }
// Bytes of one row of K codes at the given bit-width (4-bit codes are packed two per byte).
inline int64_t code_row_bytes(int K, int bits) { return bits == 4 ? K / 2 : K; }

// Number of SMs of the current device (cached per device; 148 if the query fails).
int device_sm_count();

// Device-side status word (one per loaded library image and device).
int* device_status_word();          // device address, or nullptr on failure (error recorded)

// ---- kernels' host launchers (each returns a status) ----------------------
struct EpilogueArgs {
    const float* a_scale;
    const float* a_zero;
    const int32_t* a_rowsum;
    const float* w_scale;
    const float* w_zero;
    const int32_t* w_colsum;
    const float* bias;      // may be null
    void* out;              // [M][N] f32 / bf16, or int32 when raw_acc
    int out_dtype;          // QLLM_F32 / QLLM_BF16
    int raw_acc;            // 1: store int32 accumulators, ignore everything else
};

// Per-(device, stream) library scratch, grown on demand and never shrunk.
// The map-image scratch starts with a header of kMapScratchHeader bytes whose first 8 hold the content key of the
// token-kernel image behind it (0 = none; a fresh allocation is zeroed on the stream).
enum ScratchKind { kScratchExpand = 0, kScratchMapImage = 1, kScratchKinds = 2 };
constexpr size_t kMapScratchHeader = 256;
int stream_scratch(int kind, cudaStream_t st, size_t bytes, uint8_t** out);

// The specialised fused kernels consume a compiled image of the reassembly map (0 bytes: the channel
// count has no specialised kernel; x_dtype selects the kernel: bf16 rows of 4096, 5120 or 8192 channels have
// one of their own).  map_image = nullptr compiles one per call into stream scratch.
struct MapCounts;
size_t reassemble_map_image_bytes(int C, int x_dtype);
// true when the fused kernel for C channels can write 4-bit codes one per byte (byte_lanes below)
bool reassemble_byte_lanes_supported(int C);
int compile_reassemble_map(int C, int x_dtype, const float* gamma, const float* beta, const int32_t* ptr,
                           const int32_t* src, const float* coef, void* image, cudaStream_t st);
// counts: what reassemble_map_counts returned for this image (sizes the kernel's shared memory exactly instead
// of for the largest image), or nullptr.  share_sm: another kernel of the caller runs beside this one; leave part
// of each SM's registers to it.
int launch_reassemble_quant(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                            const float* beta, float eps, const int32_t* ptr, const int32_t* src,
                            const float* coef, int bits, const void* map_image, uint8_t* codes, float* a_scale,
                            float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool byte_lanes = false,
                            const MapCounts* counts = nullptr, bool share_sm = false);
// Counts of the multi-entry rows of a compiled image (waits for the stream).
int reassemble_map_counts(int C, int x_dtype, const void* image, cudaStream_t st, MapCounts* out);
// The kernel for bf16 rows of LLaMA hidden sizes (reassemble_quant_token.cu)
bool token_kernel_serves(int C);
size_t token_image_bytes(int C);
// key (device, may be null): content key kept beside an image in library scratch; when the inputs hash to the
// value found there the image is left as it is
int compile_token_map(int C, const float* gamma, const float* beta, const int32_t* ptr, const int32_t* src,
                      const float* coef, void* image, cudaStream_t st, uint64_t* key = nullptr);
int token_map_counts(int C, const void* image, cudaStream_t st, MapCounts* out);
// device word of a compiled token image: non-zero when the token kernel serves the map
const int* token_image_served_flag(int C, const void* image);
int launch_reassemble_quant_token(const void* x, int64_t M, int C, const float* gamma, const float* beta, float eps,
                                  const int32_t* ptr, const int32_t* src, const float* coef, int bits,
                                  const void* image, const MapCounts& mc, uint8_t* codes, float* a_scale,
                                  float* a_zero, int32_t* a_rowsum, cudaStream_t st, bool byte_lanes, bool share_sm);
int launch_reassemble_quant_generic(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                                    const float* beta, float eps, const int32_t* ptr, const int32_t* src,
                                    const float* coef, int bits, uint8_t* codes, float* a_scale,
                                    float* a_zero, int32_t* a_rowsum, cudaStream_t st,
                                    const int* skip_if_nonzero = nullptr);
// y[t][c] = LayerNorm(x[t])[c] in fp32 (build-time helper)
int launch_layernorm_rows(const void* x, int x_dtype, int64_t T, int C, const float* gamma, const float* beta,
                          float eps, float* y, cudaStream_t st);
// Eq. 5 nearest-B search on the device for the host builder (see channel_distance.cu)
int eq5_nearest_device(const float* y, int64_t T, const float* w, int N, int C, const int* a_idx, int nA,
                       const int* b_idx, int nB, int* best, float* best_d, cudaStream_t st);
int launch_calib_absmax(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                        const float* beta, float eps, float* absmax, cudaStream_t st);
int launch_expand_codes(const uint8_t* packed, int64_t rows, int K, uint8_t* bytes, cudaStream_t st);
// The GEMM behind qllm_qgemm.  may_allocate = false keeps it on paths that never grow library scratch.
int gemm_entry(const uint8_t* codes, const float* a_scale, const float* a_zero, const uint8_t* w_codes,
               const float* w_scale, const float* w_zero, const int32_t* w_colsum, const float* bias, void* out,
               int64_t M, int N, int K, int a_bits, int w_bits, int out_dtype, const int32_t* a_rowsum,
               cudaStream_t st, bool may_allocate, const uint8_t* w_ready = nullptr, bool weights_static = false);
int gemm_check_args(const uint8_t* codes, const float* a_scale, const float* a_zero, const uint8_t* w_codes,
                    const float* w_scale, const float* w_zero, const int32_t* w_colsum, const void* out, int64_t M,
                    int N, int K, int a_bits, int w_bits, int out_dtype);
int launch_rowsum(const uint8_t* codes, int64_t M, int K, int bits, int32_t* rowsum, cudaStream_t st);
int launch_qgemm_plain(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, int a_bits,
                       int w_bits, const EpilogueArgs& ep, cudaStream_t st);
int launch_qgemm_decode(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, int a_bits,
                        int w_bits, const EpilogueArgs& ep, cudaStream_t st);
bool qgemm_tc_supported(int64_t M, int N, int K, int a_bits, int w_bits);
// CTA-pair (cta_group::2) variant for byte-lane codes on both operands and M > 128
bool qgemm_tc2_supported(int64_t M, int N, int K, int a_bits, int w_bits);
int launch_qgemm_tc2(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, const EpilogueArgs& ep,
                     cudaStream_t st);
// weights_static: the caller vouches that no kernel before this one on the stream writes the weights (they may then
// be requested before that kernel is complete)
int launch_qgemm_tc(const uint8_t* a, const uint8_t* w, int64_t M, int N, int K, int a_bits,
                    int w_bits, const EpilogueArgs& ep, cudaStream_t st, bool weights_static = false);
bool qgemm_decode_supported(int64_t M, int N, int K, int a_bits, int w_bits);

}  // namespace qllm
