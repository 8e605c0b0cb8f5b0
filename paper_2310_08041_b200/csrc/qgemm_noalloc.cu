// qllm_qgemm_noalloc: the integer GEMM for callers that must not allocate.
//
// qllm_qgemm needs the code sum of every activation row.  When the caller does not supply
// it, the ordinary entry point computes it into a buffer that the library grows with
// cudaMalloc.  Some callers cannot tolerate that: code running inside a memory pool or a
// real-time serving loop where an allocation may synchronise the device or fail, and code
// that has handed all device memory to another allocator.  For them the row sums go to a
// fixed array that is part of the library image instead.

#include <mutex>

#include "common.h"

namespace qllm {
namespace {

// Row-sum scratch shared by every call on a device.  Each GPU that loads the library holds
// these 256 KiB until the process exits.
static __device__ __align__(256) int32_t g_rowsum_scratch[QLLM_NOALLOC_MAX_M];

std::mutex g_mu;
int32_t* g_scratch_addr[64] = {nullptr};

// The array's name is only a host-side handle; kernels need its device address, which is
// looked up once per device (with that device current) and cached.
int scratch_address(int32_t** out) {
    int dev = 0;
    QLLM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return QLLM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_scratch_addr[dev]) {
        int32_t* p = nullptr;
        QLLM_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_rowsum_scratch));
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return QLLM_OK;
}

}  // namespace
}  // namespace qllm

extern "C" int qllm_qgemm_noalloc(const uint8_t* codes, const float* a_scale, const float* a_zero,
                                  const uint8_t* w_codes, const float* w_scale, const float* w_zero,
                                  const int32_t* w_colsum, const float* bias, void* out, int64_t M, int N,
                                  int K, int a_bits, int w_bits, int out_dtype, void* stream) {
    using namespace qllm;
    if (bits_ok(a_bits) && bits_ok(w_bits) && M > QLLM_NOALLOC_MAX_M && N > 0 && K > 0)
        return QLLM_ERR_UNSUPPORTED;                            // more rows than the fixed scratch holds
    // all of qllm_qgemm's argument checks first: a call that returns an error has launched nothing and has not
    // touched the array every call shares
    int rc = gemm_check_args(codes, a_scale, a_zero, w_codes, w_scale, w_zero, w_colsum, out, M, N, K, a_bits, w_bits,
                             out_dtype);
    if (rc != QLLM_OK) return rc;
    if (M == 0) return QLLM_OK;
    int32_t* rowsum = nullptr;
    rc = scratch_address(&rowsum);
    if (rc != QLLM_OK) return rc;
    // every one of the M entries is overwritten, so nothing left by an earlier call is read
    rc = launch_rowsum(codes, M, K, a_bits, rowsum, static_cast<cudaStream_t>(stream));
    if (rc != QLLM_OK) return rc;
    // the same GEMM as qllm_qgemm, held to the paths that never grow library scratch
    return gemm_entry(codes, a_scale, a_zero, w_codes, w_scale, w_zero, w_colsum, bias, out, M, N, K, a_bits,
                      w_bits, out_dtype, rowsum, static_cast<cudaStream_t>(stream), false);
}
