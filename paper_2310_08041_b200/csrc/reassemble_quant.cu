// Dispatch of the fused pre-GEMM stage.
#include "common.h"

namespace qllm {

int launch_reassemble_quant(const void* x, int x_dtype, int64_t M, int C, const float* gamma,
                            const float* beta, float eps, const int32_t* ptr, const int32_t* src,
                            const float* coef, int bits, uint8_t* codes, float* a_scale,
                            float* a_zero, int32_t* a_rowsum, cudaStream_t st) {
    return launch_reassemble_quant_generic(x, x_dtype, M, C, gamma, beta, eps, ptr, src, coef, bits,
                                           codes, a_scale, a_zero, a_rowsum, st);
}

}  // namespace qllm
