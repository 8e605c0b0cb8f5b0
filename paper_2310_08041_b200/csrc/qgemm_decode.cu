#include "common.h"
namespace qllm {
bool qgemm_decode_supported(int64_t, int, int, int, int) { return false; }
int launch_qgemm_decode(const uint8_t*, const uint8_t*, int64_t, int, int, int, int, const EpilogueArgs&, cudaStream_t) { return QLLM_ERR_UNSUPPORTED; }
}
