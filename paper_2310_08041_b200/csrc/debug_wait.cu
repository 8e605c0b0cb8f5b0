// qllm_debug_wait_expiry: runs the bounded wait of the tensor-core GEMM kernels into its limit, the safe way.
//
// One CTA of one warp initialises an mbarrier that nobody will ever arrive on and waits for it with the same
// wait_bounded the GEMM roles use, under a short limit (2^20 cycles, about half a millisecond).  The wait
// gives up, raises the library's status word exactly as a GEMM role would, and the kernel returns: no copy, no
// tensor memory, nothing in flight, no trap and no unbounded spin.  What the host sees afterwards (the launch
// returns, qllm_poll_status reports the timeout once, the next call works) is what it would see after a real
// expiry.

#include "qgemm_tc_common.cuh"

namespace qllm {
namespace {

__global__ void __launch_bounds__(32) wait_expiry_kernel(int* status, int* gave_up) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int flag;
    if (threadIdx.x == 0) {
        flag = 0;
        ptx::mbar_init(&bar, 1);
        ptx::fence_barrier_init();
    }
    __syncthreads();
    const tc::Abort ab{&flag, status};
    const bool arrived = tc::wait_bounded(&bar, 0, ab, 1ll << 20);
    if (threadIdx.x == 0) *gave_up = arrived ? 0 : 1;
}

}  // namespace
}  // namespace qllm

extern "C" int qllm_debug_wait_expiry(int* gave_up, void* stream) {
    using namespace qllm;
    if (!gave_up) return QLLM_ERR_NULL;
    int* status = device_status_word();
    if (!status) return QLLM_ERR_CUDA;
    wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, gave_up);
    return after_launch();
}
