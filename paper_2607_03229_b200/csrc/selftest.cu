// mpipe_selftest_wait_timeout: exercises the bounded-wait path of the attention kernels on purpose.
// One CTA waits, with the same routine the kernels use, on an mbarrier that nothing ever arrives on;
// when the cycle budget runs out the wait gives up, the kernel records MPIPE_ERR_TIMEOUT in the caller's
// status buffer and returns normally -- no trap, no fault, the context stays usable.
#include "common.h"
#include "sm100_ptx.cuh"

namespace mpipe {

__global__ void __launch_bounds__(128)
wait_timeout_kernel(long long budget_cycles, int32_t* status_buf) {
    __shared__ uint64_t never_signalled;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&never_signalled, 1);
        fence_mbar_init();
    }
    __syncthreads();
    // every warp waits, like the roles of a real kernel; the first one to run out raises the abort flag and
    // the others leave through it
    const bool ok = mbar_wait_budget(&never_signalled, 0, &abort_flag, budget_cycles);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_flag)) report_status(status_buf, MPIPE_ERR_TIMEOUT, int32_t(blockIdx.x));
}

}  // namespace mpipe

extern "C" int32_t mpipe_selftest_wait_timeout(int64_t budget_cycles, int32_t* status_buf, void* stream) {
    if (budget_cycles <= 0 || budget_cycles > 4000000000ll || status_buf == nullptr) return MPIPE_ERR_INVALID_ARG;
    mpipe::wait_timeout_kernel<<<1, 128, 0, static_cast<cudaStream_t>(stream)>>>(budget_cycles, status_buf);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}
