// Self-test of the bounded device-side wait every pipelined kernel of the library relies on.
#include "tcgen05.cuh"

namespace {

// One CTA waits on a barrier phase that nothing ever completes.  Every thread runs the library's bounded wait
// with a short limit; the first to run out records PPO_ERR_TIMEOUT and raises the CTA's abort flag, the others
// leave through that flag, and the kernel returns normally.
__global__ void __launch_bounds__(64) wait_timeout_kernel(long long limit_cycles, int32_t *status, int *gave_up) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = tc::mbar_wait_limit(&bar, 0, &abort_flag, status, limit_cycles);
    if (!ok) atomicAdd(gave_up, 1);
}

}  // namespace

extern "C" int ppo_selftest_wait_timeout(long long limit_cycles, int *dev_gave_up, void *stream) {
    if (!dev_gave_up || limit_cycles <= 0 || limit_cycles > 2000000000ll) return PPO_ERR_INVALID_ARG;
    int32_t *status = ppo_device_status_ptr();
    if (!status) return PPO_ERR_CUDA;
    wait_timeout_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(limit_cycles, status, dev_gave_up);
    PPO_LAUNCH_CHECK();
    return PPO_OK;
}
