// Self-test of the bounded device-side waits: the path from a wait that gives up to the status word the host polls.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace cprune {

// One warp waits on a barrier that is initialised for one arrival and that nothing ever signals: no copy is in
// flight, nothing else touches the barrier.  mbar_wait gives up after `limit` cycles and raises STATUS_TIMEOUT.
__global__ void __launch_bounds__(32) wait_timeout_kernel(int *status, long long limit) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) (void)mbar_wait(b, 0u, &abort_flag, status, true, limit);
    __syncwarp();
}

}  // namespace cprune

extern "C" cprune_status cprune_selftest_wait_timeout(void *stream) {
    using namespace cprune;
    int *status = device_status_word();
    if (!status) return cuda_fail(cudaGetLastError(), "status word");
    wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(status, 1LL << 16);
    CPRUNE_LAUNCH_CHECK("wait_timeout_kernel");
    return CPRUNE_OK;
}
