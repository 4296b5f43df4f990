// Self-test of the kernels' bounded-wait error path.  The attention kernels
// never spin without a limit: every mbarrier wait goes through wait_or_abort
// and, when the limit runs out, records AP_ERR_TIMEOUT in the pool's status
// word and returns.  In normal operation that branch is never taken, so this
// file provides a kernel in which it always is: one warp waits, with the same
// routine and a caller-chosen limit, on an mbarrier on which nothing ever
// arrives.  The kernel ends by itself after the limit; the context stays
// usable.
#include "internal.h"
#include "ptx.cuh"

namespace ap {

namespace {

__global__ void __launch_bounds__(32) selftest_wait_kernel(int *status, int *merge_counters, uint64_t limit_ns, int leave_counter) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    __syncwarp();
    // like a decode CTA whose stream's partial was counted in before the CTA gave up: the arrival
    // counter of merge entry 0 is left at 1, which ap_last_device_status has to clear
    if (leave_counter && threadIdx.x == 0) atomicAdd(merge_counters, 1);
    if (!ptx::wait_or_abort(&bar, 0, &abort_flag, limit_ns)) {
        if (threadIdx.x == 0) {
            ptx::record_status(status, AP_ERR_TIMEOUT);
            abort_flag = 1;
        }
    }
}

}  // namespace

cudaError_t launch_selftest_wait(const ap_kv_pool *pool, uint64_t limit_ns, int leave_counter, cudaStream_t stream) {
    selftest_wait_kernel<<<1, 32, 0, stream>>>(pool->status_dev, pool->d_counters, limit_ns, leave_counter);
    return cudaGetLastError();
}

}  // namespace ap
