// Self-test of the error path of the bounded waits: a warp waits on a barrier that nothing arms and
// nothing will ever complete, with the limit the caller gives.  The wait runs out, the warp raises
// the call's time-out flag and returns; no copy is in flight at any point, so nothing can land
// late in shared memory.
#include "excp_common.cuh"
#include "tma.cuh"

namespace excp {

__global__ void __launch_bounds__(32) wait_selftest_kernel(CallState* call, u64 limit_ns) {
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncwarp();
    if (!mbar_wait_warp(&bar, 0, limit_ns) && threadIdx.x == 0) atomicOr(&call->flags, FLAG_TIMEOUT);
}

void launch_wait_selftest(const LaunchCfg& cfg, CallState* call, u64 limit_ns) {
    wait_selftest_kernel<<<1, 32, 0, cfg.stream>>>(call, limit_ns);
}

}  // namespace excp
