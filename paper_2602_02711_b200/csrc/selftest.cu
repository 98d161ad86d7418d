// Self-test of the failure path every kernel of this library shares: a wait on an mbarrier is bounded, and a
// wait that runs out records DMR_ERR_TIMEOUT in the workspace's status word and lets the kernel return, so
// that a wrong byte count or a copy that never lands cannot hang a GPU.  The kernel below waits on a barrier
// that nothing ever arrives at, with the limit lowered to a thousand polls (well under a millisecond).
#include "sm100.cuh"

namespace dmr {

namespace {

__global__ void __launch_bounds__(32) wait_timeout_kernel(int32_t *status, int32_t *returned) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        fence_barrier_init();
    }
    __syncwarp();
    const bool ok = mbar_wait_limited(b, 0u, status, 1000u);  // nobody arrives: this gives up
    if (threadIdx.x == 0) *returned = ok ? 1 : 2;            // 2 = the wait gave up and the kernel went on to its end
}

}  // namespace

dmr_status_t launch_wait_timeout_selftest(int32_t *status, int32_t *returned, cudaStream_t st) {
    wait_timeout_kernel<<<1, 32, 0, st>>>(status, returned);
    return check_launch();
}

}  // namespace dmr
