// Self-test of the bounded device-side wait: one thread waits on an mbarrier that nothing will ever
// arrive at, with a limit of about a millisecond.  The wait gives up, the give-up is recorded in the
// device status word exactly as the head kernels record theirs, and the kernel returns normally: the
// context stays usable and rstitch_last_status reports RSTITCH_ERR_TIMEOUT.  Nothing traps or spins on.
#include "rstitch_kernels.cuh"

namespace rstitch {
namespace {

__global__ void __launch_bounds__(32)
wait_selftest_kernel(DevStat *stat, long long limit_cycles)
{
    __shared__ __align__(8) uint64_t s_bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        ptx::mbar_init(ptx::smem_u32(&s_bar), 1);
        ptx::mbar_fence_init();
        if (!ptx::mbar_wait(ptx::smem_u32(&s_bar), 0u, &s_abort, limit_cycles)) {
            s_abort = 1;
            atomicAdd(&stat->timeouts, 1u);
            atomicExch(&stat->timeout_site, kSelftestSite);
        }
        ptx::mbar_inval(ptx::smem_u32(&s_bar));
    }
}

}  // namespace

cudaError_t launch_wait_selftest(DevStat *stat, long long limit_cycles, cudaStream_t stream)
{
    wait_selftest_kernel<<<1, 32, 0, stream>>>(stat, limit_cycles);
    return cudaGetLastError();
}

}  // namespace rstitch
