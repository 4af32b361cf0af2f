// Self-test of the bounded wait every staged kernel of the library relies on: a wait that cannot be
// satisfied must run out, set the device status word and let the kernel RETURN, so that the context stays
// usable.  The kernel here waits, with the library's own wait routine, on an mbarrier nobody arrives at.
#include "iv_internal.h"
#include "tma_dev.cuh"

namespace ivk {
namespace {

__global__ void __launch_bounds__(32)
wait_timeout_selftest_kernel(long long limit_cycles, uint32_t *__restrict__ status, unsigned long long *__restrict__ waited) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = tma::smem_u32(&bar);
    if (threadIdx.x == 0) {
        tma::mbar_init(b, 1);
        tma::fence_barrier_init();
    }
    __syncwarp();
    const long long t0 = clock64();
    const bool ok = __all_sync(0xffffffffu, tma::mbar_wait_bounded(b, 0, limit_cycles));   // phase 0 never completes
    const long long t1 = clock64();
    if (threadIdx.x == 0) {
        if (!ok) atomicExch(status, (uint32_t)IVK_DEV_TIMEOUT);
        if (waited) *waited = (unsigned long long)(t1 - t0);
    }
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(uint64_t limit_cycles, uint32_t *d_status, unsigned long long *d_waited,
                                         cudaStream_t stream, uint64_t *launches) {
    if (launches) ++*launches;
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>((long long)limit_cycles, d_status, d_waited);
    return cudaGetLastError();
}

}  // namespace ivk
