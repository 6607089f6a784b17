// Self-test of the bounded device-side waits: the path a hung producer or a lost
// barrier arrival would take, exercised without hanging or faulting anything.
#include "lvspec_internal.h"
#include "sm100_ptx.cuh"

namespace lvspec {
namespace {

using namespace ptx;

// One warp waits, with the library's bounded wait, on a barrier whose phase
// nothing ever completes.  The wait gives up after `limit_ns`, the kernel
// raises LVSPEC_DEV_WAIT_EXPIRED and returns normally.
__global__ void wait_expiry_kernel(uint32_t *status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ int abort_flag;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_fence_init();
        abort_flag = 0;
    }
    __syncthreads();
    const bool ok = mbar_wait_limit(bar, 0, &abort_flag, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_flag)) atomicOr(status, LVSPEC_DEV_WAIT_EXPIRED);
}

}  // namespace

cudaError_t launch_wait_expiry(uint32_t *status, unsigned long long limit_ns, cudaStream_t stream,
                               int *launches)
{
    wait_expiry_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace lvspec
