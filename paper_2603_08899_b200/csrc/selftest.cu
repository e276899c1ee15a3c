// Self-test of the bounded wait that every mbarrier wait of the tensor-core kernels goes through.
//
// One warp waits, with the same mbar_wait, on a barrier that nothing ever arrives at.  The wait
// runs out after the given wall-clock limit, the kernel writes CONFU_ST_TIMEOUT and returns: the
// give-up branch is exercised without a kernel that misbehaves, and the context stays usable.
#include "tc_ptx.cuh"

namespace confu {

__global__ void __launch_bounds__(32) bounded_wait_kernel(unsigned long long limit_ns, int32_t* status)
{
    __shared__ uint64_t bar;
    __shared__ int abort;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool arrived = tc::mbar_wait(&bar, 0, &abort, limit_ns);
    __syncwarp();
    if (threadIdx.x == 0) status[0] = arrived ? CONFU_ST_OK : CONFU_ST_TIMEOUT;
}

cudaError_t launch_bounded_wait(unsigned long long limit_ns, int32_t* status, cudaStream_t st)
{
    bounded_wait_kernel<<<1, 32, 0, st>>>(limit_ns, status);
    return cudaGetLastError();
}

}  // namespace confu
