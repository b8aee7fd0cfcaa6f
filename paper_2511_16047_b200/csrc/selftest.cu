// Diagnostic kernel: exercises the give-up path of the bounded waits without any real failure.
// One warp waits, with a small iteration limit, on a barrier that nobody ever arrives at; the wait runs
// out, the status code is recorded exactly as the attention kernels record theirs, and the kernel
// returns normally.
#include "kernels.cuh"
#include "sm100_ptx.cuh"

namespace amskv {

namespace {

__global__ void __launch_bounds__(32) wait_gives_up_kernel(uint32_t limit, int* __restrict__ status)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // phase 0 of a barrier with one expected arrival and no arriver never completes
    const bool done = ptx::warp_wait(ptx::smem_u32(&bar), 0u, &abort_flag, limit);
    if (!done && threadIdx.x == 0) ptx::report(status, kStatusSyncTimeout, &abort_flag);
}

}  // namespace

cudaError_t launch_wait_gives_up(uint32_t limit, int* status, cudaStream_t stream)
{
    wait_gives_up_kernel<<<1, 32, 0, stream>>>(limit, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace amskv
