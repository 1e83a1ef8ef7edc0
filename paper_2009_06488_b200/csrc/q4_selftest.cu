// Diagnostic for the bounded device-side waits (no counterpart in the paper).  Every kernel
// of this library that waits on an mbarrier does so through mbar_wait*, which gives up
// after a clock limit, raises the kernel's abort flag and sets the timeout bit of the device
// status word that q4_last_device_status reports.  This kernel waits, with the short limit
// (about a millisecond), on a barrier that nothing ever arrives on, so that the whole
// reporting path can be exercised without any kernel hanging or faulting.
#include "q4_common.cuh"
#include "q4_tc_ptx.cuh"

namespace q4 {

unsigned* device_status_ptr();     // the device status word (q4_api.cu)

__global__ void wait_selftest_kernel(unsigned* status, int* outcome)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 1;                               // selects the short limit
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool completed = mbar_wait(smem_u32(&bar), 0, smem_u32(&abort_flag), status);
        if (outcome) *outcome = completed ? 1 : 2;    // 2 = the wait ran out, as it must
    }
}

cudaError_t launch_wait_selftest(int* outcome_dev, cudaStream_t st)
{
    unsigned* status = device_status_ptr();
    if (!status) return cudaErrorUnknown;
    wait_selftest_kernel<<<1, 32, 0, st>>>(status, outcome_dev);
    count_launch();
    return cudaGetLastError();
}

}  // namespace q4
