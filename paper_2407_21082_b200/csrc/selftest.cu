// Diagnostic: drives the error path of the bounded device-side waits without any fault.  One CTA waits on an
// mbarrier that nothing ever arrives at; its wait gives up after a short, fixed number of polls, records the
// error word in the control block exactly as the tensor-core kernel's roles do, and the kernel returns normally.
#include "common.cuh"
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace ee {

namespace {

constexpr unsigned int kSelftestPolls = 20000;        // about a millisecond with the sleep below

__global__ void __launch_bounds__(32) wait_timeout_selftest_kernel(Control* ctrl) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = ptx::smem_addr(&bar);
    if (threadIdx.x == 0) {
        ptx::mbar_init(b, 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        bool done = false;
        for (unsigned int i = 0; i < kSelftestPolls && !done; ++i) {
            done = ptx::mbar_try_wait(b, 0);
            if (!done) __nanosleep(50);
        }
        if (!done && atomicCAS(&ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
            ctrl->error_info = (0x7fu << 24);            // role 0x7f: the self-test
    }
}

}  // namespace

ee_status selftest_wait_timeout_launch(void* workspace, cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(static_cast<Control*>(workspace));
    return cudaGetLastError() == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace ee
