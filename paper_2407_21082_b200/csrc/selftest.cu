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

// Diagnostic: what a read-only stream reaches on this device with the mechanism the kernels stream weights with
// (contiguous bulk asynchronous copies into a shared-memory ring, one CTA per SM, one issuing thread).  Every
// CTA walks its own contiguous range of 16 KB stages; a slot is refilled as soon as its copy has landed (the
// bytes are not looked at).  Waits are bounded like everywhere else.
constexpr int kReadStage = 16384;
constexpr int kReadSlots = 12;

__global__ void __launch_bounds__(32) read_stream_selftest_kernel(const unsigned char* __restrict__ src, long long n_stages,
                                                                  Control* ctrl) {
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) unsigned long long bars[kReadSlots];
    __shared__ int abort_flag;
    if (threadIdx.x != 0) return;
    abort_flag = 0;
    const long long per = (n_stages + gridDim.x - 1) / gridDim.x;
    const long long first = per * blockIdx.x;
    const long long mine = max(0ll, min(per, n_stages - first));
    for (int s = 0; s < kReadSlots; ++s) ptx::mbar_init(ptx::smem_addr(&bars[s]), 1);
    ptx::fence_mbar_init();
    const uint32_t ring_addr = ptx::smem_addr(ring);
    auto issue = [&](long long j) {
        const int slot = (int)(j % kReadSlots);
        const uint32_t bar = ptx::smem_addr(&bars[slot]);
        ptx::mbar_arrive_expect_tx(bar, kReadStage);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(ring_addr + slot * kReadStage), "l"(src + (first + j) * kReadStage), "r"(kReadStage), "r"(bar)
                     : "memory");
    };
    long long issued = 0;
    for (; issued < mine && issued < kReadSlots; ++issued) issue(issued);
    bool ok = true;
    for (long long j = 0; j < mine; ++j) {
        const int slot = (int)(j % kReadSlots);
        const uint32_t parity = (uint32_t)((j / kReadSlots) & 1);
        if (ok && !ptx::mbar_wait(ptx::smem_addr(&bars[slot]), parity, &abort_flag)) {
            if (atomicCAS(&ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u) ctrl->error_info = (0x7eu << 24) | (unsigned)slot;
            ok = false;
        }
        if (!ok) {
            // no further copies; the ones in flight land before the shared memory is given back (bounded)
            if (j < issued)
                for (uint32_t i = 0; i < (1u << 16) && !ptx::mbar_try_wait(ptx::smem_addr(&bars[slot]), parity); ++i) __nanosleep(100);
            continue;
        }
        if (issued < mine) issue(issued++);
    }
}

}  // namespace

ee_status selftest_read_stream_launch(const void* src, size_t bytes, void* workspace, int num_sms, cudaStream_t stream) {
    const size_t smem = (size_t)kReadSlots * kReadStage;
    static int configured_device = -1;      // the attribute is per device; set it when the device changes
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return EE_ERR_CUDA;
    if (configured_device != device) {
        if (cudaFuncSetAttribute(read_stream_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return EE_ERR_CUDA;
        configured_device = device;
    }
    read_stream_selftest_kernel<<<num_sms, 32, smem, stream>>>(static_cast<const unsigned char*>(src),
                                                               (long long)(bytes / kReadStage), static_cast<Control*>(workspace));
    return cudaGetLastError() == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

ee_status selftest_wait_timeout_launch(void* workspace, cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(static_cast<Control*>(workspace));
    return cudaGetLastError() == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace ee
