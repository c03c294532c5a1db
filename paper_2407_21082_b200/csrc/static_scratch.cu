// ee_exit_head_static: the decode-sized exit head for callers that cannot hand over scratch memory.
//
// The streaming kernel needs a little global scratch (a 256-byte control block and one 16-byte partial
// softmax state per CTA and row).  Here that scratch is a fixed array that lives in the library's own
// device image, so the call needs no workspace argument and never asks CUDA (or anybody else) for memory.
#include <mutex>

#include "common.cuh"
#include "kernels.h"

namespace ee {
namespace {

constexpr size_t kStaticScratchBytes = kCtrlBytes + (size_t)kStreamMaxCtas * kStreamMaxRows * sizeof(State);

// Lives on every GPU that loads the library, from load until exit (about 128 KB).  In host code this name
// is only a handle for cudaGetSymbolAddress; the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on `device` (which must be current).  The first call on a device
// resolves the symbol and zeroes the control block on `stream`.
ee_status scratch_for_device(int device, cudaStream_t stream, void** out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[device]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return EE_ERR_CUDA;
        if (cudaMemsetAsync(ptr, 0, kCtrlBytes, stream) != cudaSuccess) return EE_ERR_CUDA;
        g_scratch_ptr[device] = ptr;
    }
    *out = g_scratch_ptr[device];
    return EE_OK;
}

}  // namespace
}  // namespace ee

using namespace ee;

extern "C" ee_status ee_exit_head_static(const void* h, long long ld_h, const float* gamma, const float* beta,
                                         float ln_eps, const void* W, int M, int d, int V, const float* tau_per_row,
                                         float tau, int* argmax, float* entropy, float* maxprob,
                                         unsigned char* exit_mask, void* stream) {
    if (M < 0 || V < 1 || d < 8 || d > 8192 || (d % 8) != 0) return EE_ERR_SHAPE;
    if (M > EE_STATIC_MAX_ROWS) return EE_ERR_SHAPE;              // beyond the built-in scratch
    if (M == 0) return EE_OK;
    if (stream_slab_rows(d, 1) < M) return EE_ERR_SHAPE;              // rows of this width do not fit one launch
    if (!h || !gamma || !beta || !W || !argmax || !entropy || !maxprob || !exit_mask) return EE_ERR_NULL;
    if (ld_h < d || (ld_h % 8) != 0) return EE_ERR_SHAPE;
    auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(h) || misaligned(W) || misaligned(gamma) || misaligned(beta)) return EE_ERR_ALIGN;

    HeadArgs a{};
    if (cudaGetDevice(&a.device) != cudaSuccess || a.device < 0 || a.device >= kMaxDevices) return EE_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, a.device) != cudaSuccess ||
        cudaDeviceGetAttribute(&a.num_sms, cudaDevAttrMultiProcessorCount, a.device) != cudaSuccess)
        return EE_ERR_CUDA;
    if (major != 10) return EE_ERR_ARCH;
    a.stream = static_cast<cudaStream_t>(stream);
    void* scratch = nullptr;
    const ee_status st = scratch_for_device(a.device, a.stream, &scratch);
    if (st != EE_OK) return st;

    a.h = h; a.ld_h = ld_h; a.gamma = gamma; a.beta = beta; a.ln_eps = ln_eps; a.W = W;
    a.M = M; a.d = d; a.V = V; a.tau_per_row = tau_per_row; a.tau = tau;
    a.argmax = argmax; a.entropy = entropy; a.maxprob = maxprob; a.exit_mask = exit_mask;
    a.workspace = scratch;
    a.workspace_bytes = kStaticScratchBytes;
    return stream_launch(&a, 1);
}

namespace {
// Device checks and the array's address for the two small calls below.
ee_status static_scratch_here(cudaStream_t stream, void** scratch) {
    int device = 0, major = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return EE_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) return EE_ERR_CUDA;
    if (major != 10) return EE_ERR_ARCH;
    return scratch_for_device(device, stream, scratch);
}
}  // namespace

extern "C" ee_status ee_exit_head_static_query_error(void* stream) {
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    void* scratch = nullptr;
    const ee_status st = static_scratch_here(s, &scratch);
    if (st != EE_OK) return st;
    unsigned int words[3] = {0, 0, 0};
    if (cudaMemcpyAsync(words, scratch, sizeof(words), cudaMemcpyDeviceToHost, s) != cudaSuccess) return EE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return EE_ERR_CUDA;
    if (words[1] == 0) return EE_OK;
    // A wait gave up: put the whole control block (error word, completion counters) back to its initial state.
    if (cudaMemsetAsync(scratch, 0, kCtrlBytes, s) != cudaSuccess) return EE_ERR_CUDA;
    return EE_ERR_TIMEOUT;
}

extern "C" ee_status ee_exit_head_static_selftest_timeout(void* stream) {
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    void* scratch = nullptr;
    const ee_status st = static_scratch_here(s, &scratch);
    if (st != EE_OK) return st;
    return selftest_wait_timeout_launch(scratch, s);
}
