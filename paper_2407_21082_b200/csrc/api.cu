// The C ABI: argument validation, device checks, kernel selection.  No compute happens here.
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "kernels.h"

namespace ee {
namespace {

struct DeviceInfo {
    bool known = false;
    bool sm100 = false;
    int num_sms = 0;
};

// Properties of the current device (cached per ordinal).
ee_status current_device(int* device, int* num_sms) {
    static DeviceInfo info[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EE_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return EE_ERR_CUDA;
    if (!info[dev].known) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return EE_ERR_CUDA;
        info[dev].sm100 = (major == 10);
        info[dev].num_sms = sms;
        info[dev].known = true;
    }
    if (!info[dev].sm100) return EE_ERR_ARCH;
    *device = dev;
    *num_sms = info[dev].num_sms;
    return EE_OK;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

bool sizes_ok(int M, int d, int V) { return M >= 0 && V >= 1 && d >= 8 && d <= 8192 && (d % 8) == 0; }

// Kernel used when the caller does not choose: the tensor-core path for every size.  (Measured per head call,
// d = 512..2560, V = 50304: it is ahead of the streaming kernel from M = 1 on, 16.3 against 17.4 us at
// d = 512 M = 1 and 41.8 against 56.7 us at d = 2048 M = 16; the other two kernels stay selectable.)
int auto_path(int, int) { return EE_PATH_TCGEN05; }

// Heads one launch (sequence) of any of the three kernels takes.
constexpr int kHeadsPerLaunch = 4;
static_assert(kStreamMaxHeads == kHeadsPerLaunch && kSkinnyMaxHeads == kHeadsPerLaunch && kGemmLaunchMaxHeads == kHeadsPerLaunch,
              "the multi-head entry point cuts its heads into groups every kernel accepts");

size_t workspace_bytes(int M, int d, int V) {
    size_t need = gemm_workspace_bytes(M, d, V, 1);
    const size_t s = stream_workspace_bytes(1);
    if (s > need) need = s;
    if (skinny_workspace_bytes(1) > need) need = skinny_workspace_bytes(1);
    return kCtrlBytes + need;
}

}  // namespace
}  // namespace ee

using namespace ee;

extern "C" {

const char* ee_status_string(ee_status status) {
    switch (status) {
        case EE_OK: return "ok";
        case EE_ERR_NULL: return "a required pointer is NULL";
        case EE_ERR_SHAPE: return "a size is out of range";
        case EE_ERR_ALIGN: return "a pointer or stride is misaligned";
        case EE_ERR_WORKSPACE: return "workspace too small";
        case EE_ERR_ARCH: return "device is not sm_100";
        case EE_ERR_CUDA: return "a CUDA call failed";
        case EE_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    }
    return "unknown status";
}

size_t ee_exit_head_workspace_bytes(int M, int d, int V) {
    if (!sizes_ok(M, d, V)) return 0;
    return workspace_bytes(M, d, V);
}

int ee_exit_head_launches(int M, int d, int V, int path) {
    if (!sizes_ok(M, d, V) || M == 0) return 0;
    if (path == EE_PATH_AUTO) path = auto_path(M, d);
    if (path == EE_PATH_STREAM) {
        const int slab = stream_slab_rows(d, 1);
        return slab > 0 ? (M + slab - 1) / slab : 0;
    }
    if (path == EE_PATH_SKINNY) return skinny_supports(M, d) ? 1 : 0;
    return path == EE_PATH_TCGEN05 ? gemm_launches(M, 1) : 0;
}

ee_status ee_workspace_init(void* workspace, size_t workspace_bytes_, void* stream) {
    if (!workspace) return EE_ERR_NULL;
    if (!aligned(workspace, 256)) return EE_ERR_ALIGN;
    if (workspace_bytes_ < (size_t)kCtrlBytes) return EE_ERR_WORKSPACE;
    return cudaMemsetAsync(workspace, 0, kCtrlBytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? EE_OK
                                                                                                       : EE_ERR_CUDA;
}

ee_status ee_exit_head_path(const void* h, long long ld_h, const float* gamma, const float* beta, float ln_eps,
                            const void* W, int M, int d, int V, const float* tau_per_row, float tau, int* argmax,
                            float* entropy, float* maxprob, unsigned char* exit_mask, void* workspace,
                            size_t workspace_bytes_, void* stream, int path) {
    if (!sizes_ok(M, d, V)) return EE_ERR_SHAPE;
    if (path < EE_PATH_AUTO || path > EE_PATH_SKINNY) return EE_ERR_SHAPE;
    if (M == 0) return EE_OK;
    if (!h || !gamma || !beta || !W || !argmax || !entropy || !maxprob || !exit_mask || !workspace) return EE_ERR_NULL;
    if (ld_h < d || (ld_h % 8) != 0) return EE_ERR_SHAPE;
    if (!aligned(h, 16) || !aligned(W, 16) || !aligned(gamma, 16) || !aligned(beta, 16) || !aligned(workspace, 256))
        return EE_ERR_ALIGN;
    if (workspace_bytes_ < workspace_bytes(M, d, V)) return EE_ERR_WORKSPACE;

    HeadArgs a{};
    const ee_status dev = current_device(&a.device, &a.num_sms);
    if (dev != EE_OK) return dev;
    a.h = h; a.ld_h = ld_h; a.gamma = gamma; a.beta = beta; a.ln_eps = ln_eps; a.W = W;
    a.M = M; a.d = d; a.V = V; a.tau_per_row = tau_per_row; a.tau = tau;
    a.argmax = argmax; a.entropy = entropy; a.maxprob = maxprob; a.exit_mask = exit_mask;
    a.workspace = workspace; a.workspace_bytes = workspace_bytes_;
    a.stream = static_cast<cudaStream_t>(stream);

    if (path == EE_PATH_AUTO) path = auto_path(M, d);
    if (path == EE_PATH_STREAM) return stream_launch(&a, 1);
    if (path == EE_PATH_SKINNY) return skinny_launch(&a, 1);
    return gemm_launch(&a, 1);
}

ee_status ee_exit_head_top2(const void* h, long long ld_h, const float* gamma, const float* beta, float ln_eps,
                            const void* W, int M, int d, int V, const float* tau_per_row, float tau, int* argmax,
                            float* entropy, float* maxprob, float* top2gap, unsigned char* exit_mask, void* workspace,
                            size_t workspace_bytes_, void* stream) {
    if (!sizes_ok(M, d, V)) return EE_ERR_SHAPE;
    if (M == 0) return EE_OK;
    if (!h || !gamma || !beta || !W || !argmax || !entropy || !maxprob || !top2gap || !exit_mask || !workspace) return EE_ERR_NULL;
    if (ld_h < d || (ld_h % 8) != 0) return EE_ERR_SHAPE;
    if (!aligned(h, 16) || !aligned(W, 16) || !aligned(gamma, 16) || !aligned(beta, 16) || !aligned(workspace, 256))
        return EE_ERR_ALIGN;
    if (workspace_bytes_ < workspace_bytes(M, d, V)) return EE_ERR_WORKSPACE;
    HeadArgs a{};
    const ee_status dev = current_device(&a.device, &a.num_sms);
    if (dev != EE_OK) return dev;
    a.h = h; a.ld_h = ld_h; a.gamma = gamma; a.beta = beta; a.ln_eps = ln_eps; a.W = W;
    a.M = M; a.d = d; a.V = V; a.tau_per_row = tau_per_row; a.tau = tau;
    a.argmax = argmax; a.entropy = entropy; a.maxprob = maxprob; a.exit_mask = exit_mask; a.top2gap = top2gap;
    a.workspace = workspace; a.workspace_bytes = workspace_bytes_;
    a.stream = static_cast<cudaStream_t>(stream);
    return gemm_launch(&a, 1);
}

size_t ee_exit_head_multi_workspace_bytes(int n_heads, int M, int d, int V) {
    if (!sizes_ok(M, d, V) || n_heads < 1) return 0;
    size_t need = workspace_bytes(M, d, V);
    const int per_launch = n_heads < kHeadsPerLaunch ? n_heads : kHeadsPerLaunch;
    if (kCtrlBytes + skinny_workspace_bytes(per_launch) > need) need = kCtrlBytes + skinny_workspace_bytes(per_launch);
    if (kCtrlBytes + stream_workspace_bytes(per_launch) > need) need = kCtrlBytes + stream_workspace_bytes(per_launch);
    if (kCtrlBytes + gemm_workspace_bytes(M, d, V, per_launch) > need) need = kCtrlBytes + gemm_workspace_bytes(M, d, V, per_launch);
    return need;
}

int ee_exit_head_multi_launches(int n_heads, int M, int d, int V) {
    if (!sizes_ok(M, d, V) || n_heads < 1 || M == 0) return 0;
    int launches = 0;
    for (int k0 = 0; k0 < n_heads; k0 += kGemmLaunchMaxHeads)
        launches += gemm_launches(M, n_heads - k0 < kGemmLaunchMaxHeads ? n_heads - k0 : kGemmLaunchMaxHeads);
    return launches;
}

ee_status ee_exit_head_multi(const ee_head* heads, int n_heads, float ln_eps, int M, int d, int V, void* workspace,
                             size_t workspace_bytes_, void* stream) {
    if (!sizes_ok(M, d, V) || n_heads < 0) return EE_ERR_SHAPE;
    if (n_heads == 0 || M == 0) return EE_OK;
    if (!heads || !workspace) return EE_ERR_NULL;
    if (!aligned(workspace, 256)) return EE_ERR_ALIGN;
    if (workspace_bytes_ < ee_exit_head_multi_workspace_bytes(n_heads, M, d, V)) return EE_ERR_WORKSPACE;
    for (int k = 0; k < n_heads; ++k) {
        const ee_head& e = heads[k];
        if (!e.h || !e.gamma || !e.beta || !e.W || !e.argmax || !e.entropy || !e.maxprob || !e.exit_mask) return EE_ERR_NULL;
        if (e.ld_h < d || (e.ld_h % 8) != 0) return EE_ERR_SHAPE;
        if (!aligned(e.h, 16) || !aligned(e.W, 16) || !aligned(e.gamma, 16) || !aligned(e.beta, 16)) return EE_ERR_ALIGN;
    }
    HeadArgs base{};
    const ee_status dev = current_device(&base.device, &base.num_sms);
    if (dev != EE_OK) return dev;
    // The tensor-core path batches the heads (one LayerNorm, one GEMM, one merge launch for up to four).
    // EE_MULTI_KERNEL=stream | skinny | gemm | none overrides the choice (for A/B timing; a kernel that does
    // not take the shape leaves the default).
    enum { kNone, kStream, kSkinny, kGemm } mode = kGemm;
    const int chunk = n_heads < kHeadsPerLaunch ? n_heads : kHeadsPerLaunch;
    const bool stream_ok = stream_slab_rows(d, chunk) >= M;
    if (const char* force = getenv("EE_MULTI_KERNEL")) {
        if (!strcmp(force, "stream") && stream_ok) mode = kStream;
        else if (!strcmp(force, "skinny") && skinny_supports(M, d)) mode = kSkinny;
        else if (!strcmp(force, "gemm")) mode = kGemm;
        else if (!strcmp(force, "none")) mode = kNone;
    }
    for (int k0 = 0; k0 < n_heads; k0 += kHeadsPerLaunch) {
        HeadArgs a[kHeadsPerLaunch];
        const int n = n_heads - k0 < kHeadsPerLaunch ? n_heads - k0 : kHeadsPerLaunch;
        for (int k = 0; k < n; ++k) {
            const ee_head& e = heads[k0 + k];
            a[k] = base;
            a[k].h = e.h; a[k].ld_h = e.ld_h; a[k].gamma = e.gamma; a[k].beta = e.beta; a[k].ln_eps = ln_eps; a[k].W = e.W;
            a[k].M = M; a[k].d = d; a[k].V = V; a[k].tau_per_row = e.tau_per_row; a[k].tau = e.tau;
            a[k].argmax = e.argmax; a[k].entropy = e.entropy; a[k].maxprob = e.maxprob; a[k].exit_mask = e.exit_mask;
            a[k].workspace = workspace; a[k].workspace_bytes = workspace_bytes_;
            a[k].stream = static_cast<cudaStream_t>(stream);
        }
        if (mode != kNone) {
            const ee_status st = mode == kStream ? stream_launch(a, n) : mode == kSkinny ? skinny_launch(a, n) : gemm_launch(a, n);
            if (st != EE_OK) return st;
        } else {
            for (int k = 0; k < n; ++k) {
                const ee_status st = auto_path(M, d) == EE_PATH_STREAM ? stream_launch(&a[k], 1) : gemm_launch(&a[k], 1);
                if (st != EE_OK) return st;
            }
        }
    }
    return EE_OK;
}

namespace {
struct PlanHeader {
    int n_groups;
    int device;
    int pad[14];
};
static_assert(sizeof(PlanHeader) == 64, "plan header");
static_assert(EE_EXIT_HEAD_PLAN_BYTES == 64 + (EE_PLAN_MAX_HEADS / kHeadsPerLaunch) * kGemmPlanBytes, "plan size in eexit.h");
}  // namespace

ee_status ee_exit_head_plan_init(ee_exit_head_plan* plan, const ee_head* heads, int n_heads, float ln_eps, int M, int d, int V,
                                 void* workspace, size_t workspace_bytes_) {
    if (!plan) return EE_ERR_NULL;
    if (!sizes_ok(M, d, V) || n_heads < 1 || n_heads > EE_PLAN_MAX_HEADS || M < 1) return EE_ERR_SHAPE;
    if (!heads || !workspace) return EE_ERR_NULL;
    if (!aligned(workspace, 256)) return EE_ERR_ALIGN;
    if (workspace_bytes_ < ee_exit_head_multi_workspace_bytes(n_heads, M, d, V)) return EE_ERR_WORKSPACE;
    for (int k = 0; k < n_heads; ++k) {
        const ee_head& e = heads[k];
        if (!e.h || !e.gamma || !e.beta || !e.W || !e.argmax || !e.entropy || !e.maxprob || !e.exit_mask) return EE_ERR_NULL;
        if (e.ld_h < d || (e.ld_h % 8) != 0) return EE_ERR_SHAPE;
        if (!aligned(e.h, 16) || !aligned(e.W, 16) || !aligned(e.gamma, 16) || !aligned(e.beta, 16)) return EE_ERR_ALIGN;
    }
    HeadArgs base{};
    const ee_status dev = current_device(&base.device, &base.num_sms);
    if (dev != EE_OK) return dev;
    unsigned char* bytes = reinterpret_cast<unsigned char*>(plan->opaque);
    PlanHeader* hdr = reinterpret_cast<PlanHeader*>(bytes);
    memset(hdr, 0, sizeof(*hdr));
    hdr->device = base.device;
    for (int k0 = 0; k0 < n_heads; k0 += kHeadsPerLaunch) {
        HeadArgs a[kHeadsPerLaunch];
        const int n = n_heads - k0 < kHeadsPerLaunch ? n_heads - k0 : kHeadsPerLaunch;
        for (int k = 0; k < n; ++k) {
            const ee_head& e = heads[k0 + k];
            a[k] = base;
            a[k].h = e.h; a[k].ld_h = e.ld_h; a[k].gamma = e.gamma; a[k].beta = e.beta; a[k].ln_eps = ln_eps; a[k].W = e.W;
            a[k].M = M; a[k].d = d; a[k].V = V; a[k].tau_per_row = e.tau_per_row; a[k].tau = e.tau;
            a[k].argmax = e.argmax; a[k].entropy = e.entropy; a[k].maxprob = e.maxprob; a[k].exit_mask = e.exit_mask;
            a[k].workspace = workspace; a[k].workspace_bytes = workspace_bytes_;
        }
        const ee_status st = gemm_plan(a, n, bytes + sizeof(PlanHeader) + (size_t)hdr->n_groups * kGemmPlanBytes);
        if (st != EE_OK) return st;
        ++hdr->n_groups;
    }
    return EE_OK;
}

ee_status ee_exit_head_plan_run(const ee_exit_head_plan* plan, void* stream) {
    if (!plan) return EE_ERR_NULL;
    const unsigned char* bytes = reinterpret_cast<const unsigned char*>(plan->opaque);
    const PlanHeader* hdr = reinterpret_cast<const PlanHeader*>(bytes);
    if (hdr->n_groups < 1 || hdr->n_groups > EE_PLAN_MAX_HEADS / kHeadsPerLaunch) return EE_ERR_SHAPE;      // not initialised
    for (int g = 0; g < hdr->n_groups; ++g) {
        const ee_status st = gemm_run(bytes + sizeof(PlanHeader) + (size_t)g * kGemmPlanBytes, static_cast<cudaStream_t>(stream));
        if (st != EE_OK) return st;
    }
    return EE_OK;
}

ee_status ee_exit_head_plan_run_host(const ee_exit_head_plan* plan, const void* h_host, void* h_dev, size_t h_bytes,
                                     void* results_host, const void* results_dev, size_t results_bytes, void* stream) {
    if (!plan || !h_host || !h_dev || !results_host || !results_dev) return EE_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(h_dev, h_host, h_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return EE_ERR_CUDA;
    const ee_status st = ee_exit_head_plan_run(plan, stream);
    if (st != EE_OK) return st;
    return cudaMemcpyAsync(results_host, results_dev, results_bytes, cudaMemcpyDeviceToHost, s) == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

ee_status ee_exit_head(const void* h, long long ld_h, const float* gamma, const float* beta, float ln_eps,
                       const void* W, int M, int d, int V, const float* tau_per_row, float tau, int* argmax,
                       float* entropy, float* maxprob, unsigned char* exit_mask, void* workspace,
                       size_t workspace_bytes_, void* stream) {
    return ee_exit_head_path(h, ld_h, gamma, beta, ln_eps, W, M, d, V, tau_per_row, tau, argmax, entropy, maxprob,
                             exit_mask, workspace, workspace_bytes_, stream, EE_PATH_AUTO);
}

ee_status ee_exit_head_host(const void* h_host, void* h_dev, const float* gamma, const float* beta, float ln_eps,
                            const void* W, int M, int d, int V, const float* tau_per_row, float tau,
                            int* argmax_host, float* entropy_host, float* maxprob_host, unsigned char* exit_mask_host,
                            int* argmax_dev, float* entropy_dev, float* maxprob_dev, unsigned char* exit_mask_dev,
                            void* workspace, size_t workspace_bytes_, void* stream) {
    if (!sizes_ok(M, d, V)) return EE_ERR_SHAPE;
    if (M == 0) return EE_OK;
    if (!h_host || !h_dev || !argmax_host || !entropy_host || !maxprob_host || !exit_mask_host) return EE_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(h_dev, h_host, (size_t)M * d * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return EE_ERR_CUDA;
    const ee_status st = ee_exit_head(h_dev, d, gamma, beta, ln_eps, W, M, d, V, tau_per_row, tau, argmax_dev,
                                      entropy_dev, maxprob_dev, exit_mask_dev, workspace, workspace_bytes_, stream);
    if (st != EE_OK) return st;
    if (cudaMemcpyAsync(argmax_host, argmax_dev, (size_t)M * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemcpyAsync(entropy_host, entropy_dev, (size_t)M * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemcpyAsync(maxprob_host, maxprob_dev, (size_t)M * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemcpyAsync(exit_mask_host, exit_mask_dev, (size_t)M, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return EE_ERR_CUDA;
    return EE_OK;
}

size_t ee_exit_head_results_bytes(int n_heads, int M) {
    if (n_heads < 1 || M < 0) return 0;
    return (size_t)n_heads * (((size_t)13 * M + 15) / 16 * 16);
}

ee_status ee_exit_head_multi_host(const ee_head* heads, int n_heads, float ln_eps, int M, int d, int V,
                                  const void* h_host, void* h_dev, void* results_host, void* results_dev,
                                  void* workspace, size_t workspace_bytes_, void* stream) {
    if (!sizes_ok(M, d, V) || n_heads < 0 || n_heads > 64) return EE_ERR_SHAPE;
    if (n_heads == 0 || M == 0) return EE_OK;
    if (!heads || !h_host || !h_dev || !results_host || !results_dev) return EE_ERR_NULL;
    if (!aligned(h_dev, 16) || !aligned(results_dev, 16)) return EE_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t h_bytes = (size_t)M * d * 2, block = ee_exit_head_results_bytes(1, M);
    ee_head dev_heads[64];
    for (int k = 0; k < n_heads; ++k) {
        unsigned char* r = static_cast<unsigned char*>(results_dev) + k * block;
        dev_heads[k] = heads[k];
        dev_heads[k].h = static_cast<unsigned char*>(h_dev) + k * h_bytes;
        dev_heads[k].ld_h = d;
        dev_heads[k].argmax = reinterpret_cast<int*>(r);
        dev_heads[k].entropy = reinterpret_cast<float*>(r + (size_t)4 * M);
        dev_heads[k].maxprob = reinterpret_cast<float*>(r + (size_t)8 * M);
        dev_heads[k].exit_mask = r + (size_t)12 * M;
    }
    if (cudaMemcpyAsync(h_dev, h_host, n_heads * h_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return EE_ERR_CUDA;
    const ee_status st = ee_exit_head_multi(dev_heads, n_heads, ln_eps, M, d, V, workspace, workspace_bytes_, stream);
    if (st != EE_OK) return st;
    if (cudaMemcpyAsync(results_host, results_dev, n_heads * block, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return EE_ERR_CUDA;
    return EE_OK;
}

ee_status ee_compact(const unsigned char* exit_mask, const void* h, long long ld_h, int M, int d, int* kept_idx,
                     int* kept_count, void* h_out, void* stream) {
    if (M < 0) return EE_ERR_SHAPE;
    if (!kept_count) return EE_ERR_NULL;
    if (M > 0 && (!exit_mask || !kept_idx)) return EE_ERR_NULL;
    if (h_out) {
        if (M > 0 && !h) return EE_ERR_NULL;
        if (d < 8 || (d % 8) != 0 || ld_h < d || (ld_h % 8) != 0) return EE_ERR_SHAPE;
        if (!aligned(h, 16) || !aligned(h_out, 16)) return EE_ERR_ALIGN;
    }
    int device, num_sms;
    const ee_status dev = current_device(&device, &num_sms);
    if (dev != EE_OK) return dev;
    return compact_launch(exit_mask, h, ld_h, M, d, kept_idx, kept_count, h_out, static_cast<cudaStream_t>(stream));
}

ee_status dssd_accept(const int* draft_tok, const unsigned char* draft_exit_mask, const int* verify_tok, int S, int k,
                      int kv, int* draft_len, int* accept_len, int* next_tok, void* stream) {
    if (S < 0 || k < 1 || kv < k) return EE_ERR_SHAPE;
    if (S == 0) return EE_OK;
    if (!draft_tok || !verify_tok || !draft_len || !accept_len || !next_tok) return EE_ERR_NULL;
    int device, num_sms;
    const ee_status dev = current_device(&device, &num_sms);
    if (dev != EE_OK) return dev;
    return accept_launch(draft_tok, draft_exit_mask, verify_tok, S, k, kv, draft_len, accept_len, next_tok,
                         static_cast<cudaStream_t>(stream));
}

ee_status ee_compact_accept(const unsigned char* exit_mask, const void* h, long long ld_h, int M, int d, int* kept_idx,
                            int* kept_count, void* h_out, const int* draft_tok, const unsigned char* draft_exit_mask,
                            const int* verify_tok, int S, int k, int kv, int* draft_len, int* accept_len,
                            int* next_tok, void* stream) {
    if (M < 0 || S < 0 || k < 1 || kv < k) return EE_ERR_SHAPE;
    if (!kept_count) return EE_ERR_NULL;
    if (M > 0 && (!exit_mask || !kept_idx)) return EE_ERR_NULL;
    if (h_out) {
        if (M > 0 && !h) return EE_ERR_NULL;
        if (d < 8 || (d % 8) != 0 || ld_h < d || (ld_h % 8) != 0) return EE_ERR_SHAPE;
        if (!aligned(h, 16) || !aligned(h_out, 16)) return EE_ERR_ALIGN;
    }
    if (S > 0 && (!draft_tok || !verify_tok || !draft_len || !accept_len || !next_tok)) return EE_ERR_NULL;
    int device, num_sms;
    const ee_status dev = current_device(&device, &num_sms);
    if (dev != EE_OK) return dev;
    return compact_accept_launch(exit_mask, h, ld_h, M, d, kept_idx, kept_count, h_out, draft_tok, draft_exit_mask,
                                 verify_tok, S, k, kv, draft_len, accept_len, next_tok,
                                 static_cast<cudaStream_t>(stream));
}

namespace {
size_t cascade_head_ws(int M, int d, int V) { return align_up(kCtrlBytes + gemm_workspace_bytes(M, d, V, 1), 256); }
size_t cascade_rows_bytes(int M) { return align_up((size_t)M * 4, 256); }
// small batches: up to four heads per launch on all rows, four result arrays per head
// Up to this many rows ee_cascade evaluates every head on every row.  Measured on the c1 shape, three heads, 45 %
// of the rows answered by the first head: 512 rows 131 us against 161 us head by head, 1024 rows 252 against
// 262; the more rows leave early, the sooner head by head wins, so the switch sits where the margin is clear.
// EE_CASCADE_ALL_ROWS_MAX in the environment (read once) moves it, for A/B timing.
constexpr int kCascadeAllRowsMax = 512;
int cascade_all_rows_max() {
    static const int v = [] {
        const char* e = getenv("EE_CASCADE_ALL_ROWS_MAX");
        const int cap = cascade_select_max_rows();
        const int x = e ? atoi(e) : kCascadeAllRowsMax;
        return x < 0 ? 0 : x > cap ? cap : x;
    }();
    return v;
}
size_t cascade_group_ws(int M, int d, int V) {
    return align_up(kCtrlBytes + gemm_workspace_bytes(M, d, V, kHeadsPerLaunch), 256);
}
}  // namespace

size_t ee_cascade_workspace_bytes(int M, int d, int V) {
    if (!sizes_ok(M, d, V)) return 0;
    const size_t by_step = cascade_head_ws(M, d, V) + 6 * cascade_rows_bytes(M) + 256;
    if (M > cascade_all_rows_max()) return by_step;
    const size_t by_group = cascade_group_ws(M, d, V) + 4 * kHeadsPerLaunch * cascade_rows_bytes(M);
    return by_group > by_step ? by_group : by_step;
}

ee_status ee_cascade(const ee_head* heads, int n_heads, float ln_eps, int M, int d, int V, int* exit_head, int* token,
                     float* entropy, int* rows_in, void* workspace, size_t workspace_bytes_, void* stream) {
    if (!sizes_ok(M, d, V) || n_heads < 1 || n_heads > 64) return EE_ERR_SHAPE;
    if (!heads || !rows_in || !workspace) return EE_ERR_NULL;
    if (M > 0 && (!exit_head || !token || !entropy)) return EE_ERR_NULL;
    if (!aligned(workspace, 256)) return EE_ERR_ALIGN;
    if (workspace_bytes_ < ee_cascade_workspace_bytes(M, d, V)) return EE_ERR_WORKSPACE;
    for (int k = 0; k < n_heads; ++k) {
        const ee_head& e = heads[k];
        if (M > 0 && (!e.h || !e.gamma || !e.beta || !e.W)) return EE_ERR_NULL;
        if (e.tau_per_row) return EE_ERR_SHAPE;          // thresholds belong to heads here, not to rows
        if (e.ld_h < d || (e.ld_h % 8) != 0) return EE_ERR_SHAPE;
        if (!aligned(e.h, 16) || !aligned(e.W, 16) || !aligned(e.gamma, 16) || !aligned(e.beta, 16)) return EE_ERR_ALIGN;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (M == 0) return cudaMemsetAsync(rows_in, 0, (size_t)n_heads * sizeof(int), s) == cudaSuccess ? EE_OK : EE_ERR_CUDA;
    HeadArgs a{};
    const ee_status dev = current_device(&a.device, &a.num_sms);
    if (dev != EE_OK) return dev;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    const size_t rb = cascade_rows_bytes(M);
    if (M <= cascade_all_rows_max()) {
        // Evaluating a head on all rows costs little more than evaluating it on the open rows while its weight
        // stream bounds the call, and sparing the per-head chain of launches pays for the rest: the heads go
        // through the batched launch four at a time and a one-CTA kernel picks each row's first answer.
        unsigned char* q = ws + cascade_group_ws(M, d, V);
        for (int k0 = 0; k0 < n_heads; k0 += kHeadsPerLaunch) {
            HeadArgs g[kHeadsPerLaunch];
            const int n = n_heads - k0 < kHeadsPerLaunch ? n_heads - k0 : kHeadsPerLaunch;
            for (int k = 0; k < n; ++k) {
                const ee_head& e = heads[k0 + k];
                g[k] = a;
                g[k].h = e.h; g[k].ld_h = e.ld_h; g[k].gamma = e.gamma; g[k].beta = e.beta; g[k].ln_eps = ln_eps; g[k].W = e.W;
                g[k].M = M; g[k].d = d; g[k].V = V; g[k].tau_per_row = nullptr; g[k].tau = e.tau;
                unsigned char* r = q + (size_t)k * 4 * rb;
                g[k].argmax = reinterpret_cast<int*>(r); g[k].entropy = reinterpret_cast<float*>(r + rb);
                g[k].maxprob = reinterpret_cast<float*>(r + 2 * rb); g[k].exit_mask = r + 3 * rb;
                g[k].workspace = workspace; g[k].workspace_bytes = cascade_group_ws(M, d, V); g[k].stream = s;
            }
            ee_status st = gemm_launch(g, n);
            if (st != EE_OK) return st;
            st = cascade_select_launch(q + 3 * rb, reinterpret_cast<const int*>(q), reinterpret_cast<const float*>(q + rb), 4 * rb,
                                       M, k0, n, n_heads, exit_head, token, entropy, rows_in, s);
            if (st != EE_OK) return st;
        }
        return EE_OK;
    }
    unsigned char* p = ws + cascade_head_ws(M, d, V);
    int* t_argmax = reinterpret_cast<int*>(p);
    float* t_entropy = reinterpret_cast<float*>(p + rb);
    float* t_maxprob = reinterpret_cast<float*>(p + 2 * rb);
    unsigned char* t_mask = p + 3 * rb;
    int* idx[2] = {reinterpret_cast<int*>(p + 4 * rb), reinterpret_cast<int*>(p + 5 * rb)};
    int* count = reinterpret_cast<int*>(p + 6 * rb);         // count[0], count[1]: survivors, ping-pong
    for (int k = 0; k < n_heads; ++k) {
        const ee_head& e = heads[k];
        a.h = e.h; a.ld_h = e.ld_h; a.gamma = e.gamma; a.beta = e.beta; a.ln_eps = ln_eps; a.W = e.W;
        a.M = M; a.d = d; a.V = V; a.tau_per_row = nullptr; a.tau = e.tau;
        a.argmax = t_argmax; a.entropy = t_entropy; a.maxprob = t_maxprob; a.exit_mask = t_mask;
        a.workspace = workspace; a.workspace_bytes = cascade_head_ws(M, d, V); a.stream = s;
        a.row_idx = k ? idx[(k - 1) & 1] : nullptr;
        a.m_dev = k ? count + ((k - 1) & 1) : nullptr;
        ee_status st = gemm_launch(&a, 1);
        if (st != EE_OK) return st;
        st = cascade_step_launch(t_mask, t_argmax, t_entropy, a.row_idx, a.m_dev, M, k, k == n_heads - 1, n_heads, exit_head,
                                 token, entropy, idx[k & 1], count + (k & 1), rows_in, s);
        if (st != EE_OK) return st;
    }
    return EE_OK;
}

size_t ee_calibrate_workspace_bytes(int n) { return n < 0 ? 0 : calibrate_workspace_bytes(n); }

ee_status ee_calibrate(const float* entropy, const int* argmax_head, const int* argmax_final, int n, double epsilon,
                       float* tau, int* counts, void* workspace, size_t workspace_bytes_, void* stream) {
    if (n < 0 || !(epsilon >= 0.0 && epsilon <= 1.0)) return EE_ERR_SHAPE;
    if (!tau || !counts || !workspace) return EE_ERR_NULL;
    if (n > 0 && (!entropy || !argmax_head || !argmax_final)) return EE_ERR_NULL;
    if (!aligned(workspace, 256)) return EE_ERR_ALIGN;
    if (workspace_bytes_ < calibrate_workspace_bytes(n)) return EE_ERR_WORKSPACE;
    int device, num_sms;
    const ee_status dev = current_device(&device, &num_sms);
    if (dev != EE_OK) return dev;
    return calibrate_launch(entropy, argmax_head, argmax_final, n, epsilon, tau, counts, workspace,
                            static_cast<cudaStream_t>(stream));
}

ee_status dssd_commit(const int* draft_tok, const unsigned char* draft_exit_mask, const int* verify_tok, int S, int k, int kv,
                      int eos_token, int* out_tok, int capacity, int* seq_len, unsigned char* finished, int* draft_len,
                      int* accept_len, int* next_tok, long long* stats, void* stream) {
    if (S < 0 || k < 1 || k > 32 || kv < k || capacity < 1) return EE_ERR_SHAPE;
    if (S == 0) return EE_OK;
    if (!draft_tok || !verify_tok || !out_tok || !seq_len || !finished || !draft_len || !accept_len || !next_tok || !stats)
        return EE_ERR_NULL;
    int device, num_sms;
    const ee_status dev = current_device(&device, &num_sms);
    if (dev != EE_OK) return dev;
    return dssd_commit_launch(draft_tok, draft_exit_mask, verify_tok, S, k, kv, eos_token, out_tok, capacity, seq_len, finished,
                              draft_len, accept_len, next_tok, stats, static_cast<cudaStream_t>(stream));
}

namespace {
// Scratch of the heads inside a round: the verification pass's single head on S (k + 1) rows, or the K draft heads
// of a step on S rows, whichever needs more.
size_t round_head_ws(int S, int k, int d, int V, int K) {
    const size_t verify = workspace_bytes(S * (k + 1), d, V), draft = ee_exit_head_multi_workspace_bytes(K, S, d, V);
    return verify > draft ? verify : draft;
}
bool round_sizes_ok(int S, int k, int d, int V, int K) {
    return S >= 0 && k >= 1 && k <= 32 && K >= 1 && K <= EE_ROUND_MAX_DRAFT_HEADS && sizes_ok(S * (k + 1), d, V);
}
}  // namespace

size_t dssd_round_multi_workspace_bytes(int S, int k, int d, int V, int n_draft_heads) {
    if (!round_sizes_ok(S, k, d, V, n_draft_heads)) return 0;
    return dssd_round_layout_bytes(S, k, d, n_draft_heads, round_head_ws(S, k, d, V, n_draft_heads));
}

size_t dssd_round_workspace_bytes(int S, int k, int d, int V) { return dssd_round_multi_workspace_bytes(S, k, d, V, 1); }

ee_status dssd_round(const ee_dssd_round_args* a) {
    if (!a) return EE_ERR_NULL;
    if (a->n_draft_heads < 0) return EE_ERR_SHAPE;
    const int K = a->n_draft_heads ? a->n_draft_heads : 1;
    const ee_head* draft = a->n_draft_heads ? a->draft_heads : &a->draft_head;
    if (a->capacity < 1 || !round_sizes_ok(a->S, a->k, a->d, a->V, K)) return EE_ERR_SHAPE;
    if (a->S == 0) return EE_OK;
    if (!a->hidden || !a->last_tok || !a->out_tok || !a->seq_len || !a->finished || !a->stats || !a->draft_len ||
        !a->accept_len || !a->next_tok || !a->workspace || !draft)
        return EE_ERR_NULL;
    for (int h = 0; h < K; ++h)
        if (!draft[h].gamma || !draft[h].beta || !draft[h].W) return EE_ERR_NULL;
    if (!a->verify_head.gamma || !a->verify_head.beta || !a->verify_head.W) return EE_ERR_NULL;
    if (!aligned(a->workspace, 256)) return EE_ERR_ALIGN;
    if (a->workspace_bytes < dssd_round_multi_workspace_bytes(a->S, a->k, a->d, a->V, K)) return EE_ERR_WORKSPACE;
    int device, num_sms;
    const ee_status dev = current_device(&device, &num_sms);
    if (dev != EE_OK) return dev;
    return dssd_round_run(*a, draft, K, round_head_ws(a->S, a->k, a->d, a->V, K));
}

size_t ee_head_kl_workspace_bytes(int M, int d, int V) {
    if (!sizes_ok(M, d, V)) return 0;
    return kl_workspace_bytes(M, d, V);
}

ee_status ee_head_kl(const void* h_head, long long ld_head, const float* gamma_head, const float* beta_head,
                     const void* W_head, const void* h_teacher, long long ld_teacher, const float* gamma_teacher,
                     const float* beta_teacher, const void* W_teacher, float ln_eps, int M, int d, int V,
                     const int* labels, float* kl, float* ce, float* loss, void* workspace, size_t workspace_bytes_,
                     void* stream) {
    if (!sizes_ok(M, d, V)) return EE_ERR_SHAPE;
    if (M == 0) return EE_OK;
    if (!h_head || !gamma_head || !beta_head || !W_head || !h_teacher || !gamma_teacher || !beta_teacher || !W_teacher || !kl ||
        !workspace)
        return EE_ERR_NULL;
    if ((ce != nullptr) != (labels != nullptr)) return EE_ERR_NULL;      // the cross-entropy needs labels, and only it does
    if (ld_head < d || (ld_head % 8) != 0 || ld_teacher < d || (ld_teacher % 8) != 0) return EE_ERR_SHAPE;
    if (!aligned(h_head, 16) || !aligned(W_head, 16) || !aligned(gamma_head, 16) || !aligned(beta_head, 16) ||
        !aligned(h_teacher, 16) || !aligned(W_teacher, 16) || !aligned(gamma_teacher, 16) || !aligned(beta_teacher, 16) ||
        !aligned(workspace, 256))
        return EE_ERR_ALIGN;
    if (workspace_bytes_ < kl_workspace_bytes(M, d, V)) return EE_ERR_WORKSPACE;
    HeadArgs a{}, t{};
    const ee_status dev = current_device(&a.device, &a.num_sms);
    if (dev != EE_OK) return dev;
    a.h = h_head; a.ld_h = ld_head; a.gamma = gamma_head; a.beta = beta_head; a.ln_eps = ln_eps; a.W = W_head;
    a.M = M; a.d = d; a.V = V; a.workspace = workspace; a.workspace_bytes = workspace_bytes_;
    a.stream = static_cast<cudaStream_t>(stream);
    t = a;
    t.h = h_teacher; t.ld_h = ld_teacher; t.gamma = gamma_teacher; t.beta = beta_teacher; t.W = W_teacher;
    return kl_launch(a, t, labels, kl, ce, loss);
}

ee_status ee_selftest_wait_timeout(void* workspace, size_t workspace_bytes_, void* stream) {
    if (!workspace) return EE_ERR_NULL;
    if (!aligned(workspace, 256)) return EE_ERR_ALIGN;
    if (workspace_bytes_ < (size_t)kCtrlBytes) return EE_ERR_WORKSPACE;
    int device, num_sms;
    const ee_status dev = current_device(&device, &num_sms);
    if (dev != EE_OK) return dev;
    return selftest_wait_timeout_launch(workspace, static_cast<cudaStream_t>(stream));
}

int ee_hidden_from_tables(void* user, const int* tokens, int n_rows, int which, void* h_out, void* stream) {
    return hidden_from_tables(static_cast<const ee_hidden_tables*>(user), tokens, n_rows, which, h_out,
                              static_cast<cudaStream_t>(stream));
}

ee_status ee_selftest_read_stream(const void* buffer, size_t bytes, void* workspace, size_t workspace_bytes_, void* stream) {
    if (!buffer || !workspace) return EE_ERR_NULL;
    if (!aligned(buffer, 16) || !aligned(workspace, 256)) return EE_ERR_ALIGN;
    if (bytes < 16384) return EE_ERR_SHAPE;
    if (workspace_bytes_ < (size_t)kCtrlBytes) return EE_ERR_WORKSPACE;
    int device, num_sms;
    const ee_status dev = current_device(&device, &num_sms);
    if (dev != EE_OK) return dev;
    return selftest_read_stream_launch(buffer, bytes, workspace, num_sms, static_cast<cudaStream_t>(stream));
}

ee_status ee_query_async_error(void* workspace, void* stream) {
    if (!workspace) return EE_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned int words[3] = {0, 0, 0};
    if (cudaMemcpyAsync(words, workspace, sizeof(words), cudaMemcpyDeviceToHost, s) != cudaSuccess) return EE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return EE_ERR_CUDA;
    if (words[1] == 0) return EE_OK;
    if (cudaMemsetAsync(static_cast<unsigned char*>(workspace) + 4, 0, 8, s) != cudaSuccess) return EE_ERR_CUDA;
    return EE_ERR_TIMEOUT;
}

}  // extern "C"
