// One step of the inference-time cascade of exit heads (paper section 3.4.2): after head k has been evaluated
// on the rows that no earlier head answered, the rows it answers are recorded under their position in the
// batch and the others are listed, in order, for head k + 1.  Integer work: ballots, popcounts.
#include "common.cuh"
#include "kernels.h"

namespace ee {

namespace {

constexpr int kStepThreads = 256;
constexpr int kStepRows = 32;             // one ballot's worth of rows per CTA

// Row j < m of this step is row idx_in[j] of the batch (j itself when idx_in is NULL).  CTA b owns rows
// [32 b, 32 b + 32): it counts the survivors before its rows itself from the mask (L2-resident), so no CTA
// waits for another.  Rows the last head leaves unanswered are marked with exit_head = n_heads.
__global__ void __launch_bounds__(kStepThreads) cascade_step_kernel(const unsigned char* exit_mask,
                                                                    const int* argmax,
                                                                    const float* entropy,
                                                                    const int* idx_in,
                                                                    const int* m_in, int M, int k,
                                                                    int is_last, int n_heads,
                                                                    int* exit_head, int* token,
                                                                    float* entropy_out,
                                                                    int* idx_out, int* m_out,
                                                                    int* rows_in) {
    __shared__ int s_warp_cnt[kStepThreads / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    launch_dependents();
    grid_dependency_wait();
    const int m = m_in ? min(max(ld_dep(m_in), 0), M) : M;
    const int row0 = blockIdx.x * kStepRows;
    if (blockIdx.x == 0 && threadIdx.x == 0) rows_in[k] = m;
    int cnt = zero_bytes_share(exit_mask, min(row0, m), threadIdx.x, kStepThreads);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0) s_warp_cnt[warp] = cnt;
    __syncthreads();
    if (warp != 0) return;
    int base = 0;
#pragma unroll
    for (int w = 0; w < kStepThreads / 32; ++w) base += s_warp_cnt[w];
    const int j = row0 + lane;
    const bool in = j < m;
    const bool answered = in && ld_dep(exit_mask + (in ? j : 0)) != 0;
    const bool moves_on = in && !answered;
    const unsigned int ballot = __ballot_sync(0xffffffffu, moves_on);
    const int orig = in ? (idx_in ? ld_dep(idx_in + j) : j) : 0;
    if (answered) {
        exit_head[orig] = k;
        token[orig] = ld_dep(argmax + j);
        entropy_out[orig] = ld_dep(entropy + j);
    }
    if (moves_on) {
        if (is_last) {
            exit_head[orig] = n_heads;
            token[orig] = -1;
            entropy_out[orig] = __int_as_float(0x7fc00000);          // no head answered: NaN
        } else {
            idx_out[base + __popc(ballot & ((1u << lane) - 1u))] = orig;
        }
    }
    // the CTA that holds the last row of the step knows the number of survivors
    if (lane == 0 && row0 < max(m, 1) && row0 + kStepRows >= m) *m_out = base + __popc(ballot);
}

// Small batches (M <= kSelectThreads): up to four heads have been evaluated on EVERY row of the batch (a head's
// weights are streamed once whatever the number of rows), and this kernel walks them in order for each row: a
// row still open takes the first head of the group that answers it.  Between groups the state of a row is its
// exit_head entry (n_heads = still open).  One CTA of M threads rounded up to whole warps, thread = row; head k
// of the group has its results at argmax0 / entropy0 / mask0 + k * stride bytes.
constexpr int kSelectThreads = 1024;

__global__ void __launch_bounds__(kSelectThreads) cascade_select_kernel(const unsigned char* mask0,
                                                                        const unsigned char* argmax0,
                                                                        const unsigned char* entropy0,
                                                                        size_t stride, int M, int k0, int n, int n_heads,
                                                                        int* exit_head, int* token,
                                                                        float* entropy_out,
                                                                        int* rows_in) {
    launch_dependents();
    grid_dependency_wait();
    const int i = threadIdx.x;
    const bool in = i < M;
    bool open = in && (k0 == 0 || ld_dep(exit_head + (in ? i : 0)) == n_heads);
    for (int k = 0; k < n; ++k) {
        const int cnt = __syncthreads_count(open);
        if (i == 0) rows_in[k0 + k] = cnt;
        if (open && ld_dep(mask0 + k * stride + i) != 0) {
            exit_head[i] = k0 + k;
            token[i] = ld_dep(reinterpret_cast<const int*>(argmax0 + k * stride) + i);
            entropy_out[i] = ld_dep(reinterpret_cast<const float*>(entropy0 + k * stride) + i);
            open = false;
        }
    }
    if (open && k0 == 0) {                                              // stays so unless a later group answers
        exit_head[i] = n_heads;
        token[i] = -1;
        entropy_out[i] = __int_as_float(0x7fc00000);
    }
}

}  // namespace

int cascade_select_max_rows() { return kSelectThreads; }

ee_status cascade_select_launch(const unsigned char* mask0, const int* argmax0, const float* entropy0, size_t stride, int M,
                                int k0, int n, int n_heads, int* exit_head, int* token, float* entropy_out, int* rows_in,
                                cudaStream_t stream) {
    if (M > kSelectThreads) return EE_ERR_SHAPE;
    return launch_pdl(cascade_select_kernel, 1, (M + 31) / 32 * 32, 0, stream, mask0, reinterpret_cast<const unsigned char*>(argmax0),
                      reinterpret_cast<const unsigned char*>(entropy0), stride, M, k0, n, n_heads, exit_head, token,
                      entropy_out, rows_in) == cudaSuccess
               ? EE_OK
               : EE_ERR_CUDA;
}

ee_status cascade_step_launch(const unsigned char* exit_mask, const int* argmax, const float* entropy,
                              const int* idx_in, const int* m_in, int M, int k, int is_last, int n_heads,
                              int* exit_head, int* token, float* entropy_out, int* idx_out, int* m_out, int* rows_in,
                              cudaStream_t stream) {
    const int grid = (M + kStepRows - 1) / kStepRows;
    return launch_pdl(cascade_step_kernel, grid, kStepThreads, 0, stream, exit_mask, argmax, entropy, idx_in, m_in, M, k,
                      is_last, n_heads, exit_head, token, entropy_out, idx_out, m_out, rows_in) == cudaSuccess
               ? EE_OK
               : EE_ERR_CUDA;
}

}  // namespace ee
