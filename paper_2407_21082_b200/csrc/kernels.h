// Internal launch interface between the C-ABI layer (api.cu) and the kernels.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

#include "eexit.h"

namespace ee {

constexpr int kMaxDevices = 64;

struct HeadArgs {
    const void* h;
    long long ld_h;
    const float* gamma;
    const float* beta;
    float ln_eps;
    const void* W;
    int M, d, V;
    const float* tau_per_row;
    float tau;
    int* argmax;
    float* entropy;
    float* maxprob;
    unsigned char* exit_mask;
    void* workspace;
    size_t workspace_bytes;
    cudaStream_t stream;
    int device;       // current device ordinal
    int num_sms;      // its multiprocessor count
    // Optional (tensor-core path, one head per launch): evaluate the rows h[row_idx[j]], j < *m_dev, instead of
    // rows 0 .. M-1; output row j belongs to input row row_idx[j], output rows at and beyond *m_dev are
    // meaningless.  Either may be NULL (identity / M).  Both are device pointers read after the stream's
    // earlier kernels have finished.
    const int* row_idx;
    const int* m_dev;
    // Optional (tensor-core path): fp32 [M], the difference between the two largest probabilities of each row.
    float* top2gap;
};

// ---- streaming kernel (fused LayerNorm + split-V mma.sync GEMV + last-CTA merge; up to four heads per launch) ----
constexpr int kStreamMaxCtas = 256;        // upper bound on the grid, used for workspace sizing
constexpr int kStreamMaxRows = 32;         // rows per launch (slab)
constexpr int kStreamMaxHeads = 4;
int stream_slab_rows(int d, int n_heads);  // rows one launch can take for this d (0 if d does not fit)
size_t stream_workspace_bytes(int n_heads);
ee_status stream_launch(const HeadArgs* heads, int n_heads);

// ---- skinny tensor-core kernel (one launch for up to four heads, weights as the MMA's M operand,
//      1 <= M <= 64, d % 64 == 0) ----
constexpr int kSkinnyMaxRows = 64;
constexpr int kSkinnyMaxHeads = 4;
bool skinny_supports(int M, int d);
size_t skinny_workspace_bytes(int n_heads);
// heads[0 .. n_heads) share M, d, V, ln_eps, workspace, stream and device; each has its own h, LayerNorm
// parameters, W, thresholds and outputs.
ee_status skinny_launch(const HeadArgs* heads, int n_heads);

// ---- tensor-core path (LayerNorm kernel, TMA + tcgen05 GEMM with fused statistics, merge): three launches
//      for up to four heads that share M, d, V, ln_eps, workspace, stream and device ----
constexpr int kGemmLaunchMaxHeads = 4;
int gemm_tile_n(int M, int V, int n_heads, int num_sms);   // vocabulary tile width used for M rows on num_sms SMs
size_t gemm_workspace_bytes(int M, int d, int V, int n_heads);
ee_status gemm_launch(const HeadArgs* heads, int n_heads);
// The same in two steps, for calls that are repeated: gemm_plan works out everything but the launches (tensor maps,
// tile width, launch shapes, instantiations) into `storage` (kGemmPlanBytes bytes, 8-byte aligned, plain data),
// gemm_run launches from it on `stream`.
constexpr size_t kGemmPlanBytes = 2048;
ee_status gemm_plan(const HeadArgs* heads, int n_heads, void* storage);
ee_status gemm_run(const void* storage, cudaStream_t stream);
int gemm_launches(int M, int n_heads);     // kernels one gemm_launch call starts

// ---- compaction and DSSD accept ----
ee_status compact_launch(const unsigned char* exit_mask, const void* h, long long ld_h, int M, int d,
                         int* kept_idx, int* kept_count, void* h_out, cudaStream_t stream);
ee_status accept_launch(const int* draft_tok, const unsigned char* draft_exit_mask, const int* verify_tok,
                        int S, int k, int kv, int* draft_len, int* accept_len, int* next_tok,
                        cudaStream_t stream);

ee_status compact_accept_launch(const unsigned char* exit_mask, const void* h, long long ld_h, int M, int d,
                                int* kept_idx, int* kept_count, void* h_out, const int* draft_tok,
                                const unsigned char* draft_exit_mask, const int* verify_tok, int S, int k, int kv,
                                int* draft_len, int* accept_len, int* next_tok, cudaStream_t stream);

// ---- calibration of a head's threshold (radix sort of the calibration tokens by entropy, scan, selection) ----
size_t calibrate_workspace_bytes(int n);
int calibrate_launches(int n);
ee_status calibrate_launch(const float* entropy, const int* argmax_head, const int* argmax_final, int n, double epsilon,
                           float* tau, int* counts, void* workspace, cudaStream_t stream);

// ---- KL divergence of a head's distribution from the teacher's, per token and mean (both logit sets fused) ----
size_t kl_workspace_bytes(int M, int d, int V);
ee_status kl_launch(const HeadArgs& head, const HeadArgs& teacher, const int* labels, float* kl, float* ce, float* loss);

// ---- commit step of a DSSD round (k <= 32) ----
ee_status dssd_commit_launch(const int* draft_tok, const unsigned char* draft_exit_mask, const int* verify_tok, int S, int k,
                             int kv, int eos, int* out_tok, int cap, int* seq_len, unsigned char* finished, int* draft_len,
                             int* accept_len, int* next_tok, long long* stats, cudaStream_t stream);

// ---- a whole DSSD round driven from the host (drafting steps, verification pass, commit) ----
size_t dssd_round_layout_bytes(int S, int k, int d, int n_draft_heads, size_t head_ws_bytes);
ee_status dssd_round_run(const ee_dssd_round_args& a, const ee_head* draft_heads, int n_draft_heads, size_t head_ws_bytes);

// ---- diagnostic: a bounded wait that is made to give up ----
int hidden_from_tables(const ee_hidden_tables* m, const int* tokens, int n_rows, int which, void* h_out, cudaStream_t stream);
ee_status selftest_wait_timeout_launch(void* workspace, cudaStream_t stream);
ee_status selftest_read_stream_launch(const void* src, size_t bytes, void* workspace, int num_sms, cudaStream_t stream);

// ---- one step of the cascade of heads: rows answered by head k are recorded, the others move on ----
int cascade_select_max_rows();
ee_status cascade_select_launch(const unsigned char* mask0, const int* argmax0, const float* entropy0, size_t stride, int M,
                                int k0, int n, int n_heads, int* exit_head, int* token, float* entropy_out, int* rows_in,
                                cudaStream_t stream);
ee_status cascade_step_launch(const unsigned char* exit_mask, const int* argmax, const float* entropy,
                              const int* idx_in, const int* m_in, int M, int k, int is_last, int n_heads,
                              int* exit_head, int* token, float* entropy_out, int* idx_out, int* m_out, int* rows_in,
                              cudaStream_t stream);

}  // namespace ee
