// Commit step of one DSSD round (paper section 4.3.1) for S sequences that keep their committed tokens in a
// buffer on the device: draft length with the three stop conditions (buffer limit, end-of-sequence token, first
// slot without confidence), accepted prefix, the full model's token after it, append, finished flags, and the
// round's statistics.  One warp per sequence, lane j = draft slot j (k <= 32).  Integer work: ballots, ffs.
#include "common.cuh"
#include "kernels.h"

namespace ee {

namespace {

__global__ void __launch_bounds__(128) dssd_commit_kernel(const int* draft_tok,
                                                          const unsigned char* draft_exit_mask,
                                                          const int* verify_tok, int S, int k, int kv, int eos,
                                                          int* out_tok, int cap, int* seq_len,
                                                          unsigned char* finished,
                                                          int* draft_len, int* accept_len,
                                                          int* next_tok,
                                                          unsigned long long* stats) {
    const int s = blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    launch_dependents();
    if (s >= S) return;
    grid_dependency_wait();                              // tokens, masks and the sequences' state come from earlier kernels
    // Lane 0 rewrites finished[s] and seq_len[s] at the end: every lane reads both here, and the warp meets again
    // before those stores, so no lane can see this round's values.
    const bool was_finished = ld_dep(finished + s) != 0;
    const int have = ld_dep(seq_len + s);
    __syncwarp();
    if (was_finished) {                                  // a finished sequence takes no part in the round
        if (lane == 0) { draft_len[s] = 0; accept_len[s] = 0; next_tok[s] = -1; }
        return;
    }
    const bool in = lane < k;
    const int d = in ? ld_dep(draft_tok + (size_t)s * k + lane) : 0;
    const int v = in ? ld_dep(verify_tok + (size_t)s * kv + lane) : 0;
    const bool conf = in && (draft_exit_mask == nullptr || ld_dep(draft_exit_mask + (size_t)s * k + lane) != 0);
    const unsigned int stop_b = __ballot_sync(0xffffffffu, in && !conf);               // slots the head is not sure of
    const unsigned int eos_b = __ballot_sync(0xffffffffu, in && eos >= 0 && d == eos);   // end-of-sequence drafted
    const unsigned int mis_b = __ballot_sync(0xffffffffu, in && d != v);
    int n = stop_b ? __ffs(stop_b) - 1 : k;                                           // stops (i) and (iii)
    if (eos_b && __ffs(eos_b) <= n) n = __ffs(eos_b);                                 // stop (ii): that token is the last drafted
    const int first_mis = mis_b ? __ffs(mis_b) - 1 : k;
    const int a = min(first_mis, n);
    const bool ended = a > 0 && eos >= 0 && __shfl_sync(0xffffffffu, d, a - 1) == eos;
    const int nxt = (!ended && a < kv) ? ld_dep(verify_tok + (size_t)s * kv + a) : -1;
    const int want = a + ((!ended && a < kv) ? 1 : 0);
    const int count = min(want, cap - have);
    int* row = out_tok + (size_t)s * cap + have;
    if (lane < count) row[lane] = lane < a ? d : nxt;     // count <= k + 1 <= 33: lane 31 may have one more below
    __syncwarp();
    if (lane == 0) {
        if (count == 33) row[32] = nxt;
        const bool eos_committed = eos >= 0 && ((ended && count >= a) || (nxt == eos && count == want && want > a));
        seq_len[s] = have + count;
        if (eos_committed || have + count >= cap) finished[s] = 1;
        draft_len[s] = n;
        accept_len[s] = a;
        next_tok[s] = nxt;
        atomicAdd(&stats[0], (unsigned long long)n);
        atomicAdd(&stats[1], (unsigned long long)a);
        atomicAdd(&stats[2], (unsigned long long)count);
        atomicAdd(&stats[3], 1ull);
    }
}

}  // namespace

ee_status dssd_commit_launch(const int* draft_tok, const unsigned char* draft_exit_mask, const int* verify_tok, int S, int k,
                             int kv, int eos, int* out_tok, int cap, int* seq_len, unsigned char* finished, int* draft_len,
                             int* accept_len, int* next_tok, long long* stats, cudaStream_t stream) {
    if (S == 0) return EE_OK;
    return launch_pdl(dssd_commit_kernel, (S + 3) / 4, 128, 0, stream, draft_tok, draft_exit_mask, verify_tok, S, k, kv, eos,
                      out_tok, cap, seq_len, finished, draft_len, accept_len, next_tok,
                      reinterpret_cast<unsigned long long*>(stats)) == cudaSuccess
               ? EE_OK
               : EE_ERR_CUDA;
}

}  // namespace ee
