// Order-preserving compaction of the rows that did not exit (with the gather of their hidden states),
// and the DSSD draft-length / accepted-prefix count.  Integer work: ballots, popcounts, first-set-bit.
#include "common.cuh"
#include "kernels.h"

namespace ee {

namespace {

constexpr int kCompactThreads = 256;
constexpr int kRowsPerCta = 32;           // one ballot's worth of rows per CTA

// CTA b owns rows [32b, 32b + 32).  Its output offset is the number of surviving rows before 32b, which it
// counts itself from the mask (M bytes at most, L2-resident, sixteen bytes per load), so no CTA waits for another
// and the call needs no scratch memory; over all CTAs that is M^2 / 1024 loads -- four megabytes of L2 traffic for
// 16 K rows, 160 MB for 100 K rows.
__device__ __forceinline__ void compact_body(int cta, const unsigned char* exit_mask,
                                             const __nv_bfloat16* h, long long ld_h, int M, int d,
                                             int* kept_idx, int* kept_count,
                                             __nv_bfloat16* h_out) {
    __shared__ int s_warp_cnt[kCompactThreads / 32];
    __shared__ int s_src[kRowsPerCta];
    __shared__ int s_base, s_n;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row0 = cta * kRowsPerCta;

    int cnt = zero_bytes_share(exit_mask, row0, threadIdx.x, kCompactThreads);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0) s_warp_cnt[warp] = cnt;
    __syncthreads();
    if (warp == 0) {
        int base = 0;
#pragma unroll
        for (int w = 0; w < kCompactThreads / 32; ++w) base += s_warp_cnt[w];
        const int row = row0 + lane;
        const bool keep = (row < M) && (ld_dep(exit_mask + min(row, M - 1)) == 0);
        const unsigned int ballot = __ballot_sync(0xffffffffu, keep);
        const int rank = __popc(ballot & ((1u << lane) - 1u));
        if (keep) {
            kept_idx[base + rank] = row;
            s_src[rank] = row;
        }
        if (lane == 0) {
            s_base = base;
            s_n = __popc(ballot);
            if (row0 + kRowsPerCta >= M) *kept_count = base + __popc(ballot);     // the last CTA knows the total
        }
    }
    __syncthreads();
    if (h_out == nullptr) return;
    const int nvec = d >> 3;
    for (int r = warp; r < s_n; r += kCompactThreads / 32) {
        const uint4* src = reinterpret_cast<const uint4*>(h + (size_t)s_src[r] * ld_h);
        uint4* dst = reinterpret_cast<uint4*>(h_out + (size_t)(s_base + r) * d);
        // Four loads in flight per lane before the first store: source and destination may alias as far as the
        // compiler knows, so it would otherwise finish every store before it starts the next load.
        for (int c = lane; c < nvec; c += 128) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (c + 32 * u < nvec) v[u] = ld_dep(src + c + 32 * u);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (c + 32 * u < nvec) dst[c + 32 * u] = v[u];
        }
    }
}

__global__ void __launch_bounds__(kCompactThreads) compact_kernel(const unsigned char* exit_mask,
                                                                  const __nv_bfloat16* h, long long ld_h,
                                                                  int M, int d, int* kept_idx,
                                                                  int* kept_count,
                                                                  __nv_bfloat16* h_out) {
    launch_dependents();
    grid_dependency_wait();                              // the mask and h come from earlier kernels of the stream
    compact_body(blockIdx.x, exit_mask, h, ld_h, M, d, kept_idx, kept_count, h_out);
}

// One warp per sequence s; lane j looks at draft slot j (slots beyond 32 in further rounds).
__device__ __forceinline__ void accept_body(int s, int lane, const int* draft_tok,
                                            const unsigned char* draft_exit_mask,
                                            const int* verify_tok, int k, int kv,
                                            int* draft_len, int* accept_len,
                                            int* next_tok) {
    int n = k;             // first slot that is not confident (draft length)
    int first_mis = k;     // first slot whose drafted token differs from the verifier's
    for (int base = 0; base < k; base += 32) {
        const int j = base + lane;
        const bool in = j < k;
        const bool conf = in && (draft_exit_mask == nullptr || ld_dep(draft_exit_mask + (size_t)s * k + j) != 0);
        const bool same = in && (ld_dep(draft_tok + (size_t)s * k + j) == ld_dep(verify_tok + (size_t)s * kv + j));
        const unsigned int stop_b = __ballot_sync(0xffffffffu, in && !conf);
        const unsigned int mis_b = __ballot_sync(0xffffffffu, in && !same);
        if (first_mis == k && mis_b) first_mis = base + __ffs(mis_b) - 1;
        if (stop_b) { n = base + __ffs(stop_b) - 1; break; }     // slots after the stop are never drafted
    }
    const int a = first_mis < n ? first_mis : n;
    if (lane == 0) {
        draft_len[s] = n;
        accept_len[s] = a;
        next_tok[s] = (a < kv) ? ld_dep(verify_tok + (size_t)s * kv + a) : -1;
    }
}

__global__ void __launch_bounds__(128) accept_kernel(const int* draft_tok,
                                                     const unsigned char* draft_exit_mask,
                                                     const int* verify_tok, int S, int k, int kv,
                                                     int* draft_len, int* accept_len,
                                                     int* next_tok) {
    const int s = blockIdx.x * 4 + (threadIdx.x >> 5);
    launch_dependents();
    if (s >= S) return;
    grid_dependency_wait();                              // tokens and mask come from earlier kernels of the stream
    accept_body(s, threadIdx.x & 31, draft_tok, draft_exit_mask, verify_tok, k, kv, draft_len, accept_len, next_tok);
}

// Both in one launch: the first n_compact CTAs compact, the others take eight sequences each.  The two parts
// read the same head outputs and write disjoint results, so they need no order between them.
struct TailArgs {
    const unsigned char* exit_mask;
    const __nv_bfloat16* h;
    long long ld_h;
    int M, d;
    int* kept_idx;
    int* kept_count;
    __nv_bfloat16* h_out;
    const int* draft_tok;
    const unsigned char* draft_exit_mask;
    const int* verify_tok;
    int S, k, kv;
    int* draft_len;
    int* accept_len;
    int* next_tok;
    int n_compact;
};

__global__ void __launch_bounds__(kCompactThreads) compact_accept_kernel(const __grid_constant__ TailArgs a) {
    launch_dependents();
    grid_dependency_wait();
    if ((int)blockIdx.x < a.n_compact) {
        compact_body(blockIdx.x, a.exit_mask, a.h, a.ld_h, a.M, a.d, a.kept_idx, a.kept_count, a.h_out);
    } else {
        const int s = ((int)blockIdx.x - a.n_compact) * (kCompactThreads / 32) + (threadIdx.x >> 5);
        if (s < a.S)
            accept_body(s, threadIdx.x & 31, a.draft_tok, a.draft_exit_mask, a.verify_tok, a.k, a.kv, a.draft_len,
                        a.accept_len, a.next_tok);
    }
}

}  // namespace

ee_status compact_launch(const unsigned char* exit_mask, const void* h, long long ld_h, int M, int d, int* kept_idx,
                         int* kept_count, void* h_out, cudaStream_t stream) {
    if (M == 0) return cudaMemsetAsync(kept_count, 0, sizeof(int), stream) == cudaSuccess ? EE_OK : EE_ERR_CUDA;
    const int grid = (M + kRowsPerCta - 1) / kRowsPerCta;
    return launch_pdl(compact_kernel, grid, kCompactThreads, 0, stream, exit_mask, static_cast<const __nv_bfloat16*>(h),
                      ld_h, M, d, kept_idx, kept_count, static_cast<__nv_bfloat16*>(h_out)) == cudaSuccess
               ? EE_OK
               : EE_ERR_CUDA;
}

ee_status accept_launch(const int* draft_tok, const unsigned char* draft_exit_mask, const int* verify_tok, int S, int k,
                        int kv, int* draft_len, int* accept_len, int* next_tok, cudaStream_t stream) {
    if (S == 0) return EE_OK;
    return launch_pdl(accept_kernel, (S + 3) / 4, 128, 0, stream, draft_tok, draft_exit_mask, verify_tok, S, k, kv,
                      draft_len, accept_len, next_tok) == cudaSuccess
               ? EE_OK
               : EE_ERR_CUDA;
}

ee_status compact_accept_launch(const unsigned char* exit_mask, const void* h, long long ld_h, int M, int d,
                                int* kept_idx, int* kept_count, void* h_out, const int* draft_tok,
                                const unsigned char* draft_exit_mask, const int* verify_tok, int S, int k, int kv,
                                int* draft_len, int* accept_len, int* next_tok, cudaStream_t stream) {
    if (M == 0 || S == 0) {      // one part is empty: the plain launches handle it
        const ee_status st = compact_launch(exit_mask, h, ld_h, M, d, kept_idx, kept_count, h_out, stream);
        if (st != EE_OK) return st;
        return accept_launch(draft_tok, draft_exit_mask, verify_tok, S, k, kv, draft_len, accept_len, next_tok, stream);
    }
    TailArgs a;
    a.exit_mask = exit_mask; a.h = static_cast<const __nv_bfloat16*>(h); a.ld_h = ld_h; a.M = M; a.d = d;
    a.kept_idx = kept_idx; a.kept_count = kept_count; a.h_out = static_cast<__nv_bfloat16*>(h_out);
    a.draft_tok = draft_tok; a.draft_exit_mask = draft_exit_mask; a.verify_tok = verify_tok;
    a.S = S; a.k = k; a.kv = kv; a.draft_len = draft_len; a.accept_len = accept_len; a.next_tok = next_tok;
    a.n_compact = (M + kRowsPerCta - 1) / kRowsPerCta;
    const int per_cta = kCompactThreads / 32;
    const int grid = a.n_compact + (S + per_cta - 1) / per_cta;
    return launch_pdl(compact_accept_kernel, grid, kCompactThreads, 0, stream, a) == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace ee
