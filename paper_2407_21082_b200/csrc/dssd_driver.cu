// One whole DSSD round (paper section 4.3.1) for S sequences, driven from the host without any synchronisation:
// k drafting steps with the draft head, one verification pass with the full model's head over the k draft
// positions plus a bonus position, then the commit.  The hidden states come from the caller's model through a
// callback that is handed device buffers and the stream; everything between the heads (recording the drafted
// tokens, building the verifier's inputs, the sequences' state) stays on the device.
#include <math.h>

#include "common.cuh"
#include "kernels.h"

namespace ee {

namespace {

// After drafting step j: for every sequence the first of the K draft heads (shallowest first) that is confident
// supplies token and confidence of column j of the draft buffers, and the token becomes the next step's input.
// Where no head is confident the slot is marked so (the draft ends there) and carries the deepest head's token,
// which only feeds the later, ignored steps.  Head h's results start h * stride bytes after argmax0 / mask0.
__global__ void __launch_bounds__(256) record_draft_kernel(const unsigned char* argmax0, const unsigned char* mask0, size_t stride,
                                                           int n_heads, int S, int j, int k, int* draft_tok,
                                                           unsigned char* draft_mask, int* draft_head, int* cur_tok) {
    launch_dependents();
    const int s = blockIdx.x * 256 + threadIdx.x;
    if (s >= S) return;
    grid_dependency_wait();
    int head = n_heads;
    for (int h = n_heads - 1; h >= 0; --h)
        if (ld_dep(mask0 + h * stride + s) != 0) head = h;
    const int from = head < n_heads ? head : n_heads - 1;
    const int t = ld_dep(reinterpret_cast<const int*>(argmax0 + from * stride) + s);
    draft_tok[(size_t)s * k + j] = t;
    draft_mask[(size_t)s * k + j] = head < n_heads ? 1 : 0;
    draft_head[(size_t)s * k + j] = head;
    cur_tok[s] = t;
}

// After the commit: which head supplied the positions inside each draft (sequences that took part only).
__global__ void __launch_bounds__(256) head_use_kernel(const int* draft_head, const int* draft_len, const unsigned char* was_finished,
                                                       int S, int k, int n_heads, unsigned long long* head_use) {
    launch_dependents();
    const int s = blockIdx.x * 256 + threadIdx.x;
    if (s >= S) return;
    grid_dependency_wait();
    if (ld_dep(was_finished + s)) return;
    const int n = min(ld_dep(draft_len + s), k);
    for (int j = 0; j < n; ++j) {
        const int h = ld_dep(draft_head + (size_t)s * k + j);
        if (h >= 0 && h < n_heads) atomicAdd(&head_use[h], 1ull);
    }
}

// The verifier's row (s, j) reads the token before position j: the last committed token for j = 0, the token
// drafted at j - 1 after that (j = k is the bonus row).
__global__ void __launch_bounds__(256) verify_inputs_kernel(const int* last_tok,
                                                            const int* draft_tok, int S, int k,
                                                            int* prev_all) {
    launch_dependents();
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= S * (k + 1)) return;
    grid_dependency_wait();
    const int s = i / (k + 1), j = i - s * (k + 1);
    prev_all[i] = j == 0 ? ld_dep(last_tok + s) : ld_dep(draft_tok + (size_t)s * k + j - 1);
}

// Sequences that took part in the round continue from their last committed token.
__global__ void __launch_bounds__(256) last_token_kernel(const int* out_tok, int cap,
                                                         const int* seq_len,
                                                         const unsigned char* was_finished, int S,
                                                         int* last_tok) {
    launch_dependents();
    const int s = blockIdx.x * 256 + threadIdx.x;
    if (s >= S) return;
    grid_dependency_wait();
    const int len = ld_dep(seq_len + s);
    if (!ld_dep(was_finished + s) && len > 0) last_tok[s] = ld_dep(out_tok + (size_t)s * cap + len - 1);
}

__global__ void __launch_bounds__(256) copy_bytes_kernel(const unsigned char* src, int n,
                                                         unsigned char* dst, const int* src_i,
                                                         int* dst_i) {
    launch_dependents();
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    grid_dependency_wait();
    dst[i] = ld_dep(src + i);
    dst_i[i] = ld_dep(src_i + i);
}

struct Layout {
    size_t head_ws, h, outs, draft_tok, draft_mask, draft_head, prev_all, cur_tok, was_finished, total;
    size_t out_stride_draft;      // bytes between the result blocks of consecutive draft heads
};

// K: number of draft heads.  The hidden-state buffer holds the K drafting layers' rows of a step, or the
// verification pass's rows, whichever is more; likewise the result arrays.
Layout layout(int S, int k, int d, int K, size_t head_ws_bytes) {
    Layout L;
    const size_t rows_v = (size_t)S * (k + 1), rows_d = (size_t)S * K;
    size_t o = 0;
    auto take = [&](size_t bytes) { const size_t at = o; o += align_up(bytes, 256); return at; };
    L.head_ws = take(head_ws_bytes);
    L.h = take((rows_v > rows_d ? rows_v : rows_d) * d * 2);
    L.out_stride_draft = 4 * align_up((size_t)S * 4, 256);
    const size_t outs_v = 4 * align_up(rows_v * 4, 256), outs_d = (size_t)K * L.out_stride_draft;
    L.outs = take(outs_v > outs_d ? outs_v : outs_d);
    L.draft_tok = take((size_t)S * k * 4);
    L.draft_mask = take((size_t)S * k);
    L.draft_head = take((size_t)S * k * 4);
    L.prev_all = take(rows_v * 4);
    L.cur_tok = take((size_t)S * 4);
    L.was_finished = take((size_t)S);
    L.total = o;
    return L;
}

}  // namespace

size_t dssd_round_layout_bytes(int S, int k, int d, int K, size_t head_ws_bytes) { return layout(S, k, d, K, head_ws_bytes).total; }

ee_status dssd_round_run(const ee_dssd_round_args& a, const ee_head* draft_heads, int K, size_t head_ws_bytes) {
    const int S = a.S, k = a.k, d = a.d, V = a.V;
    const Layout L = layout(S, k, d, K, head_ws_bytes);
    unsigned char* ws = static_cast<unsigned char*>(a.workspace);
    cudaStream_t s = static_cast<cudaStream_t>(a.stream);
    const size_t rows = (size_t)S * (k + 1);
    unsigned char* h = ws + L.h;
    const size_t ob = align_up(rows * 4, 256), ob_s = align_up((size_t)S * 4, 256);
    int* t_argmax = reinterpret_cast<int*>(ws + L.outs);
    float* t_entropy = reinterpret_cast<float*>(ws + L.outs + ob);
    float* t_maxprob = reinterpret_cast<float*>(ws + L.outs + 2 * ob);
    unsigned char* t_mask = ws + L.outs + 3 * ob;
    int* draft_tok = reinterpret_cast<int*>(ws + L.draft_tok);
    unsigned char* draft_mask = ws + L.draft_mask;
    int* draft_head = reinterpret_cast<int*>(ws + L.draft_head);
    int* prev_all = reinterpret_cast<int*>(ws + L.prev_all);
    int* cur_tok = reinterpret_cast<int*>(ws + L.cur_tok);
    unsigned char* was_finished = ws + L.was_finished;
    const int gs = (S + 255) / 256;

    // the K draft heads on the K drafting layers' rows of a step; head hd's results at outs + hd * out_stride_draft
    ee_head step_heads[EE_ROUND_MAX_DRAFT_HEADS];
    for (int hd = 0; hd < K; ++hd) {
        unsigned char* r = ws + L.outs + (size_t)hd * L.out_stride_draft;
        step_heads[hd] = draft_heads[hd];
        step_heads[hd].h = h + (size_t)hd * S * d * 2;
        step_heads[hd].ld_h = d;
        step_heads[hd].tau_per_row = nullptr;
        step_heads[hd].argmax = reinterpret_cast<int*>(r);
        step_heads[hd].entropy = reinterpret_cast<float*>(r + ob_s);
        step_heads[hd].maxprob = reinterpret_cast<float*>(r + 2 * ob_s);
        step_heads[hd].exit_mask = r + 3 * ob_s;
    }
    // the round's inputs: who is still running, and every sequence's last committed token
    if (launch_pdl(copy_bytes_kernel, gs, 256, 0, s, (const unsigned char*)a.finished, S, was_finished, (const int*)a.last_tok,
                   cur_tok) != cudaSuccess)
        return EE_ERR_CUDA;
    for (int j = 0; j < k; ++j) {
        if (a.hidden_all_layers) {                        // one forward pass of the caller's model for all K layers
            if (a.hidden(a.hidden_user, cur_tok, S, -1, h, a.stream) != 0) return EE_ERR_CUDA;
        } else {
            for (int hd = 0; hd < K; ++hd)
                if (a.hidden(a.hidden_user, cur_tok, S, hd, h + (size_t)hd * S * d * 2, a.stream) != 0) return EE_ERR_CUDA;
        }
        ee_status st = ee_exit_head_multi(step_heads, K, a.ln_eps, S, d, V, ws + L.head_ws, head_ws_bytes, a.stream);
        if (st != EE_OK) return st;
        if (launch_pdl(record_draft_kernel, gs, 256, 0, s, (const unsigned char*)(ws + L.outs),
                       (const unsigned char*)(ws + L.outs + 3 * ob_s), L.out_stride_draft, K, S, j, k, draft_tok, draft_mask,
                       draft_head, cur_tok) != cudaSuccess)
            return EE_ERR_CUDA;
    }
    if (launch_pdl(verify_inputs_kernel, (int)((rows + 255) / 256), 256, 0, s, (const int*)a.last_tok, (const int*)draft_tok, S, k,
                   prev_all) != cudaSuccess)
        return EE_ERR_CUDA;
    if (a.hidden(a.hidden_user, prev_all, (int)rows, K, h, a.stream) != 0) return EE_ERR_CUDA;
    ee_status st = ee_exit_head(h, d, a.verify_head.gamma, a.verify_head.beta, a.ln_eps, a.verify_head.W, (int)rows, d, V, nullptr,
                                HUGE_VALF, t_argmax, t_entropy, t_maxprob, t_mask, ws + L.head_ws, head_ws_bytes, a.stream);
    if (st != EE_OK) return st;
    st = dssd_commit_launch(draft_tok, draft_mask, t_argmax, S, k, k + 1, a.eos_token, a.out_tok, a.capacity, a.seq_len,
                            a.finished, a.draft_len, a.accept_len, a.next_tok, a.stats, s);
    if (st != EE_OK) return st;
    if (launch_pdl(last_token_kernel, gs, 256, 0, s, (const int*)a.out_tok, a.capacity, (const int*)a.seq_len,
                   (const unsigned char*)was_finished, S, a.last_tok) != cudaSuccess)
        return EE_ERR_CUDA;
    if (a.head_use &&
        launch_pdl(head_use_kernel, gs, 256, 0, s, (const int*)draft_head, (const int*)a.draft_len, (const unsigned char*)was_finished,
                   S, k, K, reinterpret_cast<unsigned long long*>(a.head_use)) != cudaSuccess)
        return EE_ERR_CUDA;
    return EE_OK;
}

// Stand-in for the caller's model: the hidden state of a row is row `token` of a table (a token outside the
// table gives a zero row).  Warp per row, 16-byte vectors.  With `chained` the kernel takes part in the chain of
// programmatic dependent launches like the library's own kernels: it lets its dependents start at once and waits
// for its predecessors before it reads the tokens or writes a hidden state.
namespace {
struct TableList {
    const uint4* table[EE_ROUND_MAX_DRAFT_HEADS];
};
// blockIdx.y = table: layer y's rows go to h_out + y * n_rows rows (one table: the plain lookup).
__global__ void __launch_bounds__(256) hidden_from_table_kernel(const __grid_constant__ TableList tl, int V, int nvec,
                                                                const int* tokens, int n_rows, uint4* h_out, int chained) {
    if (chained) launch_dependents();
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (r >= n_rows) return;
    if (chained) grid_dependency_wait();
    const uint4* table = tl.table[blockIdx.y];
    uint4* out = h_out + ((size_t)blockIdx.y * n_rows + r) * nvec;
    const int t = ld_dep(tokens + r);
    const bool in = t >= 0 && t < V;
    for (int c = lane; c < nvec; c += 32) out[c] = in ? __ldg(table + (size_t)t * nvec + c) : make_uint4(0, 0, 0, 0);
}
}  // namespace

int hidden_from_tables(const ee_hidden_tables* m, const int* tokens, int n_rows, int which, void* h_out, cudaStream_t stream) {
    if (!m || !tokens || !h_out || which < -1 || which > EE_ROUND_MAX_DRAFT_HEADS) return 1;
    if (m->d < 8 || (m->d % 8) != 0 || m->V < 1 || n_rows < 0) return 1;
    TableList tl = {};
    int n_tables = 1;
    if (which >= 0) {
        tl.table[0] = static_cast<const uint4*>(m->table[which]);
    } else {
        // all draft tables: every non-NULL entry but the last (the verification pass's)
        int filled = 0;
        while (filled <= EE_ROUND_MAX_DRAFT_HEADS && m->table[filled]) ++filled;
        n_tables = filled - 1;
        if (n_tables < 1) return 1;
        for (int i = 0; i < n_tables; ++i) tl.table[i] = static_cast<const uint4*>(m->table[i]);
    }
    for (int i = 0; i < n_tables; ++i)
        if (!tl.table[i] || (reinterpret_cast<uintptr_t>(tl.table[i]) & 15) != 0) return 1;
    if (n_rows == 0) return 0;
    const dim3 grid((n_rows + 7) / 8, n_tables);
    if (m->chained)
        return launch_pdl(hidden_from_table_kernel, grid, 256, 0, stream, tl, m->V, m->d / 8, tokens, n_rows,
                          static_cast<uint4*>(h_out), 1) == cudaSuccess ? 0 : 1;
    // An ordinary launch, like any kernel of a caller's model: it starts when everything before it in the stream
    // has finished and what follows starts when it has.
    hidden_from_table_kernel<<<grid, 256, 0, stream>>>(tl, m->V, m->d / 8, tokens, n_rows, static_cast<uint4*>(h_out), 0);
    return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

}  // namespace ee
