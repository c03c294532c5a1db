/*
 * eexit -- early-exit head decision and DSSD verify step for sm_100a (B200).
 *
 * C ABI.  Unless a parameter says otherwise every pointer is a DEVICE pointer owned by the caller.
 * Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default stream), never
 * allocate, never synchronise and never take ownership.  Outputs are fully overwritten.  Argument
 * errors are detected on the host before anything is launched and reported through the return code;
 * there is no CPU fallback: a device that is not compute capability 10.x yields EE_ERR_ARCH.
 * Identical inputs give bit-identical outputs (all reductions run in a fixed order).
 *
 * Constants of the stream.  A head's parameters -- W, gamma, beta of every call, ee_head_kl's teacher
 * included -- are read while earlier work of the stream may still be running (the kernels request them
 * ahead of their dependency on that work, through the read-only path).  They must therefore be complete
 * in memory before the call is issued and must not be written by anything still in flight on `stream`
 * or on any other stream: after updating weights, synchronise (or wait on an event on the host) before
 * the next call.  Everything else -- hidden states, thresholds, masks, tokens -- may be produced by
 * earlier work of the same stream, by ordinary or by programmatic dependent launches.
 *
 * Environment switches, read by the library for comparisons and tests (none is needed in normal use):
 * EE_MULTI_KERNEL=stream|skinny|gemm|none forces the kernel of multi-head calls (read per call);
 * EE_GEMM_PAIRS=0 keeps every CTA on its own 128-row tiles and EE_GEMM_K2=0 keeps one k-block per ring slot
 * (both read once per process); EE_MERGE_LOOKS=n sets how often a row group's owner looks for the launch's
 * other CTAs before it hands its rows over (read when a call is planned); EE_CASCADE_ALL_ROWS_MAX=m moves
 * the batch size at which ee_cascade changes path (read once).  They change which kernel or tile width runs, so
 * entropy and max-probability may differ in their last bits (sums taken in another order); decisions away from
 * the tolerance band do not change.
 *
 * Notation follows the paper: a head h_k maps the hidden features of a transformer block to a
 * distribution p_k over the vocabulary V (section 3.1 "Early exit heads", section 3.2); the confidence
 * is the entropy of p_k (section 3.4.1); tau_k is the calibrated threshold of head k (section 3.4.1);
 * a row exits when H(p_k) < tau_k (section 3.4.2 and the drafting paragraph of section 4.3.1).
 */
#ifndef EEXIT_H_
#define EEXIT_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EE_OK = 0,
    EE_ERR_NULL = 1,       /* a required pointer is NULL                                    */
    EE_ERR_SHAPE = 2,      /* a size is out of range (see each call)                        */
    EE_ERR_ALIGN = 3,      /* a pointer or stride breaks the stated alignment               */
    EE_ERR_WORKSPACE = 4,  /* workspace smaller than ee_exit_head_workspace_bytes()         */
    EE_ERR_ARCH = 5,       /* current device is not sm_100                                  */
    EE_ERR_CUDA = 6,       /* a CUDA runtime/driver call failed                             */
    EE_ERR_TIMEOUT = 7     /* a bounded device-side wait gave up (see ee_query_async_error) */
} ee_status;

/* Kernel selection for ee_exit_head_path(). */
typedef enum {
    EE_PATH_AUTO = 0,      /* the library's choice: the tensor-core path for every size             */
    EE_PATH_STREAM = 1,    /* fused LayerNorm + split-V streaming kernel (any M, in slabs of rows)  */
    EE_PATH_TCGEN05 = 2,   /* LayerNorm kernel + TMA/tcgen05 GEMM with fused softmax statistics
                              (+ a merge kernel above 512 rows)                                      */
    EE_PATH_SKINNY = 3     /* one-launch tcgen05 kernel with W as the MMA's M operand: M <= 64, d % 64 == 0,
                              M_pad * d <= 64 Ki elements; other sizes return EE_ERR_SHAPE                */
} ee_path;

/* Static, human-readable name of a status code. */
const char* ee_status_string(ee_status status);

/*
 * Bytes of device scratch ee_exit_head needs for these sizes (host-only, pure; 0 if a size is invalid).
 * The scratch holds the per-(row, vocabulary-slice) partial softmax states, the bf16 LayerNorm output
 * on the tensor-core path, and a 256-byte control block (completion ticket, error word).
 */
size_t ee_exit_head_workspace_bytes(int M, int d, int V);

/*
 * Number of kernels one ee_exit_head_path call launches for these sizes and `path` (host-only, pure;
 * 0 if a size is invalid).  For callers that account for launches, e.g. when sizing a CUDA graph.
 */
int ee_exit_head_launches(int M, int d, int V, int path);

/*
 * Zeroes the control block at the start of `workspace`.  Must run once after the workspace is
 * allocated (and after ee_query_async_error reported EE_ERR_TIMEOUT); every ee_exit_head call leaves
 * the block ready for the next one.  The workspace must be 256-byte aligned.  One workspace serves one
 * call at a time: calls sharing a workspace must be ordered on one stream.  Calls with workspaces of their own
 * may run on different streams at the same time, any number of them: no kernel of the library makes one of its
 * thread blocks wait for another block to be scheduled.
 */
ee_status ee_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * The exit decision of one head for M hidden-state rows (sections 3.2, 3.4.1, 3.4.2):
 *   y      = bf16( LayerNorm(h; gamma, beta, ln_eps) )       biased variance, eps under the root
 *   z[v]   = sum_j W[v, j] * y[j]                            fp32 accumulation, logits never stored
 *   argmax = lowest v attaining max z   (the head's prediction, as in Eq. 2)
 *   entropy= ln sum exp(z - max) - sum exp(z - max)(z - max) / sum exp(z - max)      (nats)
 *   maxprob= 1 / sum exp(z - max)                            (the max-probability metric of 3.4.1)
 *   exit   = entropy < tau                                   (strict; NaN entropy never exits)
 *
 * h      bf16 [M, d], row stride ld_h elements (ld_h >= d, ld_h % 8 == 0), 16-byte aligned
 * gamma, beta  fp32 [d], 16-byte aligned
 * W      bf16 [V, d] row-major contiguous, 16-byte aligned;  d % 8 == 0, 8 <= d <= 8192, V >= 1
 * tau_per_row  fp32 [M] thresholds in nats, or NULL to use the scalar `tau` for every row
 * argmax int32 [M]; entropy fp32 [M]; maxprob fp32 [M]; exit_mask uint8 [M] (1 = exit)
 * workspace    >= ee_exit_head_workspace_bytes(M, d, V) bytes, 256-byte aligned, initialised once
 * M = 0 is a no-op returning EE_OK.
 */
ee_status ee_exit_head(const void* h, long long ld_h, const float* gamma, const float* beta, float ln_eps,
                       const void* W, int M, int d, int V, const float* tau_per_row, float tau,
                       int* argmax, float* entropy, float* maxprob, unsigned char* exit_mask,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * ee_exit_head with the third confidence metric of section 3.4.1 as well: top2gap fp32 [M] = the difference
 * between the two largest probabilities of each row's distribution (the paper's tie-breaking metric; 0 when the maximum is
 * attained twice, p itself when V = 1).  Everything else as in ee_exit_head (same workspace size); the
 * tensor-core path is used for every size.
 */
ee_status ee_exit_head_top2(const void* h, long long ld_h, const float* gamma, const float* beta, float ln_eps,
                            const void* W, int M, int d, int V, const float* tau_per_row, float tau,
                            int* argmax, float* entropy, float* maxprob, float* top2gap, unsigned char* exit_mask,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * Several heads on batches of the same shape in one call -- what the calibration pass of section 3.4.1 does
 * (every head is evaluated on every token of the calibration set) and what a verify step with several
 * heads does.  Equivalent to n_heads calls of ee_exit_head with the same M, d, V, ln_eps and workspace; up to
 * four heads share one sequence of kernel launches, which keeps the weight stream going from one head to
 * the next and pays the LayerNorm and merge steps once.  `heads` is a HOST array read during the call;
 * the pointers inside follow the rules of ee_exit_head (each head has its own h, LayerNorm parameters, W,
 * thresholds and outputs; h may be the same for all).  Workspace: ee_exit_head_multi_workspace_bytes().
 */
typedef struct {
    const void* h;             /* bf16 [M, d], row stride ld_h */
    long long ld_h;
    const float* gamma;        /* fp32 [d] */
    const float* beta;         /* fp32 [d] */
    const void* W;             /* bf16 [V, d] */
    const float* tau_per_row;  /* fp32 [M] or NULL */
    float tau;
    int* argmax;               /* int32 [M] */
    float* entropy;            /* fp32 [M] */
    float* maxprob;            /* fp32 [M] */
    unsigned char* exit_mask;  /* uint8 [M] */
} ee_head;
size_t    ee_exit_head_multi_workspace_bytes(int n_heads, int M, int d, int V);
int       ee_exit_head_multi_launches(int n_heads, int M, int d, int V);   /* kernels one call launches; host-only */
ee_status ee_exit_head_multi(const ee_head* heads, int n_heads, float ln_eps, int M, int d, int V,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * ee_exit_head_multi in two steps, for a call that is repeated with the same buffers (a decoding loop): the host
 * work of a call -- argument checks, tensor maps of the weights, tile width, launch shapes, environment overrides --
 * is done once by ee_exit_head_plan_init into a caller-owned, fixed-size plan (plain data, no allocation, nothing
 * to release), and ee_exit_head_plan_run only launches (two or three kernel launches per four heads).  Same
 * passages, results and workspace as ee_exit_head_multi; up to EE_PLAN_MAX_HEADS heads.  Every pointer given at
 * initialisation (the heads' inputs, parameters, weights, thresholds, outputs, the workspace) is captured: the
 * buffers must stay where they are, their CONTENTS may change between runs.  The device that is current at
 * initialisation must be current at every run; a plan may be run on any stream, one run at a time (it shares its
 * workspace).  ee_exit_head_plan_run_host is the plan's counterpart of ee_exit_head_multi_host: h_host (h_bytes,
 * pinned for an asynchronous copy) is copied to h_dev, the plan is run, results_dev (results_bytes) is copied to
 * results_host; the plan must have been initialised with heads whose h and outputs lie inside h_dev and results_dev.
 */
#define EE_PLAN_MAX_HEADS 16
#define EE_EXIT_HEAD_PLAN_BYTES (64 + (EE_PLAN_MAX_HEADS / 4) * 2048)
typedef struct {
    unsigned long long opaque[EE_EXIT_HEAD_PLAN_BYTES / 8];
} ee_exit_head_plan;
ee_status ee_exit_head_plan_init(ee_exit_head_plan* plan, const ee_head* heads, int n_heads, float ln_eps, int M, int d,
                                 int V, void* workspace, size_t workspace_bytes);
ee_status ee_exit_head_plan_run(const ee_exit_head_plan* plan, void* stream);
ee_status ee_exit_head_plan_run_host(const ee_exit_head_plan* plan, const void* h_host, void* h_dev, size_t h_bytes,
                                     void* results_host, const void* results_dev, size_t results_bytes, void* stream);

/* Same operation with the kernel chosen by the caller (`path` is an ee_path); used to cross-check the
 * kernels against each other and to time them separately. */
ee_status ee_exit_head_path(const void* h, long long ld_h, const float* gamma, const float* beta, float ln_eps,
                            const void* W, int M, int d, int V, const float* tau_per_row, float tau,
                            int* argmax, float* entropy, float* maxprob, unsigned char* exit_mask,
                            void* workspace, size_t workspace_bytes, void* stream, int path);

/*
 * ee_exit_head for a caller whose activations and results live in HOST memory (pinned memory makes
 * the copies asynchronous).  Copies h_host -> h_dev on `stream`, runs the head, copies the four outputs
 * to the *_host arrays.  The device arrays are caller-provided staging of the same shapes as in
 * ee_exit_head; weights, thresholds and workspace stay device pointers.  Returns without synchronising:
 * the host arrays are valid after the caller synchronises `stream`.
 * h_host is dense [M, d] (row stride d); h_dev receives it with row stride d.
 */
ee_status ee_exit_head_host(const void* h_host, void* h_dev, const float* gamma, const float* beta, float ln_eps,
                            const void* W, int M, int d, int V, const float* tau_per_row, float tau,
                            int* argmax_host, float* entropy_host, float* maxprob_host, unsigned char* exit_mask_host,
                            int* argmax_dev, float* entropy_dev, float* maxprob_dev, unsigned char* exit_mask_dev,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * ee_exit_head without a workspace argument, for callers that have no way to provide scratch memory.
 * (The paper has no counterpart for this call; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs after a serving process has handed all device memory to its own pool
 * and banned cudaMalloc (which stalls the whole device and can fail on a fragmented heap), plug-ins
 * and callbacks hosted by a runtime whose allocator they may not call, and latency-critical loops
 * where no allocator of any kind is permitted.  This entry point calls no cudaMalloc, no cudaFree and no
 * allocating library routine.  Its scratch is a fixed ~128 KB array inside the library's device image;
 * every GPU that loads the library carries that array until the process exits.
 *
 * Same arguments, results and error codes as ee_exit_head, minus workspace, with these limits:
 *   - M <= EE_STATIC_MAX_ROWS (decode-sized batches; the fused streaming kernel is always used) and the
 *     rows must fit one launch of that kernel (any d <= 2048 does for 32 rows).  Larger sizes return
 *     EE_ERR_SHAPE and launch nothing: use ee_exit_head with a workspace for them.
 *   - The first call on each device looks up the array's device address and zeroes its control block
 *     (on `stream`, ahead of the kernel).  Make that first call during start-up, before any stream
 *     capture, with the device it is meant for current.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the kernel
 *     rewrites what it reads and leaves the control block zeroed.  Calls that overlap on the GPU (two
 *     streams, two host threads) therefore race: order them on one stream or with events.
 *   - A bounded device-side wait that gives up is recorded in the array's control block, which the caller
 *     cannot address: ee_exit_head_static_query_error reads it (ee_query_async_error needs a workspace pointer
 *     and does not apply here).
 */
#define EE_STATIC_MAX_ROWS 32
ee_status ee_exit_head_static(const void* h, long long ld_h, const float* gamma, const float* beta, float ln_eps,
                              const void* W, int M, int d, int V, const float* tau_per_row, float tau,
                              int* argmax, float* entropy, float* maxprob, unsigned char* exit_mask, void* stream);

/*
 * ee_query_async_error for the built-in array of ee_exit_head_static on the current device (no counterpart in the
 * paper): synchronises `stream`, returns EE_OK if no wait gave up since the last query, else EE_ERR_TIMEOUT -- the
 * outputs of that call are undefined -- after zeroing the array's whole control block on `stream`, which is the
 * recovery step: the next ee_exit_head_static call starts from a clean state.  Allocates nothing.
 */
ee_status ee_exit_head_static_query_error(void* stream);

/*
 * ee_selftest_wait_timeout aimed at the built-in array (diagnostic, no counterpart in the paper): one small kernel
 * whose only wait runs out after about a millisecond and records the error word there; nothing faults.  The next
 * ee_exit_head_static_query_error returns EE_ERR_TIMEOUT.  For tests of a caller's error handling.
 */
ee_status ee_exit_head_static_selftest_timeout(void* stream);

/*
 * ee_exit_head_multi for a caller whose activations and results live in HOST memory: one copy in, the heads,
 * one copy out (same passage as ee_exit_head_multi; pinned host memory makes the copies asynchronous).
 *   h_host        bf16 [n_heads][M][d], dense: head k's input rows
 *   h_dev         device staging of the same size
 *   results_host  packed results, ee_exit_head_results_bytes(n_heads, M) bytes; head k's block starts at
 *                 byte k * ee_exit_head_results_bytes(1, M) and holds argmax int32 [M], entropy fp32 [M],
 *                 maxprob fp32 [M], exit_mask uint8 [M] back to back (the block is padded to 16 bytes)
 *   results_dev   device staging of the same size and layout; the device copies of the results stay valid
 *                 there for later calls on the stream (ee_compact, dssd_accept)
 * Of each ee_head only gamma, beta, W, tau_per_row and tau are read; its h, ld_h and output pointers are
 * ignored.  Returns without synchronising: results_host is valid after the caller synchronises `stream`.
 */
size_t    ee_exit_head_results_bytes(int n_heads, int M);      /* host-only, pure; 0 if a size is invalid */
ee_status ee_exit_head_multi_host(const ee_head* heads, int n_heads, float ln_eps, int M, int d, int V,
                                  const void* h_host, void* h_dev, void* results_host, void* results_dev,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Continuation of the rows that did not exit (section 3.4.2: an input keeps going through the model's
 * layers until a head is confident).  Order-preserving stream compaction:
 *   kept_idx   int32 [M]: ascending indices i with exit_mask[i] == 0 (first *kept_count entries valid)
 *   kept_count int32 [1] on the device
 *   h_out      bf16 [M, d] capacity (row stride d): h_out[r, :] = h[kept_idx[r], :] bit for bit;
 *              may be NULL to skip the gather.  Rows at and beyond *kept_count are left untouched.
 * h is the head's INPUT (pre-LayerNorm) rows: bf16 [M, d], row stride ld_h, d % 8 == 0, 16-byte
 * aligned (h may be NULL iff h_out is NULL).  Any non-zero mask byte counts as "exited".  M = 0 writes
 * kept_count = 0.
 */
ee_status ee_compact(const unsigned char* exit_mask, const void* h, long long ld_h, int M, int d,
                     int* kept_idx, int* kept_count, void* h_out, void* stream);

/*
 * DSSD drafting stop and verification (section 4.3.1).  For each of S sequences with k draft slots:
 *   draft_len[s]  = number of leading slots with draft_exit_mask[s, j] != 0, at most k  (drafting stops
 *                   at the buffer limit or at the first position where the head is not confident)
 *   accept_len[s] = number of leading j < draft_len[s] with draft_tok[s, j] == verify_tok[s, j]
 *                   (the accepted prefix)
 *   next_tok[s]   = verify_tok[s, accept_len[s]] if accept_len[s] < kv, else -1  (the full model's token
 *                   that rewrites the first mismatch, or follows a fully accepted draft)
 * draft_tok int32 [S, k]; draft_exit_mask uint8 [S, k] or NULL (all confident); verify_tok int32
 * [S, kv], kv >= k >= 1; outputs int32 [S].  S = 0 is a no-op.
 */
ee_status dssd_accept(const int* draft_tok, const unsigned char* draft_exit_mask, const int* verify_tok,
                      int S, int k, int kv, int* draft_len, int* accept_len, int* next_tok, void* stream);

/*
 * Commit step of one DSSD round for S sequences whose committed tokens live in device buffers (section 4.3.1:
 * the three stop conditions of the drafting phase and the atomic commit of the verification phase).  For a
 * sequence with finished[s] == 0:
 *   draft_len[s]  = leading confident draft slots, at most k (the buffer limit), and not beyond the first
 *                   drafted token equal to eos_token (that token is the last one drafted); eos_token < 0
 *                   switches that stop off
 *   accept_len[s] = leading j < draft_len[s] with draft_tok[s, j] == verify_tok[s, j]
 *   committed     = the accepted tokens, then verify_tok[s, accept_len[s]] if accept_len[s] < kv and the last
 *                   accepted token is not eos_token (next_tok[s]; -1 when nothing follows), appended to
 *                   out_tok[s, seq_len[s] ...] and cut at `capacity`
 *   seq_len[s] grows by the number appended; finished[s] becomes 1 when eos_token was appended or the buffer
 *   is full.
 * A sequence with finished[s] != 0 is left untouched (its draft_len, accept_len = 0, next_tok = -1).
 * stats int64 [4] accumulates over calls: tokens drafted, accepted, appended, and sequences that took part (the
 * paper's acceptance rate is accepted / drafted, its wasted tokens drafted - accepted); the caller zeroes it.
 * draft_tok int32 [S, k], draft_exit_mask uint8 [S, k] or NULL, verify_tok int32 [S, kv], 1 <= k <= 32,
 * kv >= k; out_tok int32 [S, capacity]; seq_len int32 [S]; finished uint8 [S]; the three outputs int32 [S].
 */
ee_status dssd_commit(const int* draft_tok, const unsigned char* draft_exit_mask, const int* verify_tok, int S,
                      int k, int kv, int eos_token, int* out_tok, int capacity, int* seq_len,
                      unsigned char* finished, int* draft_len, int* accept_len, int* next_tok, long long* stats,
                      void* stream);

/*
 * One whole DSSD round for S sequences (section 4.3.1: drafting phase, verification phase, commit), issued on
 * the stream without any synchronisation.  Drafting uses K >= 1 draft heads, shallowest first: at every position
 * the first head whose entropy is below its threshold supplies the token (the paper's per-token head selection);
 * a position that no head is sure of ends the draft (stop iii, the fallback to the full model).
 * The transformer is the caller's: `hidden` is called K times per drafting step, k steps (which = h, 0 <= h < K:
 * n_rows = S tokens, one per sequence, the token each sequence's next position follows; the hidden states AT HEAD
 * h'S LAYER are wanted) and once for the verification pass (which = K: n_rows = S * (k + 1) tokens, row (s, j) =
 * the token before draft position j, j = k being the bonus position; the full model's final hidden states); it
 * must enqueue on `stream` work that writes the hidden states bf16 [n_rows, d] (dense) of the positions FOLLOWING
 * those tokens to h_out, and return 0.  A real model produces the states of all its exit layers in one forward
 * pass: with hidden_all_layers != 0 the drafting steps call `hidden` ONCE per step, with which = -1, and it must
 * write layer h's states to h_out + h * n_rows * d elements for every h < K (the verification call is unchanged).
 * Both pointers it receives are device buffers inside `workspace`.  The work it enqueues may be ordinary stream
 * work, or kernels launched with programmatic stream serialization that trigger their dependents early -- the
 * round's own kernels are chained that way -- provided every such kernel executes griddepcontrol.wait before it
 * reads `tokens` or writes `h_out`, and reads `tokens` through L2 (ld.global.cg or an equivalent coherent load,
 * not the read-only path): the token buffer is rewritten by a kernel that may still be running when the model's
 * kernel becomes resident.
 *   drafting step j : the K draft heads (their gamma, beta, W; tau is each head's threshold) on the step's hidden
 *                     states, all in one launch sequence; per sequence the first confident head's argmax = drafted
 *                     token; the token feeds step j + 1
 *   verification    : verify head (the full model's; its tau is ignored) on all S * (k + 1) rows
 *   commit          : dssd_commit with kv = k + 1 and the given eos_token; then last_tok[s] = the last token
 *                     committed, for the sequences that took part
 * Every sequence goes through all k drafting steps (what lies beyond its stop is ignored by the commit), so
 * the launch sequence does not depend on device data.  State (device, in/out): last_tok int32 [S], out_tok
 * int32 [S, capacity], seq_len int32 [S], finished uint8 [S], stats int64 [4]; outputs of the round: draft_len,
 * accept_len, next_tok int32 [S].  n_draft_heads = 0 means one draft head, `draft_head` (then `which` is 0 while
 * drafting and 1 for the verification pass); otherwise draft_heads is a HOST array of n_draft_heads <=
 * EE_ROUND_MAX_DRAFT_HEADS heads and `draft_head` is ignored.  head_use (device int64 [K], may be NULL) accumulates
 * over calls, per head, the drafted positions it supplied -- positions inside a draft (j < draft_len) of sequences
 * that took part: the head-usage statistic of the paper's DSSD experiments (the mean exit head while drafting is
 * sum h * head_use[h] / sum head_use[h]); the caller zeroes it.
 * Workspace: dssd_round_multi_workspace_bytes(S, k, d, V, K) (dssd_round_workspace_bytes = the same with K = 1),
 * 256-byte aligned, initialised once with ee_workspace_init.  1 <= k <= 32.
 */
#define EE_ROUND_MAX_DRAFT_HEADS 8
typedef int (*ee_hidden_fn)(void* user, const int* tokens, int n_rows, int which, void* h_out, void* stream);
typedef struct {
    int S, k, d, V;
    float ln_eps;
    int eos_token;
    ee_head draft_head, verify_head;    /* gamma, beta, W, tau are read; h, ld_h and the outputs are ignored */
    ee_hidden_fn hidden;
    void* hidden_user;
    int* last_tok;
    int* out_tok;
    int capacity;
    int* seq_len;
    unsigned char* finished;
    long long* stats;
    int* draft_len;
    int* accept_len;
    int* next_tok;
    void* workspace;
    size_t workspace_bytes;
    void* stream;
    int n_draft_heads;
    const ee_head* draft_heads;
    long long* head_use;
    int hidden_all_layers;              /* non-zero: one call of `hidden` per drafting step fills every draft head's layer */
} ee_dssd_round_args;
size_t    dssd_round_workspace_bytes(int S, int k, int d, int V);     /* host-only, pure; 0 if a size is invalid */
size_t    dssd_round_multi_workspace_bytes(int S, int k, int d, int V, int n_draft_heads);
ee_status dssd_round(const ee_dssd_round_args* args);

/*
 * A ready-made ee_hidden_fn for tests and benchmarks (no counterpart in the paper; the transformer is the
 * caller's): the hidden state of a row is row `token` of table[which] -- table[h] for draft head h's layer,
 * table[K] for the verification pass -- each bf16 [V, d] on the device, contiguous, 16-byte aligned; a token
 * outside [0, V) gives a zero row; which = -1 (hidden_all_layers) fills the layers of all draft tables -- every
 * non-NULL table but the last -- with one launch.  Give dssd_round `ee_hidden_from_tables` as `hidden` and a pointer to an
 * ee_hidden_tables (host memory that outlives the call) as `hidden_user`.  One kernel launch on `stream` per call;
 * returns 0, or 1 if an argument is unusable or the launch failed.  chained = 0: an ordinary launch; chained != 0:
 * the kernel is launched with programmatic stream serialization, lets its dependents start at once and waits for
 * its predecessors before it touches the tokens, like the library's own kernels.
 */
typedef struct {
    const void* table[EE_ROUND_MAX_DRAFT_HEADS + 1];
    int d, V;
    int chained;
} ee_hidden_tables;
int ee_hidden_from_tables(void* user, const int* tokens, int n_rows, int which, void* h_out, void* stream);

/*
 * ee_compact and dssd_accept in one kernel launch, for a decoding step that needs both (section 3.4.2 and
 * section 4.3.1): both read the heads' outputs and write disjoint results, so one launch does the work of two
 * and a step saves a launch boundary.  Arguments, layouts and results are exactly those of the two calls;
 * the mask given to the compaction (exit_mask, M rows) and the one given to the draft-length count
 * (draft_exit_mask, S x k) may be the same buffer or different ones.
 */
ee_status ee_compact_accept(const unsigned char* exit_mask, const void* h, long long ld_h, int M, int d,
                            int* kept_idx, int* kept_count, void* h_out, const int* draft_tok,
                            const unsigned char* draft_exit_mask, const int* verify_tok, int S, int k, int kv,
                            int* draft_len, int* accept_len, int* next_tok, void* stream);

/*
 * The inference-time cascade of section 3.4.2 ("Inference Process") for a batch: the heads are tried in the
 * order given; head k is evaluated (as by ee_exit_head, scalar threshold heads[k].tau, rule H < tau) on the
 * rows that no earlier head answered, reading row i of the batch from ITS OWN hidden states heads[k].h
 * (bf16 [M, d], row stride heads[k].ld_h: the batch at head k's layer); a row stops at the first head that
 * answers it.  A last head with tau = +infinity plays the full model.
 * Outputs (device): exit_head int32 [M] = index of the answering head, n_heads if none; token int32 [M] = that
 * head's argmax, -1 if none; entropy fp32 [M] = that head's entropy, NaN if none; rows_in int32 [n_heads] =
 * the number of rows each head was evaluated on (head usage = rows_in[k] - rows_in[k+1]).
 * Of each ee_head the output pointers are ignored and tau_per_row must be NULL.  The row counts stay on the
 * device: no synchronisation between heads; head k's weights are streamed once whatever the count.  Above 512
 * rows its LayerNorm and statistics run on the surviving rows only (three launches per head).  With at most 512
 * rows (where the weight stream and the chain of launches, not the rows, set the time) the heads are evaluated
 * on every row, four heads per launch, and a row takes the first head that answers it: same results, two
 * launches plus one small one per four heads.  Workspace: ee_cascade_workspace_bytes(M, d, V), 256-byte aligned, initialised once with
 * ee_workspace_init.  M = 0 writes rows_in = 0.
 */
size_t    ee_cascade_workspace_bytes(int M, int d, int V);      /* host-only, pure; 0 if a size is invalid */
ee_status ee_cascade(const ee_head* heads, int n_heads, float ln_eps, int M, int d, int V, int* exit_head,
                     int* token, float* entropy, int* rows_in, void* workspace, size_t workspace_bytes,
                     void* stream);

/*
 * Forward pass of a head's self-supervised training objective (section 3.3, paragraph "Losses":
 * L_KL(y_hat || f_theta) with y_hat the head's distribution and f_theta the main model's).  For each of M tokens
 * the head's logits come from its hidden states (h_head, LayerNorm gamma_head / beta_head, W_head) and the
 * teacher's from the final hidden states and the main model's head, both exactly as in ee_exit_head; neither
 * M x V logit matrix is ever stored.
 *   kl   fp32 [M]: sum_v p_head(v) (log p_head(v) - log p_teacher(v)), nats
 *   ce   fp32 [M]: -log p_head(labels[i]), the supervised objective L_CE of the same paragraph; ce and labels
 *                  (int32 [M], 0 <= label < V) are given together or both NULL
 *   loss fp32 [2]: the means of kl and (when asked for) of ce, each summed in a fixed order (bit-identical from
 *                  run to run); may be NULL.  The hybrid objective is alpha * loss[1] + (1 - alpha) * loss[0].
 * h_* bf16 [M, d] (row strides ld_* elements), gamma_*, beta_* fp32 [d], W_* bf16 [V, d]; alignment as in
 * ee_exit_head.  Workspace: ee_head_kl_workspace_bytes(M, d, V), 256-byte aligned, initialised once with
 * ee_workspace_init.  M = 0 is a no-op.
 */
size_t    ee_head_kl_workspace_bytes(int M, int d, int V);      /* host-only, pure; 0 if a size is invalid */
ee_status ee_head_kl(const void* h_head, long long ld_head, const float* gamma_head, const float* beta_head,
                     const void* W_head, const void* h_teacher, long long ld_teacher, const float* gamma_teacher,
                     const float* beta_teacher, const void* W_teacher, float ln_eps, int M, int d, int V,
                     const int* labels, float* kl, float* ce, float* loss, void* workspace, size_t workspace_bytes,
                     void* stream);

/*
 * Calibration of one head's threshold from a calibration set (section 3.4.1, "Calibration of Confidence
 * Thresholds": Eq. 3 and the two equations that define the index j-hat and tau_k = c_{k, j-hat}), with the
 * entropy as the confidence metric.  Over n calibration tokens:
 *   t_j = [argmax_head[j] == argmax_final[j]]                                   (Eq. 3)
 *   the candidate sets are { j : entropy[j] <= v } for the distinct entropies v (tokens of equal entropy
 *   enter together, so the result does not depend on how equal values are ordered);
 *   the largest candidate set whose proportion of t_j = 1 is >= epsilon is chosen (the comparison
 *   correct >= epsilon * count is made in fp64) -- the paper's smallest index j-hat in ascending confidence.
 * Outputs (device): tau fp32 [1] = the largest entropy inside the chosen set (the paper's tau; a token AT the
 * threshold is inside the set, so a caller of ee_exit_head, whose rule is H < tau, passes the next float
 * above it), or -inf if no set qualifies (the head then never exits); counts int32 [3] = size of the chosen
 * set, number of correct predictions in it, j-hat (1-based, 0 if none).
 * entropy fp32 [n] must not contain NaN; argmax_head, argmax_final int32 [n]; 0 <= epsilon <= 1; n = 0 gives
 * tau = -inf.  Workspace: ee_calibrate_workspace_bytes(n) bytes, 256-byte aligned (two copies of one
 * 64-bit word per token and the sort's histograms); needs no initialisation.
 */
size_t    ee_calibrate_workspace_bytes(int n);       /* host-only, pure; 0 if n < 0 */
ee_status ee_calibrate(const float* entropy, const int* argmax_head, const int* argmax_final, int n,
                       double epsilon, float* tau, int* counts, void* workspace, size_t workspace_bytes,
                       void* stream);

/*
 * Synchronises `stream`, then reads and clears the error word of the workspace's control block.
 * Every device-side wait in the tensor-core kernel is bounded; one that gives up records itself there
 * and the kernel drains and returns.  EE_OK if nothing was recorded, EE_ERR_TIMEOUT otherwise (outputs
 * of that call are then undefined; call ee_workspace_init before reusing the workspace).
 */
ee_status ee_query_async_error(void* workspace, void* stream);

/*
 * Diagnostic for the error path above (no counterpart in the paper): launches one small kernel whose only wait
 * is on a barrier that nothing signals.  The wait gives up after about a millisecond, the kernel records the
 * error word in `workspace`'s control block as the real kernels would and returns normally -- nothing faults,
 * the context and the workspace stay usable.  The next ee_query_async_error on that workspace returns
 * EE_ERR_TIMEOUT (and clears the word).  For tests of a caller's error handling.
 */
ee_status ee_selftest_wait_timeout(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Diagnostic for the roofline (no counterpart in the paper): reads `bytes` bytes (rounded down to whole 16 KB
 * stages; at least one) of the device buffer `buffer` (16-byte aligned) once, with the mechanism the kernels
 * stream weights with -- one CTA per SM, contiguous bulk asynchronous copies into a shared-memory ring -- and
 * looks at none of them.  Timed by the caller over a buffer larger than L2 it gives the rate a read-only
 * stream reaches on this device, to set beside the copy figure the roofline fractions are quoted against.
 * Writes nothing but the error word of `workspace`'s control block if a bounded wait gives up
 * (ee_query_async_error reports it).  Asynchronous on `stream`.
 */
ee_status ee_selftest_read_stream(const void* buffer, size_t bytes, void* workspace, size_t workspace_bytes,
                                  void* stream);

#ifdef __cplusplus
}
#endif
#endif /* EEXIT_H_ */
