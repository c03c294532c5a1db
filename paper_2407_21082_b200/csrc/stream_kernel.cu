// Decode-sized exit head: one launch does LayerNorm, the V x d projection and the softmax statistics.
//
// The kernel is bound by the single read of W from HBM, so W is read the way HBM likes it: every CTA owns
// one contiguous range of vocabulary rows and walks it front to back in 16-row stages that are fetched by
// bulk asynchronous copies (cp.async.bulk) into a shared-memory ring guarded by mbarriers.  For rows of up
// to 2 KB a stage is one contiguous 16-row block fetched by a single copy; wider rows are cut into column
// segments fetched row by row.  Every worker warp owns a private set of ring slots and a share of the row
// groups: it issues the copies for its own stages, waits for them, consumes them and re-arms the slot, so no
// barrier is shared between warps.  A worker reads its 16 x 32 sub-blocks of W straight into mma.sync
// m16n8k16 A-fragments (the K permutation this implies is applied to the activations too, which a dot
// product does not notice) and multiplies them with the M <= 32 LayerNorm'ed rows that sit in shared memory
// as bf16.  Each thread folds the logits it owns into an online (max, sum exp, sum exp*(z-max), argmax)
// state; states merge by warp shuffles, through shared memory across warps, and the last CTA to finish
// (atomic ticket, no spinning) merges the per-CTA partials and writes argmax / entropy / max-prob / exit mask.
//
// Up to four heads can share a launch: a worker simply continues with the next head's weights, warps that own no
// ring slots normalise the later heads' activations meanwhile, and one of them completes each head (CTA partial,
// ticket, final merge in the last CTA) as soon as the workers are through with it, so that only the last head's
// merge is not hidden behind the stream.
#include "common.cuh"
#include "layer_norm.cuh"
#include "kernels.h"
#include "sm100_ptx.cuh"

namespace ee {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kStageRows = 16;                        // one m16 row group per stage
constexpr int kSegMax = 1024;                         // columns of W per stage (2 KB per row)
constexpr int kMaxStages = 32;
constexpr size_t kSmemBudget = 226 * 1024;

struct StreamHead {
    const __nv_bfloat16* h;
    long long ld_h;
    const float* gamma;
    const float* beta;
    const __nv_bfloat16* W;
    const float* tau_per_row;
    float tau;
    int* argmax;
    float* entropy;
    float* maxprob;
    unsigned char* exit_mask;
};

struct StreamParams {
    StreamHead head[kStreamMaxHeads];
    int n_heads;
    float ln_eps;
    int M, d, V;                           // M: rows of this slab
    State* partials;                       // [n_heads][gridDim.x][8 * NT]
    Control* ctrl;
    int y_stride;                          // bf16 elements between rows of y in shared memory
    int seg_cols;                          // columns of W per stage
    int n_segs;                            // stages per 16-row group = ceil(d / seg_cols)
    int stage_row_bytes;                   // bytes between rows of a stage
    int n_stages;                          // ring slots in total = n_workers * slots_per_warp
    int n_workers;                         // warps that take row groups (<= kWarps)
    int slots_per_warp;                    // each worker owns this many ring slots
    int contiguous;                        // 1: a stage is 16 whole rows fetched by one copy (rows unpadded)
};

// Row stride (in bf16 elements) of y in shared memory: d rounded up to the 32-wide k-chunk, padded so
// that the stride is 64 mod 128 bytes -- the eight rows a quarter-warp reads then fall in distinct banks.
__host__ __device__ inline int y_stride_elems(int d) {
    const int kpad = (d + 31) / 32 * 32;
    return ((2 * kpad) % 128 == 0) ? kpad + 32 : kpad;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void cp_async_16(void* dst_smem, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_addr(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// Starts the asynchronous copies of everything LayerNorm reads -- the slab's rows of h (into their rows of
// y), gamma and beta -- 16 bytes per thread and step.
__device__ void stage_layer_norm_inputs(const StreamParams& p, const StreamHead& hd, __nv_bfloat16* y_s, float* gamma_s,
                                        float* beta_s, int tid, int nthreads) {
    const int nvec = p.d >> 3;
    for (int i = tid; i < p.M * nvec; i += nthreads) {
        const int r = i / nvec, c = i - r * nvec;
        cp_async_16(reinterpret_cast<uint4*>(y_s + (size_t)r * p.y_stride) + c,
                    reinterpret_cast<const uint4*>(hd.h + (size_t)r * hd.ld_h) + c);
    }
    for (int i = tid; i < (p.d >> 2); i += nthreads) {
        cp_async_16(reinterpret_cast<float4*>(gamma_s) + i, reinterpret_cast<const float4*>(hd.gamma) + i);
        cp_async_16(reinterpret_cast<float4*>(beta_s) + i, reinterpret_cast<const float4*>(hd.beta) + i);
    }
}

// LayerNorm in shared memory: the rows of y hold raw h on entry and the normalised bf16 rows on exit.  The
// 8 * NT rows are shared out over the `nw` warps of a group (this warp being number `w`).  Rows >= M and the k
// padding are zero-filled so that they contribute nothing and stay finite.
template <int NT>
__device__ void layer_norm_in_smem(const StreamParams& p, __nv_bfloat16* y_s, const float* gamma_s,
                                   const float* beta_s, int w, int nw, int lane) {
    constexpr int MPAD = 8 * NT;
    const int nvec = p.d >> 3;                                   // 16-byte vectors per row
    const int svec = p.y_stride >> 3;
    auto vec = [&](int r, int c) { return reinterpret_cast<uint4*>(y_s + (size_t)r * p.y_stride) + c; };
    for (int r0 = w; r0 < MPAD; r0 += 2 * nw) {
        const int rows[2] = {r0, r0 + nw};
        const int live = (rows[0] < p.M) + (rows[1] < MPAD && rows[1] < p.M);
        if (live > 0) layer_norm_rows_in_smem<2>(vec, rows, live, nvec, p.ln_eps, gamma_s, beta_s, lane);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = rows[i];
            if (r < MPAD)
                for (int c = (r < p.M ? nvec : 0) + lane; c < svec; c += 32) *vec(r, c) = make_uint4(0, 0, 0, 0);
        }
    }
}

template <int NT>
__global__ void __launch_bounds__(kThreads, 1) exit_head_stream_kernel(const StreamParams p) {
    constexpr int MPAD = 8 * NT;
    constexpr int CH = (NT >= 4) ? 1 : 4 / NT;                    // independent accumulator chains per n-tile
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // layout: ring stages | y of every head | per-warp partial states of every head | gamma, beta (fp32) | barriers
    const int stage_bytes = kStageRows * p.stage_row_bytes;
    const size_t y_head_elems = (size_t)MPAD * p.y_stride;
    unsigned char* ring = smem_raw;
    __nv_bfloat16* y_all = reinterpret_cast<__nv_bfloat16*>(ring + (size_t)p.n_stages * stage_bytes);
    State* wpart = reinterpret_cast<State*>(y_all + p.n_heads * y_head_elems);      // [head][warp][MPAD]
    float* gamma_s = reinterpret_cast<float*>(wpart + p.n_heads * kWarps * MPAD);
    float* beta_s = gamma_s + p.d;
    uint64_t* bars = reinterpret_cast<uint64_t*>(beta_s + p.d);
    __shared__ int s_head_done[kStreamMaxHeads];                  // workers of this CTA that have finished a head
    __shared__ int s_abort;
    const uint32_t bar_base = ptx::smem_addr(bars);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto yready_bar = [&](int k) { return bar_base + 8u * (kMaxStages + k); };
    auto hdone_bar = [&](int k) { return bar_base + 8u * (kMaxStages + kStreamMaxHeads + k); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) ptx::mbar_init(full_bar(s), 1);
        for (int k = 0; k < kStreamMaxHeads; ++k) {
            ptx::mbar_init(yready_bar(k), kWarps - p.n_workers > 0 ? kWarps - p.n_workers : 1);
            ptx::mbar_init(hdone_bar(k), p.n_workers);
            s_head_done[k] = 0;
        }
        s_abort = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();

    // This CTA's contiguous slice of the vocabulary, in 16-row groups.
    const int r_begin = (int)(((long long)p.V * blockIdx.x) / gridDim.x);
    const int r_end = (int)(((long long)p.V * (blockIdx.x + 1)) / gridDim.x);
    const int ngroups = (r_end - r_begin + kStageRows - 1) / kStageRows;
    const uint32_t ring_addr = ptx::smem_addr(ring);

    // Row group grp belongs to worker warp grp % n_workers.  The warp's stages, in order, are the column
    // segments of its groups; stage j of the warp uses its private slot j % slots_per_warp, phase
    // (j / slots_per_warp) & 1.  One warp arms, waits for, reads and re-arms a slot, so parity waits are exact.
    // With several heads the sequence simply continues with the next head's weights (same rows, same groups).
    const bool worker = warp < p.n_workers;
    const int my_groups = worker ? (ngroups - warp + p.n_workers - 1) / p.n_workers : 0;
    const int stages_per_head = my_groups * p.n_segs;
    const int my_stages = stages_per_head * p.n_heads;
    auto issue_stage = [&](int j) {
        const int hk = j / stages_per_head, jj = j - hk * stages_per_head;
        const __nv_bfloat16* W = p.head[hk].W;
        const int grp = warp + (jj / p.n_segs) * p.n_workers;
        const int seg = jj % p.n_segs;
        const int slot = warp * p.slots_per_warp + j % p.slots_per_warp;
        const int row0 = r_begin + grp * kStageRows;
        const int nrows = min(kStageRows, r_end - row0);
        const int k0 = seg * p.seg_cols;
        const uint32_t seg_bytes = (uint32_t)(min(p.seg_cols, p.d - k0) * 2);
        if (p.contiguous) {
            if (lane == 0) {
                ptx::mbar_arrive_expect_tx(full_bar(slot), seg_bytes * nrows);
                bulk_copy_g2s(ring_addr + slot * stage_bytes, W + (size_t)row0 * p.d, seg_bytes * nrows, full_bar(slot));
            }
            return;
        }
        if (lane == 0) ptx::mbar_arrive_expect_tx(full_bar(slot), seg_bytes * nrows);
        __syncwarp();
        if (lane < nrows)
            bulk_copy_g2s(ring_addr + slot * stage_bytes + lane * p.stage_row_bytes,
                          W + (size_t)(row0 + lane) * p.d + k0, seg_bytes, full_bar(slot));
    };
    int issued = 0;
    for (; issued < my_stages && issued < p.slots_per_warp; ++issued) issue_stage(issued);   // W is in flight ...

    grid_dependency_wait();                                       // h and the workspace may come from earlier kernels
    // Completion of head hk in this CTA, by one warp, once every worker has stored its per-warp states: CTA
    // partial, ticket, and in the last CTA to arrive the final merge and the decision.
    auto finalize_head = [&](int hk) {
        State* part = p.partials + ((size_t)hk * gridDim.x + blockIdx.x) * MPAD;
        for (int tok = lane; tok < MPAD; tok += 32) {
            State all[kWarps];
#pragma unroll
            for (int w = 0; w < kWarps; ++w)
                all[w] = w < p.n_workers ? wpart[(hk * kWarps + w) * MPAD + tok] : state_empty();
            part[tok] = state_combine<kWarps>(all);
        }
        __syncwarp();
        int last = 0;
        if (lane == 0) last = ticket_arrive_is_last(&p.ctrl->head_ticket[hk], gridDim.x) ? 1 : 0;
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            const StreamHead& hd = p.head[hk];
            merge_tokens(p.partials + (size_t)hk * gridDim.x * MPAD, false, (int)gridDim.x, MPAD, p.M, 0, 1, lane,
                         hd.tau_per_row, hd.tau, hd.argmax, hd.entropy, hd.maxprob, hd.exit_mask);
            if (lane == 0) p.ctrl->head_ticket[hk] = 0;            // ready for the next call
        }
    };

    // ... while LayerNorm runs.  Every warp works on the first head; the later heads are left to the warps that
    // own no ring slots (if there are any), which signal yready[k] when head k's activations are in place.
    const int n_helpers = kWarps - p.n_workers;
    const int heads_by_all = n_helpers > 0 ? 1 : p.n_heads;
    for (int hk = 0; hk < heads_by_all; ++hk) {
        __nv_bfloat16* y_s = y_all + hk * y_head_elems;
        stage_layer_norm_inputs(p, p.head[hk], y_s, gamma_s, beta_s, threadIdx.x, kThreads);
        cp_async_wait_all();
        __syncthreads();
        layer_norm_in_smem<NT>(p, y_s, gamma_s, beta_s, warp, kWarps, lane);
        __syncthreads();
    }
    if (warp >= p.n_workers) {
        const int hw = warp - p.n_workers;
        for (int hk = 1; hk < p.n_heads; ++hk) {
            __nv_bfloat16* y_s = y_all + hk * y_head_elems;
            stage_layer_norm_inputs(p, p.head[hk], y_s, gamma_s, beta_s, hw * 32 + lane, n_helpers * 32);
            cp_async_wait_all();
            asm volatile("bar.sync 2, %0;" ::"r"(n_helpers * 32) : "memory");
            layer_norm_in_smem<NT>(p, y_s, gamma_s, beta_s, hw, n_helpers, lane);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(yready_bar(hk));
            asm volatile("bar.sync 2, %0;" ::"r"(n_helpers * 32) : "memory");      // gamma_s / beta_s are reused
        }
        // The first of these warps then completes each head as soon as the workers are through with it, so that
        // no worker ever leaves its ring waiting.
        if (hw == 0) {
            bool good = true;
            for (int hk = 0; hk < p.n_heads; ++hk) {
                if (good) {
                    const bool done = ptx::mbar_wait(hdone_bar(hk), 0, &s_abort);
                    good = __all_sync(0xffffffffu, done);         // false: a worker gave up; it has recorded the error
                }
                // After a failure the head's outputs are undefined, but the CTA still takes its ticket, so that the
                // counters in the control block return to zero whatever happened.
                finalize_head(hk);
            }
        }
        return;
    }

    const int g = lane >> 2, t = lane & 3;
    bool ok = true;
    int j = 0;                                                    // this warp's stage counter over all heads
    for (int hk = 0; hk < p.n_heads; ++hk) {
      State st[NT][2];
#pragma unroll
      for (int n = 0; n < NT; ++n) {
          st[n][0] = state_empty();
          st[n][1] = state_empty();
      }
      if (ok && hk > 0 && n_helpers > 0) {
          const bool ready = ptx::mbar_wait(yready_bar(hk), 0, &s_abort);
          if (!__all_sync(0xffffffffu, ready)) {
              if (lane == 0) {
                  if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                      p.ctrl->error_info = (4u << 24) | (unsigned)hk;
                  s_abort = 1;
              }
              ok = false;
          }
      }
      if (worker && ok) {
        const uint4* y_lane = reinterpret_cast<const uint4*>(y_all + hk * y_head_elems + (size_t)g * p.y_stride + t * 8);
        const int y_tile_vecs = p.y_stride;                       // 8 rows * y_stride elements / 8 per vector
        const bool k_ragged = (p.d & 31) != 0;
        for (int grp = warp; ok && grp < ngroups; grp += p.n_workers) {
            float acc[NT][CH][4];
#pragma unroll
            for (int n = 0; n < NT; ++n)
#pragma unroll
                for (int u = 0; u < CH; ++u) acc[n][u][0] = acc[n][u][1] = acc[n][u][2] = acc[n][u][3] = 0.f;

            for (int seg = 0; seg < p.n_segs; ++seg, ++j) {
                const int slot = warp * p.slots_per_warp + j % p.slots_per_warp;
                const uint32_t phase = (uint32_t)(j / p.slots_per_warp) & 1u;
                const bool landed = ptx::mbar_wait(full_bar(slot), phase, &s_abort);
                if (!__all_sync(0xffffffffu, landed)) {
                    if (lane == 0) {
                        if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                            p.ctrl->error_info = (2u << 24) | ((unsigned)slot << 16) | ((unsigned)j & 0xffffu);
                        s_abort = 1;
                    }
                    ok = false;
                    break;
                }
                const int k0 = seg * p.seg_cols;
                const int nch = (min(p.seg_cols, p.d - k0) + 31) >> 5;
                const unsigned char* a_lo = ring + (size_t)slot * stage_bytes + g * p.stage_row_bytes + t * 16;
                const unsigned char* a_hi = a_lo + 8 * p.stage_row_bytes;
                const uint4* yk = y_lane + (k0 >> 3);
                // Four 32-column chunks per step: all operand loads first, then the MMAs ordered so that
                // consecutive ones are independent (chains of different chunks).
                int c = 0;
                for (; c + 4 <= nch && !(k_ragged && c + 4 == nch); c += 4) {
                    uint4 lo[4], hi[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        lo[u] = *reinterpret_cast<const uint4*>(a_lo + (c + u) * 64);
                        hi[u] = *reinterpret_cast<const uint4*>(a_hi + (c + u) * 64);
                    }
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        uint4 yv[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) yv[u] = yk[(size_t)n * y_tile_vecs + (c + u) * 4];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            mma_bf16_16816(acc[n][u % CH], lo[u].x, hi[u].x, lo[u].y, hi[u].y, yv[u].x, yv[u].y);
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            mma_bf16_16816(acc[n][u % CH], lo[u].z, hi[u].z, lo[u].w, hi[u].w, yv[u].z, yv[u].w);
                    }
                }
                for (; c < nch; ++c) {                                 // remainder, and the chunk that straddles d
                    uint4 lo = *reinterpret_cast<const uint4*>(a_lo + c * 64);
                    uint4 hi = *reinterpret_cast<const uint4*>(a_hi + c * 64);
                    if (k_ragged && k0 + c * 32 + t * 8 >= p.d) {      // beyond d: whatever the ring holds
                        lo = make_uint4(0, 0, 0, 0);
                        hi = make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        const uint4 yv = yk[(size_t)n * y_tile_vecs + c * 4];
                        mma_bf16_16816(acc[n][0], lo.x, hi.x, lo.y, hi.y, yv.x, yv.y);
                        mma_bf16_16816(acc[n][0], lo.z, hi.z, lo.w, hi.w, yv.z, yv.w);
                    }
                }
                // The slot has been read; hand it back to the copy engine for this warp's next stage.
                __syncwarp();
                if (issued < my_stages) {
                    ptx::fence_proxy_async();
                    issue_stage(issued);
                    ++issued;
                }
            }
            if (!ok) break;
            // The 16 x MPAD logits of this row group are complete.
            const int rowA = r_begin + grp * kStageRows + g, rowB = rowA + 8;
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                float z[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    z[q] = acc[n][0][q];
#pragma unroll
                    for (int u = 1; u < CH; ++u) z[q] += acc[n][u][q];
                }
                if (rowA < r_end) {
                    state_push(st[n][0], z[0], rowA);
                    state_push(st[n][1], z[1], rowA);
                }
                if (rowB < r_end) {
                    state_push(st[n][0], z[2], rowB);
                    state_push(st[n][1], z[3], rowB);
                }
            }
        }
      }
      // Head hk of this warp is done: reduce over the eight row lanes of the warp (lane bits 2..4); lanes 0..3 then
      // hold tokens 2t, 2t+1.  No CTA-wide barrier: the last worker of the CTA to get here finishes the head (CTA
      // partial, ticket, and in the last CTA the final merge) while the others are already on the next head.
#pragma unroll
      for (int n = 0; n < NT; ++n)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
              const State r = state_reduce_lanes<4, 16>(st[n][e]);
              if (g == 0) wpart[(hk * kWarps + warp) * MPAD + n * 8 + t * 2 + e] = r;
          }
      __syncwarp();
      if (n_helpers > 0) {
          if (lane == 0) ptx::mbar_arrive(hdone_bar(hk));         // release: the states above are visible to the waiter
      } else {
          // No idle warp: the last worker of the CTA to get here completes the head itself.
          __threadfence_block();
          int arrived = 0;
          if (lane == 0) arrived = atomicAdd(&s_head_done[hk], 1);
          arrived = __shfl_sync(0xffffffffu, arrived, 0);
          if (arrived == p.n_workers - 1) {
              __threadfence_block();
              finalize_head(hk);
          }
      }
    }
    if (!ok && lane == 0) {
        // Let this warp's copies that are still in flight land before the CTA gives its shared memory back.
        for (int q = max(0, issued - p.slots_per_warp); q < issued; ++q) {
            const int slot = warp * p.slots_per_warp + q % p.slots_per_warp;
            const uint32_t par = (uint32_t)(q / p.slots_per_warp) & 1u;
            for (uint32_t n = 0; n < (1u << 14) && !ptx::mbar_try_wait(full_bar(slot), par); ++n) __nanosleep(100);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Host side: shared-memory plan and launch
// ---------------------------------------------------------------------------------------------
struct SmemPlan {
    int seg_cols, n_segs, stage_row_bytes, n_stages, n_workers, slots_per_warp, contiguous;
    size_t bytes;
};

// Splits n ring slots of `stage` bytes into private rings: the split with the most slots wins, with at
// least min(6, n) workers (the MMAs of several stages then overlap) and at most four slots per worker.
bool split_slots(long long n, int min_workers, SmemPlan& s) {
    int best_total = 0;
    for (int c = kWarps; c >= 1; --c) {
        int b = (int)(n / c);
        if (b < 1) continue;
        if (b > 4) b = 4;
        if (c < 6 && c < n) continue;
        if (c < min_workers && n >= min_workers) continue;
        if (c * b > best_total) {
            best_total = c * b;
            s.n_workers = c;
            s.slots_per_warp = b;
        }
    }
    s.n_stages = best_total;
    return best_total > 0;
}

// Ring geometry for hidden size d with 8*nt rows of y resident; n_stages = 0 if it does not fit.
SmemPlan plan_smem(int d, int nt, int n_heads) {
    SmemPlan none = {};
    const int d64 = (d + 63) / 64 * 64;
    const size_t fixed = (size_t)n_heads * ((size_t)8 * nt * y_stride_elems(d) * sizeof(__nv_bfloat16) +
                                            (size_t)kWarps * 8 * nt * sizeof(State)) +
                         (size_t)2 * d * sizeof(float) + (kMaxStages + 2 * kStreamMaxHeads) * sizeof(uint64_t);
    const long long room = (long long)kSmemBudget - (long long)fixed;
    if (room <= 0) return none;
    if (d <= kSegMax) {
        // Rows of up to 2 KB: a stage is 16 whole rows, contiguous in W, fetched by a single copy into an
        // unpadded block (adjacent rows then share banks: a two-way conflict on the A loads, which is cheap
        // next to issuing sixteen copies of about a hundred cycles each).
        SmemPlan s = {};
        s.contiguous = 1;
        s.seg_cols = d;
        s.n_segs = 1;
        s.stage_row_bytes = 2 * d;
        const long long stage = (long long)kStageRows * s.stage_row_bytes;
        long long n = room / stage;
        if (n > kMaxStages) n = kMaxStages;
        if (n >= 2 && split_slots(n, 1, s)) {
            s.bytes = fixed + (size_t)s.n_stages * (size_t)stage;
            return s;
        }
    }
    // Wider rows: column segments of up to 1024 / 512 / 256, rows padded by 64 bytes (conflict-free), one copy
    // per row; enough workers to issue the copies faster than HBM delivers them.
    SmemPlan best = none;
    long long best_bytes = 0;
    for (int seg = kSegMax; seg >= 256; seg >>= 1) {
        SmemPlan s = {};
        s.contiguous = 0;
        s.seg_cols = d64 < seg ? d64 : seg;
        s.n_segs = (d + s.seg_cols - 1) / s.seg_cols;
        s.stage_row_bytes = 2 * s.seg_cols + 64;
        const long long stage = (long long)kStageRows * s.stage_row_bytes;
        long long n = room / stage;
        if (n > kMaxStages) n = kMaxStages;
        int min_workers = (1700 + s.seg_cols - 1) / s.seg_cols;
        if (min_workers > kWarps) min_workers = kWarps;
        if (n >= 2 && split_slots(n, min_workers, s) && (long long)s.n_stages * stage > best_bytes) {
            best_bytes = (long long)s.n_stages * stage;
            s.bytes = fixed + (size_t)best_bytes;
            best = s;
        }
        if (d64 <= seg / 2) break;          // a narrower cap would not change the stage
    }
    return best;
}

template <int NT>
ee_status launch_one(StreamParams& p, int grid, int device, cudaStream_t stream) {
    const SmemPlan plan = plan_smem(p.d, NT, p.n_heads);
    if (plan.n_stages == 0) return EE_ERR_SHAPE;
    p.seg_cols = plan.seg_cols;
    p.n_segs = plan.n_segs;
    p.stage_row_bytes = plan.stage_row_bytes;
    p.n_stages = plan.n_stages;
    p.n_workers = plan.n_workers;
    p.slots_per_warp = plan.slots_per_warp;
    p.contiguous = plan.contiguous;
    static bool configured[kMaxDevices] = {};
    if (!configured[device]) {
        if (cudaFuncSetAttribute(exit_head_stream_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSmemBudget) != cudaSuccess)
            return EE_ERR_CUDA;
        configured[device] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = plan.bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, exit_head_stream_kernel<NT>, p) == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace

int stream_slab_rows(int d, int n_heads) {
    for (int nt = kStreamMaxRows / 8; nt >= 1; nt >>= 1)
        if (plan_smem(d, nt, n_heads).n_stages > 0) return 8 * nt;
    return 0;
}

size_t stream_workspace_bytes(int n_heads) {
    return (size_t)n_heads * kStreamMaxCtas * kStreamMaxRows * sizeof(State);
}

// heads[0 .. n_heads) share M, d, V, ln_eps, workspace and stream.  Several heads go into one launch when all
// M rows fit one slab with every head's activations resident; a single head may be cut into slabs of rows.
ee_status stream_launch(const HeadArgs* heads, int n_heads) {
    const HeadArgs& a = heads[0];
    if (n_heads < 1 || n_heads > kStreamMaxHeads) return EE_ERR_SHAPE;
    const int slab = stream_slab_rows(a.d, n_heads);
    if (slab == 0 || (n_heads > 1 && a.M > slab)) return EE_ERR_SHAPE;
    const int grid = a.num_sms < kStreamMaxCtas ? a.num_sms : kStreamMaxCtas;
    unsigned char* ws = static_cast<unsigned char*>(a.workspace);
    for (int m0 = 0; m0 < a.M; m0 += slab) {
        const int rows = (a.M - m0 < slab) ? a.M - m0 : slab;
        StreamParams p;
        for (int k = 0; k < kStreamMaxHeads; ++k) {
            const HeadArgs& h = heads[k < n_heads ? k : 0];
            StreamHead& s = p.head[k];
            s.h = static_cast<const __nv_bfloat16*>(h.h) + (size_t)m0 * h.ld_h;
            s.ld_h = h.ld_h;
            s.gamma = h.gamma;
            s.beta = h.beta;
            s.W = static_cast<const __nv_bfloat16*>(h.W);
            s.tau_per_row = h.tau_per_row ? h.tau_per_row + m0 : nullptr;
            s.tau = h.tau;
            s.argmax = h.argmax + m0;
            s.entropy = h.entropy + m0;
            s.maxprob = h.maxprob + m0;
            s.exit_mask = h.exit_mask + m0;
        }
        p.n_heads = n_heads;
        p.ln_eps = a.ln_eps;
        p.M = rows;
        p.d = a.d;
        p.V = a.V;
        p.partials = reinterpret_cast<State*>(ws + kCtrlBytes);
        p.ctrl = reinterpret_cast<Control*>(ws);
        p.y_stride = y_stride_elems(a.d);
        ee_status st;
        if (rows <= 8) st = launch_one<1>(p, grid, a.device, a.stream);
        else if (rows <= 16) st = launch_one<2>(p, grid, a.device, a.stream);
        else st = launch_one<4>(p, grid, a.device, a.stream);
        if (st != EE_OK) return st;
    }
    return EE_OK;
}

}  // namespace ee
