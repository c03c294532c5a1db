// Shared device helpers: the mergeable softmax state, workspace layout, small load/pack wrappers.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <math_constants.h>

#include "eexit.h"

namespace ee {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ---------------------------------------------------------------------------------------------
// Softmax state of a subset of the vocabulary.  For logits z_v over the subset:
//   m = max z_v,  s = sum e^(z_v - m),  t = sum e^(z_v - m) (z_v - m)  (<= 0),  idx = lowest v with z_v = m.
// Entropy of the full softmax = ln s - t / s, max probability = 1 / s.  States of disjoint subsets
// merge exactly (up to rounding), so the reduction can be split across threads, warps and CTAs.
// ---------------------------------------------------------------------------------------------
struct __align__(16) State {
    float m, s, t;
    int idx;
};

__device__ __forceinline__ State state_empty() { return State{-CUDART_INF_F, 0.f, 0.f, 0x7fffffff}; }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Fold one logit into a state.  Indices arrive in increasing order within a thread, so a strict
// comparison keeps the lowest index among equal maxima.
__device__ __forceinline__ void state_push(State& a, float z, int idx) {
    if (z > a.m) {
        const float dl = a.m - z;                                  // <= 0, -inf for an empty state
        const bool was_empty = (a.s == 0.f);
        const float al = was_empty ? 0.f : ex2(dl * kLog2e);
        a.t = was_empty ? 0.f : al * fmaf(dl, a.s, a.t);
        a.s = fmaf(al, a.s, 1.f);
        a.m = z;
        a.idx = idx;
    } else {
        const float dz = z - a.m;                                  // <= 0 (NaN propagates into s, t)
        const float e = ex2(dz * kLog2e);
        a.s += e;
        a.t = fmaf(e, dz, a.t);
    }
}

// a <- merge(a, b).  Ties on the maximum keep the lower index.  Bitwise symmetric in (a, b).
__device__ __forceinline__ void state_merge(State& a, const State& b) {
    if (b.s == 0.f) return;                                        // b empty (a non-empty state has s >= 1)
    if (a.s == 0.f) { a = b; return; }                             // a empty
    const float m = fmaxf(a.m, b.m);
    const float da = a.m - m, db = b.m - m;                        // <= 0
    const float ea = ex2(da * kLog2e), eb = ex2(db * kLog2e);
    const float s = ea * a.s + eb * b.s;
    const float t = ea * fmaf(da, a.s, a.t) + eb * fmaf(db, b.s, b.t);
    const bool take_a = (a.m > b.m) || (a.m == b.m && a.idx < b.idx);
    a.idx = take_a ? a.idx : b.idx;
    a.m = (a.m != a.m || b.m != b.m) ? CUDART_NAN_F : m;
    a.s = s;
    a.t = t;
}

__device__ __forceinline__ State state_shfl_xor(const State& a, int mask) {
    State b;
    b.m = __shfl_xor_sync(0xffffffffu, a.m, mask);
    b.s = __shfl_xor_sync(0xffffffffu, a.s, mask);
    b.t = __shfl_xor_sync(0xffffffffu, a.t, mask);
    b.idx = __shfl_xor_sync(0xffffffffu, a.idx, mask);
    return b;
}

__device__ __forceinline__ State state_load_cg(const State* p) {
    const int4 raw = __ldcg(reinterpret_cast<const int4*>(p));
    State o;
    o.m = __int_as_float(raw.x);
    o.s = __int_as_float(raw.y);
    o.t = __int_as_float(raw.z);
    o.idx = raw.w;
    return o;
}

// Merge of C states held by one thread, and of one state per lane across the lanes that differ in the bits
// LO, 2*LO, .., HI of the lane index.  Unlike a chain of state_merge calls these take the maximum first and
// then add the rescaled sums, so the work per state is independent of the others (and pipelines) and the
// cross-lane part is plain shuffles of scalars.  The result is bitwise identical in every participating lane.
template <int C>
__device__ __forceinline__ State state_combine(const State (&v)[C]) {
    float m = -CUDART_INF_F;
#pragma unroll
    for (int c = 0; c < C; ++c) m = fmaxf(m, v[c].m);
    float s = 0.f, t = 0.f;
    int idx = 0x7fffffff;
#pragma unroll
    for (int c = 0; c < C; ++c) {
        const bool live = !(v[c].s == 0.f);                        // NaN counts as live and propagates
        const float dl = v[c].m - m;
        const float al = live ? ex2(dl * kLog2e) : 0.f;
        s += live ? al * v[c].s : 0.f;
        t += live ? al * fmaf(dl, v[c].s, v[c].t) : 0.f;
        idx = (live && v[c].m == m) ? min(idx, v[c].idx) : idx;
    }
    return State{(s == 0.f) ? -CUDART_INF_F : m, s, t, idx};
}

template <int LO, int HI>
__device__ __forceinline__ State state_reduce_lanes(const State& a) {
    float m = a.m;
#pragma unroll
    for (int msk = LO; msk <= HI; msk <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, msk));
    const bool live = !(a.s == 0.f);
    const float dl = a.m - m;
    const float al = live ? ex2(dl * kLog2e) : 0.f;
    float s = live ? al * a.s : 0.f;
    float t = live ? al * fmaf(dl, a.s, a.t) : 0.f;
    int idx = (live && a.m == m) ? a.idx : 0x7fffffff;
#pragma unroll
    for (int msk = LO; msk <= HI; msk <<= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, msk);
        t += __shfl_xor_sync(0xffffffffu, t, msk);
        idx = min(idx, __shfl_xor_sync(0xffffffffu, idx, msk));
    }
    return State{(s == 0.f) ? -CUDART_INF_F : m, s, t, idx};
}

// Final statistics of a full-vocabulary state, and the exit decision.
__device__ __forceinline__ void state_finish(const State& a, float tau, int* argmax, float* entropy,
                                             float* maxprob, unsigned char* exit_mask, int row) {
    const float H = logf(a.s) - a.t / a.s;
    argmax[row] = a.idx;
    entropy[row] = H;
    maxprob[row] = 1.f / a.s;
    exit_mask[row] = (H < tau) ? 1 : 0;
}

// ---------------------------------------------------------------------------------------------
// Workspace layout.  [0, 256): control block.  Then the partial states, then (tensor-core path) y.
// ---------------------------------------------------------------------------------------------
struct Control {
    unsigned int ticket;      // CTAs that have stored their partial states; returns to 0 after every call
    unsigned int error;       // 0, or a code recorded by a bounded wait that gave up
    unsigned int error_info;  // where it gave up (role << 24 | stage << 16 | low bits of the tile index)
    unsigned int pad0;
    unsigned int head_ticket[8];   // completion counters of the heads of a multi-head launch; return to 0 as well
    unsigned int merge_seen;  // unused (kept so that the layout of the words above stays as it was)
    unsigned int merge_abandon[2];   // tensor-core kernel, in-kernel merge: one bit per group of rows whose owner gave up
    unsigned int merge_pair_bits[4]; // ... and two bits per group (owner claims / last arriver takes) for the rare tie;
                                     // `ticket` and these are zeroed by the LayerNorm kernel of the next call
    unsigned int pad[45];
};
static_assert(sizeof(Control) == 256, "control block is 256 bytes");

constexpr int kCtrlBytes = 256;

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---------------------------------------------------------------------------------------------
// Loads, packing, warp reductions
// ---------------------------------------------------------------------------------------------
// Reads of data that an earlier kernel of the stream produced (activations, masks, tokens, counts, partial
// states).  Under programmatic dependent launch a kernel is resident -- possibly next to the previous launch of
// itself on the same SM -- before its producer has finished, so such data is not read-only for the kernel's
// lifetime: the non-coherent path (ld.global.nc, which the compiler also picks for const __restrict__
// parameters) may return a line an earlier co-resident kernel left in the SM's L1.  These loads go to L2, the
// point of coherence; the parameters they read through carry no __restrict__.  Weights and LayerNorm
// parameters, which no kernel of the stream writes, keep the read-only path.
template <class T>
__device__ __forceinline__ T ld_dep(const T* p) { return __ldcg(p); }

// This thread's share of the number of zero bytes among mask[0 .. n) (a mask an earlier kernel may have written):
// sixteen bytes per load once the address is aligned, four bytes per comparison.  The threads' shares add up to
// the count; used by the kernels that rank surviving rows.
__device__ __forceinline__ int zero_bytes_share(const unsigned char* mask, int n, int tid, int n_threads) {
    int cnt = 0;
    const int head = min(n, (int)((16u - (unsigned)(reinterpret_cast<uintptr_t>(mask) & 15u)) & 15u));
    for (int i = tid; i < head; i += n_threads) cnt += ld_dep(mask + i) == 0;
    const int n_vec = (n - head) >> 4;
    const uint4* v = reinterpret_cast<const uint4*>(mask + head);
    for (int i = tid; i < n_vec; i += n_threads) {
        const uint4 w = ld_dep(v + i);
        cnt += (__popc(__vcmpeq4(w.x, 0u)) + __popc(__vcmpeq4(w.y, 0u)) + __popc(__vcmpeq4(w.z, 0u)) + __popc(__vcmpeq4(w.w, 0u))) >> 3;
    }
    for (int i = head + (n_vec << 4) + tid; i < n; i += n_threads) cnt += ld_dep(mask + i) == 0;
    return cnt;
}

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&p);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  The next kernel of the stream may start once every CTA of this one has
// passed launch_dependents(); a kernel calls grid_dependency_wait() before it touches anything an earlier
// kernel of the stream writes or still reads (it returns when those kernels have completed and their stores
// are visible).  Every kernel of the head, compaction, cascade, round and loss calls is launched through
// launch_pdl and waits before it completes, so completions stay in stream order; the calibration kernels and
// the diagnostic self-tests are ordinary launches, which wait for everything before them anyway.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, int block, size_t smem, cudaStream_t stream,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// The same with the grid grouped into clusters of two CTAs (grid.x even).
inline void pair_launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute (&attr)[2], dim3 grid, int block, size_t smem,
                               cudaStream_t stream) {
    cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
}
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl_pairs(void (*kernel)(KArgs...), dim3 grid, int block, size_t smem, cudaStream_t stream,
                                    Args... args) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    pair_launch_config(cfg, attr, grid, block, smem, stream);
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// ---------------------------------------------------------------------------------------------
// Completion ticket and final merge shared by the one-launch kernels.
// ---------------------------------------------------------------------------------------------
// Thread 0 of a CTA, after a CTA-wide barrier that follows the CTA's partial-state stores: one acquire-release
// atomic publishes those stores and tells whether every other CTA has published before.
__device__ __forceinline__ bool ticket_arrive_is_last(unsigned int* counter, unsigned int n_cta) {
    unsigned int old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
    return old == n_cta - 1;
}

// The threads of the last CTA that take part (n_warps whole warps, this one being number `warp`): merge
// partials [n_cta][np] per token and write the outputs.  A warp takes TB tokens at a time; every lane first
// loads all the states it is responsible for (CTAs lane, lane + 32, .., NL of them), so the loads of a batch
// are one round trip, then combines them and the lanes reduce.
template <int TB, int NL>
__device__ __forceinline__ void merge_token_batches(const State* src, bool src_is_smem, int n_cta, int np, int M,
                                                    int warp, int n_warps, int lane, const float* tau_per_row, float tau,
                                                    int* argmax, float* entropy, float* maxprob,
                                                    unsigned char* exit_mask) {
    for (int tok0 = warp * TB; tok0 < M; tok0 += n_warps * TB) {
        State v[TB][NL];
#pragma unroll
        for (int i = 0; i < NL; ++i) {
            const int b = lane + 32 * i;
#pragma unroll
            for (int q = 0; q < TB; ++q) {
                v[q][i] = state_empty();
                if (b < n_cta && tok0 + q < M) {
                    const size_t at = (size_t)b * np + tok0 + q;
                    v[q][i] = src_is_smem ? src[at] : state_load_cg(src + at);
                }
            }
        }
        State mine = state_empty();
#pragma unroll
        for (int q = 0; q < TB; ++q) {
            const State r = state_reduce_lanes<1, 16>(state_combine<NL>(v[q]));
            if (lane == q) mine = r;
        }
        if (lane < TB && tok0 + lane < M) {
            const int tok = tok0 + lane;
            state_finish(mine, tau_per_row ? ld_dep(tau_per_row + tok) : tau, argmax, entropy, maxprob, exit_mask, tok);
        }
    }
}

// Up to 256 CTAs; grids of at most 160 CTAs (a B200 has 148 SMs) take eight tokens per batch.
__device__ __forceinline__ void merge_tokens(const State* src, bool src_is_smem, int n_cta, int np, int M, int warp,
                                             int n_warps, int lane, const float* tau_per_row, float tau, int* argmax,
                                             float* entropy, float* maxprob, unsigned char* exit_mask) {
    // as few tokens per warp and batch as keeps every warp busy: a batch's tokens are reduced one after the other
    const int per_warp = (M + n_warps - 1) / n_warps;
    if (n_cta <= 160 && per_warp <= 1)
        merge_token_batches<1, 5>(src, src_is_smem, n_cta, np, M, warp, n_warps, lane, tau_per_row, tau, argmax, entropy,
                                  maxprob, exit_mask);
    else if (n_cta <= 160 && per_warp <= 2)
        merge_token_batches<2, 5>(src, src_is_smem, n_cta, np, M, warp, n_warps, lane, tau_per_row, tau, argmax, entropy,
                                  maxprob, exit_mask);
    else if (n_cta <= 160 && per_warp <= 4)
        merge_token_batches<4, 5>(src, src_is_smem, n_cta, np, M, warp, n_warps, lane, tau_per_row, tau, argmax, entropy,
                                  maxprob, exit_mask);
    else if (n_cta <= 160)
        merge_token_batches<8, 5>(src, src_is_smem, n_cta, np, M, warp, n_warps, lane, tau_per_row, tau, argmax, entropy,
                                  maxprob, exit_mask);
    else
        merge_token_batches<4, 8>(src, src_is_smem, n_cta, np, M, warp, n_warps, lane, tau_per_row, tau, argmax, entropy,
                                  maxprob, exit_mask);
}

}  // namespace ee
