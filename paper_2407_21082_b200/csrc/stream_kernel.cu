// Decode-sized exit head: one launch does LayerNorm, the V x d projection and the softmax statistics.
//
// The kernel is bound by the single read of W from HBM.  The vocabulary is split evenly over all warps
// of the grid; a warp streams its rows with 128-bit loads that land directly in mma.sync A-fragment
// layout (the K permutation this implies is applied to the activations as well, which is legal because
// a dot product does not care about the order of its terms).  The M <= 32 normalised rows live in shared
// memory as bf16 and serve as the B operand.  Each thread folds the logits it owns into an online
// (max, sum exp, sum exp*(z-max), argmax) state; states merge by warp shuffles, through shared memory
// across warps, and the last CTA to finish (atomic ticket, no spinning) merges the per-CTA partials and
// writes argmax / entropy / max-prob / exit mask.
#include "common.cuh"
#include "kernels.h"

namespace ee {

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kDepth = 4;                  // k-chunks of W in flight per thread (2 x 16 B each)
constexpr size_t kSmemBudget = 200 * 1024;

struct StreamParams {
    const __nv_bfloat16* h;
    long long ld_h;
    const float* gamma;
    const float* beta;
    float ln_eps;
    const __nv_bfloat16* W;
    int M, d, V;                           // M: rows of this slab
    const float* tau_per_row;
    float tau;
    int* argmax;
    float* entropy;
    float* maxprob;
    unsigned char* exit_mask;
    State* partials;                       // [gridDim.x][8 * NT]
    Control* ctrl;
    int y_stride;                          // bf16 elements between rows of y in shared memory
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

// LayerNorm of the slab's rows into shared memory (bf16), one warp per row.  Rows >= M and the k padding
// are zero-filled so that they contribute nothing and stay finite.
__device__ void layer_norm_to_smem(const StreamParams& p, __nv_bfloat16* y_s, int m_pad) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nvec = p.d >> 3;                                   // 16-byte vectors per row
    const int svec = p.y_stride >> 3;
    const float inv_d = 1.f / (float)p.d;
    for (int r = warp; r < m_pad; r += kWarps) {
        uint4* yrow = reinterpret_cast<uint4*>(y_s + (size_t)r * p.y_stride);
        if (r >= p.M) {
            for (int c = lane; c < svec; c += 32) yrow[c] = make_uint4(0, 0, 0, 0);
            continue;
        }
        const uint4* hrow = reinterpret_cast<const uint4*>(p.h + (size_t)r * p.ld_h);
        float sum = 0.f;
        for (int c = lane; c < nvec; c += 32) {
            const uint4 v = __ldg(hrow + c);
            yrow[c] = v;
            sum += vec8_sum(v);
        }
        const float mu = warp_sum(sum) * inv_d;
        float sq = 0.f;
        for (int c = lane; c < nvec; c += 32) sq = vec8_sqdev(yrow[c], mu, sq);
        const float rstd = 1.f / sqrtf(warp_sum(sq) * inv_d + p.ln_eps);
        for (int c = lane; c < svec; c += 32)
            yrow[c] = (c < nvec) ? layer_norm_vec8(yrow[c], mu, rstd, p.gamma, p.beta, c) : make_uint4(0, 0, 0, 0);
    }
}

template <int NT>
__global__ void __launch_bounds__(kThreads, 1) exit_head_stream_kernel(const StreamParams p) {
    constexpr int MPAD = 8 * NT;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* y_s = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    State* wpart = reinterpret_cast<State*>(smem_raw + (size_t)MPAD * p.y_stride * sizeof(__nv_bfloat16));
    __shared__ int s_is_last;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;

    // This warp's slice of the vocabulary.
    const long long nw = (long long)gridDim.x * kWarps;
    const long long gw = (long long)blockIdx.x * kWarps + warp;
    const int r_begin = (int)(((long long)p.V * gw) / nw);
    const int r_end = (int)(((long long)p.V * (gw + 1)) / nw);
    const int ngroups = (r_end - r_begin + 15) >> 4;
    const int nchunks = (p.d + 31) >> 5;
    const int total = ngroups * nchunks;

    // Prefetch cursor (group, chunk) and the loader.
    int pg = 0, pc = 0;
    auto load_next = [&](uint4& lo, uint4& hi) {
        lo = make_uint4(0, 0, 0, 0);
        hi = make_uint4(0, 0, 0, 0);
        if (pg < ngroups) {
            const int k = pc * 32 + t * 8;
            const int row0 = r_begin + pg * 16 + g;
            if (k < p.d) {
                if (row0 < r_end) lo = ld_stream_v4(p.W + (size_t)row0 * p.d + k);
                if (row0 + 8 < r_end) hi = ld_stream_v4(p.W + (size_t)(row0 + 8) * p.d + k);
            }
            if (++pc == nchunks) { pc = 0; ++pg; }
        }
    };

    uint4 lo[kDepth], hi[kDepth];
#pragma unroll
    for (int u = 0; u < kDepth; ++u) load_next(lo[u], hi[u]);     // W is in flight while LayerNorm runs

    layer_norm_to_smem(p, y_s, MPAD);
    __syncthreads();

    float acc[NT][4];
    State st[NT][2];
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
        st[n][0] = state_empty();
        st[n][1] = state_empty();
    }

    // y for n-tile n, row g, elements [cc*32 + t*8, +8): one 16-byte vector.
    const uint4* y_lane = reinterpret_cast<const uint4*>(y_s + (size_t)g * p.y_stride + t * 8);
    const int y_tile_vecs = p.y_stride;                           // 8 rows * y_stride elements / 8 per vector
    int cg = 0, cc = 0;
    for (int it = 0; it < total; it += kDepth) {
#pragma unroll
        for (int u = 0; u < kDepth; ++u) {
            if (it + u < total) {
                const uint4 a_lo = lo[u], a_hi = hi[u];
                load_next(lo[u], hi[u]);
#pragma unroll
                for (int n = 0; n < NT; ++n) {
                    const uint4 yv = y_lane[(size_t)n * y_tile_vecs + cc * 4];
                    mma_bf16_16816(acc[n], a_lo.x, a_hi.x, a_lo.y, a_hi.y, yv.x, yv.y);
                    mma_bf16_16816(acc[n], a_lo.z, a_hi.z, a_lo.w, a_hi.w, yv.z, yv.w);
                }
                if (++cc == nchunks) {
                    // The 16 x MPAD logits of this row group are complete.
                    const int rowA = r_begin + cg * 16 + g, rowB = rowA + 8;
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        if (rowA < r_end) {
                            state_push(st[n][0], acc[n][0], rowA);
                            state_push(st[n][1], acc[n][1], rowA);
                        }
                        if (rowB < r_end) {
                            state_push(st[n][0], acc[n][2], rowB);
                            state_push(st[n][1], acc[n][3], rowB);
                        }
                        acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
                    }
                    cc = 0;
                    ++cg;
                }
            }
        }
    }

    // Merge over the eight row lanes of the warp (lane bits 2..4); lanes 0..3 then own tokens 2t, 2t+1.
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
#pragma unroll
            for (int msk = 4; msk <= 16; msk <<= 1) {
                const State o = state_shfl_xor(st[n][e], msk);
                state_merge(st[n][e], o);
            }
            if (g == 0) wpart[warp * MPAD + n * 8 + t * 2 + e] = st[n][e];
        }
    __syncthreads();

    // Merge over the CTA's warps in vocabulary order; publish the CTA partial.
    if (threadIdx.x < MPAD) {
        State a = wpart[threadIdx.x];
        for (int w = 1; w < kWarps; ++w) state_merge(a, wpart[w * MPAD + threadIdx.x]);
        p.partials[(size_t)blockIdx.x * MPAD + threadIdx.x] = a;
        __threadfence();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int old = atomicAdd(&p.ctrl->ticket, 1u);
        s_is_last = (old == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_is_last) return;

    // Last CTA: merge the partials of all CTAs, one warp per token, and decide.
    __threadfence();
    for (int tok = warp; tok < p.M; tok += kWarps) {
        State a = state_empty();
        for (int b = lane; b < (int)gridDim.x; b += 32) {
            const State o = state_load_cg(p.partials + (size_t)b * MPAD + tok);
            state_merge(a, o);
        }
#pragma unroll
        for (int msk = 1; msk <= 16; msk <<= 1) {
            const State o = state_shfl_xor(a, msk);
            state_merge(a, o);
        }
        if (lane == 0) {
            const float tau = p.tau_per_row ? p.tau_per_row[tok] : p.tau;
            state_finish(a, tau, p.argmax, p.entropy, p.maxprob, p.exit_mask, tok);
        }
    }
    if (threadIdx.x == 0) p.ctrl->ticket = 0;                     // ready for the next call
}

size_t stream_smem_bytes(int d, int nt) {
    return (size_t)8 * nt * y_stride_elems(d) * sizeof(__nv_bfloat16) + (size_t)kWarps * 8 * nt * sizeof(State);
}

template <int NT>
ee_status launch_one(const StreamParams& p, int grid, int device, cudaStream_t stream) {
    const size_t smem = stream_smem_bytes(p.d, NT);
    static bool configured[kMaxDevices] = {};
    if (!configured[device]) {
        if (cudaFuncSetAttribute(exit_head_stream_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSmemBudget) != cudaSuccess)
            return EE_ERR_CUDA;
        configured[device] = true;
    }
    exit_head_stream_kernel<NT><<<grid, kThreads, smem, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace

int stream_slab_rows(int d) {
    for (int nt = kStreamMaxRows / 8; nt >= 1; nt >>= 1)
        if (stream_smem_bytes(d, nt) <= kSmemBudget) return 8 * nt;
    return 0;
}

size_t stream_workspace_bytes(int M, int d, int V) {
    (void)M; (void)d; (void)V;
    return (size_t)kStreamMaxCtas * kStreamMaxRows * sizeof(State);
}

ee_status stream_launch(const HeadArgs& a) {
    const int slab = stream_slab_rows(a.d);
    if (slab == 0) return EE_ERR_SHAPE;
    const int grid = a.num_sms < kStreamMaxCtas ? a.num_sms : kStreamMaxCtas;
    unsigned char* ws = static_cast<unsigned char*>(a.workspace);
    for (int m0 = 0; m0 < a.M; m0 += slab) {
        const int rows = (a.M - m0 < slab) ? a.M - m0 : slab;
        StreamParams p;
        p.h = static_cast<const __nv_bfloat16*>(a.h) + (size_t)m0 * a.ld_h;
        p.ld_h = a.ld_h;
        p.gamma = a.gamma;
        p.beta = a.beta;
        p.ln_eps = a.ln_eps;
        p.W = static_cast<const __nv_bfloat16*>(a.W);
        p.M = rows;
        p.d = a.d;
        p.V = a.V;
        p.tau_per_row = a.tau_per_row ? a.tau_per_row + m0 : nullptr;
        p.tau = a.tau;
        p.argmax = a.argmax + m0;
        p.entropy = a.entropy + m0;
        p.maxprob = a.maxprob + m0;
        p.exit_mask = a.exit_mask + m0;
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
