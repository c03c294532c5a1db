// Exit head for 1 <= M <= 64 rows on the tcgen05 tensor cores, one launch, bound by the single read of W.
//
// Operands are swapped with respect to the large-M kernel: a tile of 128 vocabulary rows of W is the MMA's
// M-side operand (streamed from HBM by TMA into a shared-memory ring, 128-byte swizzle), and the N = 16 / 32 /
// 64 LayerNorm'ed activation rows are the N-side operand, resident in shared memory for the whole kernel (each
// CTA normalises them itself, writing the swizzled layout directly).  The MMAs are issued by one thread and
// cost the SM nothing else, so a ring slot is free again as soon as the tensor core has read it.  The
// accumulator [128 vocabulary rows x N tokens] lives in TMEM (two buffers).  Epilogue warps read it back with
// the vocabulary row on the lane; every thread keeps one online state per token (at most 32 tokens per thread:
// for N = 64 a second set of epilogue warps takes tokens 32..63), so a tile costs one state update per logit and
// no cross-lane traffic.  At the end the per-lane states are transposed through shared memory (the ring is
// free by then) and merged per token.  Per-CTA partial states, atomic ticket, last CTA merges and decides, as
// in the streaming kernel.
#include "common.cuh"
#include "kernels.h"
#include "sm100_ptx.cuh"
#include "tensor_map.h"

namespace ee {

namespace {

// warp 0 TMA, warp 1 MMA, then four epilogue warps per group of up to 32 tokens
__host__ __device__ constexpr int sk_groups(int n) { return n <= 32 ? 1 : n / 32; }
__host__ __device__ constexpr int sk_threads(int n) { return 64 + 128 * sk_groups(n); }
constexpr int kTileRows = 128;             // MMA M
constexpr int kBK = 64;
constexpr int kStageBytes = kTileRows * kBK * 2;      // 16 KB
constexpr int kSkMaxStages = 12;
constexpr size_t kSkSmemBudget = 226 * 1024;

struct SkinnyParams {
    const __nv_bfloat16* h;
    long long ld_h;
    const float* gamma;
    const float* beta;
    float ln_eps;
    int M, d, V;
    const float* tau_per_row;
    float tau;
    int* argmax;
    float* entropy;
    float* maxprob;
    unsigned char* exit_mask;
    State* partials;                       // [gridDim.x][N]
    Control* ctrl;
    int k_blocks;                          // d / 64
    int box_rows;                          // vocabulary rows per tile (<= 128), the TMA box height
    int n_stages;
};

__device__ __forceinline__ void sk_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void sk_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void sk_cp_async_16(void* dst_smem, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_addr(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void sk_cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// Address of 16-byte vector c (columns 8c .. 8c+7) of activation row r inside the swizzled y tiles:
// tile kb = c / 8 holds [N rows][64 columns], rows of 128 bytes, 16-byte chunks XOR-ed with (row & 7).
template <int N>
__device__ __forceinline__ uint4* y_vec(unsigned char* y_tiles, int r, int c) {
    const int kb = c >> 3, chunk = c & 7;
    return reinterpret_cast<uint4*>(y_tiles + (size_t)kb * (N * 128) + r * 128 + ((chunk ^ (r & 7)) << 4));
}

template <int N>
__global__ void __launch_bounds__(sk_threads(N), 1)
exit_head_skinny_kernel(const __grid_constant__ CUtensorMap tm_w, const SkinnyParams p) {
    constexpr int TOK = N < 32 ? N : 32;                          // tokens per epilogue thread
    constexpr int GROUPS = sk_groups(N);
    constexpr int kSkThreads = sk_threads(N);
    constexpr int kSkWarps = kSkThreads / 32;
    constexpr int TMEM_COLS = (2 * N < 32) ? 32 : 2 * N;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
    const int S = p.n_stages;
    // layout: W stages | y tiles | gamma, beta | per-quarter states | barriers
    unsigned char* y_tiles = smem + (size_t)S * kStageBytes;
    float* gamma_s = reinterpret_cast<float*>(y_tiles + (size_t)p.k_blocks * N * 128);
    float* beta_s = gamma_s + p.d;
    State* qpart = reinterpret_cast<State*>(beta_s + p.d);       // [4][N]
    unsigned char* bar_mem = reinterpret_cast<unsigned char*>(qpart + 4 * N);
    const uint32_t w_base = ptx::smem_addr(smem);
    const uint32_t y_base = ptx::smem_addr(y_tiles);
    const uint32_t bar_base = ptx::smem_addr(bar_mem);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kSkMaxStages + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kSkMaxStages + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kSkMaxStages + 2 + b); };
    const uint32_t drain_bar = bar_base + 8u * (2 * kSkMaxStages + 4);
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(bar_mem + 8 * (2 * kSkMaxStages + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * kSkMaxStages + 5) + 4);
    __shared__ int s_is_last;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    sk_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull_bar(b), 1);
            ptx::mbar_init(tempty_bar(b), 4 * GROUPS);
        }
        ptx::mbar_init(drain_bar, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tm_w);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    // This CTA's contiguous slice of the vocabulary, in tiles of box_rows rows.
    const int r_begin = (int)(((long long)p.V * blockIdx.x) / gridDim.x);
    const int r_end = (int)(((long long)p.V * (blockIdx.x + 1)) / gridDim.x);
    const int n_tiles = (r_end - r_begin + p.box_rows - 1) / p.box_rows;
    const int total_loads = n_tiles * p.k_blocks;
    const uint32_t stage_tx = (uint32_t)p.box_rows * 128u;

    // The weights do not depend on earlier kernels of the stream: fill the ring before waiting for them.
    int preloaded = 0;
    if (threadIdx.x == 0) {
        for (; preloaded < total_loads && preloaded < S; ++preloaded) {
            const int tile = preloaded / p.k_blocks, kb = preloaded - tile * p.k_blocks;
            ptx::mbar_arrive_expect_tx(full_bar(preloaded), stage_tx);
            ptx::tma_load_2d(w_base + preloaded * kStageBytes, &tm_w, kb * kBK, r_begin + tile * p.box_rows,
                             full_bar(preloaded));
        }
    }

    // ------------------------------------------------------------------ LayerNorm into the swizzled y tiles
    sk_grid_dependency_wait();
    {
        const int nvec = p.d >> 3;
        for (int i = threadIdx.x; i < p.M * nvec; i += kSkThreads) {
            const int r = i / nvec, c = i - r * nvec;
            sk_cp_async_16(y_vec<N>(y_tiles, r, c), reinterpret_cast<const uint4*>(p.h + (size_t)r * p.ld_h) + c);
        }
        for (int i = threadIdx.x; i < (p.d >> 2); i += kSkThreads) {
            sk_cp_async_16(reinterpret_cast<float4*>(gamma_s) + i, reinterpret_cast<const float4*>(p.gamma) + i);
            sk_cp_async_16(reinterpret_cast<float4*>(beta_s) + i, reinterpret_cast<const float4*>(p.beta) + i);
        }
        sk_cp_async_wait_all();
        __syncthreads();
        const float inv_d = 1.f / (float)p.d;
        auto vec = [&](int r, int c) { return y_vec<N>(y_tiles, r, c); };
        for (int r = p.M + warp; r < N; r += kSkWarps)            // padding rows
            for (int c = lane; c < nvec; c += 32) *vec(r, c) = make_uint4(0, 0, 0, 0);
        if (nvec <= 256) {
            // Rows held in registers: one pass over shared memory, two rows at a time.
            for (int r = warp; r < p.M; r += 2 * kSkWarps) {
                const int rows[2] = {r, r + kSkWarps};
                const int live = 1 + (rows[1] < p.M);
                if (nvec <= 128) layer_norm_rows_in_regs<2, 4>(vec, rows, live, nvec, inv_d, p.ln_eps, gamma_s, beta_s, lane);
                else layer_norm_rows_in_regs<2, 8>(vec, rows, live, nvec, inv_d, p.ln_eps, gamma_s, beta_s, lane);
            }
        } else {
            for (int r = warp; r < p.M; r += kSkWarps) {
                float sum = 0.f;
                for (int c = lane; c < nvec; c += 32) sum += vec8_sum(*vec(r, c));
                const float mu = warp_sum(sum) * inv_d;
                float sq = 0.f;
                for (int c = lane; c < nvec; c += 32) sq = vec8_sqdev(*vec(r, c), mu, sq);
                const float rstd = 1.f / sqrtf(warp_sum(sq) * inv_d + p.ln_eps);
                for (int c = lane; c < nvec; c += 32) {
                    const float4* g4 = reinterpret_cast<const float4*>(gamma_s) + 2 * c;
                    const float4* b4 = reinterpret_cast<const float4*>(beta_s) + 2 * c;
                    uint4* v = vec(r, c);
                    *v = layer_norm_vec8(*v, mu, rstd, g4[0], g4[1], b4[0], b4[1]);
                }
            }
        }
        ptx::fence_proxy_async();                                 // y was written by threads, is read by the MMA
        __syncthreads();
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (continues the ring)
        if (lane == 0) {
            int armed = preloaded;
            for (int i = preloaded; i < total_loads; ++i) {
                const int stage = i % S;
                const uint32_t phase = (uint32_t)(i / S) & 1u;
                if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
                    if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                        p.ctrl->error_info = (1u << 24) | ((unsigned)stage << 16) | ((unsigned)i & 0xffffu);
                    *abort_flag = 1;
                    break;
                }
                const int tile = i / p.k_blocks, kb = i - tile * p.k_blocks;
                ptx::mbar_arrive_expect_tx(full_bar(stage), stage_tx);
                ptx::tma_load_2d(w_base + stage * kStageBytes, &tm_w, kb * kBK, r_begin + tile * p.box_rows,
                                 full_bar(stage));
                armed = i + 1;
            }
            if (*abort_flag) {
                // Let the copies still in flight land before the CTA gives its shared memory back.
                for (int i = max(0, armed - S); i < armed; ++i) {
                    const uint32_t par = (uint32_t)(i / S) & 1u;
                    for (uint32_t n = 0; n < (1u << 14) && !ptx::mbar_try_wait(full_bar(i % S), par); ++n) __nanosleep(100);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16_f32(kTileRows, N);
            bool ok = true;
            int i = 0;
            for (int tile = 0; ok && tile < n_tiles; ++tile) {
                const int buf = tile & 1;
                const uint32_t acc_phase = (uint32_t)(tile >> 1) & 1u;
                if (!ptx::mbar_wait(tempty_bar(buf), acc_phase ^ 1u, abort_flag)) {
                    if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                        p.ctrl->error_info = (2u << 24) | (0x80u << 16) | ((unsigned)tile & 0xffffu);
                    *abort_flag = 1;
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * N);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++i) {
                    const int stage = i % S;
                    const uint32_t phase = (uint32_t)(i / S) & 1u;
                    if (!ptx::mbar_wait(full_bar(stage), phase, abort_flag)) {
                        if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                            p.ctrl->error_info = (2u << 24) | ((unsigned)stage << 16) | ((unsigned)i & 0xffffu);
                        *abort_flag = 1;
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint64_t adesc = ptx::smem_desc_k128(w_base + stage * kStageBytes);
                    const uint64_t bdesc = ptx::smem_desc_k128(y_base + kb * (N * 128));
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)
                        ptx::mma_bf16_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    ptx::mma_commit(empty_bar(stage));            // the slot is free once the tensor core has read it
                }
                if (ok) ptx::mma_commit(tfull_bar(buf));
            }
            if (*abort_flag) {
                ptx::mma_commit(drain_bar);
                for (uint32_t n = 0; n < (1u << 16) && !ptx::mbar_try_wait(drain_bar, 0); ++n) __nanosleep(100);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2 ..)
        const int quarter = warp & 3;                             // TMEM lanes 32*quarter .. +31
        const int group = (warp - 2) >> 2;                        // tokens group*32 .. +TOK-1
        const int row_in_tile = quarter * 32 + lane;
        State own[TOK];
#pragma unroll
        for (int k = 0; k < TOK; ++k) own[k] = state_empty();
        for (int tile = 0; tile < n_tiles; ++tile) {
            const int buf = tile & 1;
            const uint32_t acc_phase = (uint32_t)(tile >> 1) & 1u;
            const bool landed = ptx::mbar_wait(tfull_bar(buf), acc_phase, abort_flag);
            if (!__all_sync(0xffffffffu, landed)) {
                if (lane == 0) {
                    if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                        p.ctrl->error_info = (3u << 24) | ((unsigned)buf << 16) | ((unsigned)tile & 0xffffu);
                    *abort_flag = 1;
                }
                break;
            }
            ptx::tc_fence_after_sync();
            const int row = r_begin + tile * p.box_rows + row_in_tile;       // this lane's vocabulary row
            const bool valid = row_in_tile < p.box_rows && row < r_end;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * N + group * 32);
#pragma unroll
            for (int c = 0; c < TOK / 16; ++c) {
                float v[16];
                ptx::tmem_ld_32x16(taddr + c * 16, v);
                ptx::tmem_ld_wait();
                if (valid) {
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj) state_push(own[c * 16 + jj], v[jj], row);
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(tempty_bar(buf));
        }
        // Transpose through shared memory (ring and y are no longer read: the last tile's MMAs have completed):
        // lane t then merges token t's 32 per-lane states in row order.
        State* stash = reinterpret_cast<State*>(smem) + (size_t)(warp - 2) * 32 * TOK;
#pragma unroll
        for (int k = 0; k < TOK; ++k) stash[lane * TOK + (k ^ (lane & (TOK - 1)))] = own[k];   // XOR spreads the banks
        __syncwarp();
        if (lane < TOK) {
            State a[4];                                           // four interleaved chains over the 32 rows
#pragma unroll
            for (int q = 0; q < 4; ++q) a[q] = stash[q * TOK + (lane ^ (q & (TOK - 1)))];
            for (int l = 4; l < 32; l += 4) {
#pragma unroll
                for (int q = 0; q < 4; ++q) state_merge(a[q], stash[(l + q) * TOK + (lane ^ ((l + q) & (TOK - 1)))]);
            }
            state_merge(a[0], a[1]);
            state_merge(a[2], a[3]);
            state_merge(a[0], a[2]);
            qpart[quarter * N + group * 32 + lane] = a[0];
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }

    // Merge the four quarters in vocabulary order; publish the CTA partial.
    if (threadIdx.x < N) {
        State a = qpart[threadIdx.x];
        for (int q = 1; q < 4; ++q) state_merge(a, qpart[q * N + threadIdx.x]);
        p.partials[(size_t)blockIdx.x * N + threadIdx.x] = a;
    }
    __syncthreads();
    if (threadIdx.x == 0) s_is_last = ticket_arrive_is_last(p.ctrl, gridDim.x);
    __syncthreads();
    if (!s_is_last) return;

    // Last CTA: merge the partials of all CTAs and decide (ring and y are free by now and serve as scratch).
    merge_partials_and_decide<kSkThreads>(p.partials, (int)gridDim.x, N, p.M, reinterpret_cast<State*>(smem),
                                          (size_t)S * kStageBytes + (size_t)p.k_blocks * N * 128, p.tau_per_row, p.tau,
                                          p.argmax, p.entropy, p.maxprob, p.exit_mask);
    if (threadIdx.x == 0) p.ctrl->ticket = 0;                     // ready for the next call
}

int pad_rows(int M) { return M <= 16 ? 16 : (M <= 32 ? 32 : 64); }

// Shared-memory bytes besides the W ring.
size_t skinny_fixed_bytes(int n, int d) {
    return (size_t)n * d * 2 + (size_t)2 * d * sizeof(float) + (size_t)4 * n * sizeof(State) +
           (size_t)(2 * kSkMaxStages + 6) * 8 + 1024;
}

int skinny_stages(int n, int d) {
    const long long room = (long long)kSkSmemBudget - (long long)skinny_fixed_bytes(n, d);
    long long s = room / kStageBytes;
    if (s > kSkMaxStages) s = kSkMaxStages;
    return s >= 4 ? (int)s : 0;
}

template <int N>
ee_status launch_skinny(const CUtensorMap& tm_w, const SkinnyParams& p, int grid, int device, cudaStream_t stream) {
    const size_t smem = skinny_fixed_bytes(N, p.d) + (size_t)p.n_stages * kStageBytes;
    static bool configured[kMaxDevices] = {};
    if (!configured[device]) {
        if (cudaFuncSetAttribute(exit_head_skinny_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSkSmemBudget) != cudaSuccess)
            return EE_ERR_CUDA;
        configured[device] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(sk_threads(N));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, exit_head_skinny_kernel<N>, tm_w, p) == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace

bool skinny_supports(int M, int d) {
    if (M < 1 || M > kSkinnyMaxRows || (d % 64) != 0) return false;
    return skinny_stages(pad_rows(M), d) > 0;
}

size_t skinny_workspace_bytes() { return (size_t)kStreamMaxCtas * kSkinnyMaxRows * sizeof(State); }

ee_status skinny_launch(const HeadArgs& a) {
    if (!skinny_supports(a.M, a.d)) return EE_ERR_SHAPE;
    const int n = pad_rows(a.M);
    const int grid = a.num_sms < kStreamMaxCtas ? a.num_sms : kStreamMaxCtas;
    unsigned char* ws = static_cast<unsigned char*>(a.workspace);

    SkinnyParams p;
    p.h = static_cast<const __nv_bfloat16*>(a.h);
    p.ld_h = a.ld_h;
    p.gamma = a.gamma;
    p.beta = a.beta;
    p.ln_eps = a.ln_eps;
    p.M = a.M;
    p.d = a.d;
    p.V = a.V;
    p.tau_per_row = a.tau_per_row;
    p.tau = a.tau;
    p.argmax = a.argmax;
    p.entropy = a.entropy;
    p.maxprob = a.maxprob;
    p.exit_mask = a.exit_mask;
    p.partials = reinterpret_cast<State*>(ws + kCtrlBytes);
    p.ctrl = reinterpret_cast<Control*>(ws);
    p.k_blocks = a.d / kBK;
    // Tile height: the CTA with the most rows splits them evenly over as few tiles of <= 128 rows as possible,
    // so that the last tile of a CTA reaches at most a few rows into its neighbour's range.
    const int rows_max = (a.V + grid - 1) / grid;
    const int tiles = (rows_max + kTileRows - 1) / kTileRows;
    int box = (rows_max + tiles - 1) / tiles;
    if (box > kTileRows) box = kTileRows;
    p.box_rows = box;
    p.n_stages = skinny_stages(n, a.d);

    CUtensorMap tm_w;
    if (!make_tile_map(&tm_w, a.W, a.V, a.d, box)) return EE_ERR_CUDA;
    if (n == 16) return launch_skinny<16>(tm_w, p, grid, a.device, a.stream);
    if (n == 32) return launch_skinny<32>(tm_w, p, grid, a.device, a.stream);
    return launch_skinny<64>(tm_w, p, grid, a.device, a.stream);
}

}  // namespace ee
