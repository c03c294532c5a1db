// Exit heads for 1 <= M <= 64 rows on the tcgen05 tensor cores: up to four heads in one launch, bound by the
// single read of their weights.
//
// Operands are swapped with respect to the large-M kernel: a tile of up to 128 vocabulary rows of W is the
// MMA's M-side operand (streamed from HBM by TMA into a shared-memory ring, 128-byte swizzle), and the N = 16 /
// 32 / 64 LayerNorm'ed activation rows are the N-side operand, resident in shared memory while their head is
// being evaluated (each CTA normalises them itself, writing the swizzled layout directly).  The MMAs are issued
// by one thread and cost the SM nothing else, so a ring slot is free again as soon as the tensor core has read
// it.  The accumulator [128 vocabulary rows x N tokens] lives in TMEM (two buffers).  Epilogue warps read it
// back with the vocabulary row on the lane; every thread keeps one online state per token (at most 32 tokens
// per thread: for N = 64 a second set of epilogue warps takes tokens 32..63), so a tile costs one state update
// per logit and no cross-lane traffic.
//
// Several heads in one launch keep HBM busy across the per-head latency chains: the TMA producer runs ahead
// into the next head's weights while the epilogue warps finish a head (cross-lane merge of the states, per-CTA
// partial, acquire-release ticket, and -- in the last CTA to arrive -- the final merge and the decision) and
// normalise the next head's activations (into a second buffer when shared memory allows, so that the tensor
// core never waits).  Waits between warps use mbarriers with bounded polling; nothing spins on another CTA.
#include "common.cuh"
#include "layer_norm.cuh"
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
constexpr int kSkMaxStages = 12;
constexpr size_t kSkSmemBudget = 227 * 1024;

struct SkinnyHead {
    const __nv_bfloat16* h;
    long long ld_h;
    const float* gamma;
    const float* beta;
    const float* tau_per_row;
    float tau;
    int* argmax;
    float* entropy;
    float* maxprob;
    unsigned char* exit_mask;
};

struct SkinnyParams {
    SkinnyHead head[kSkinnyMaxHeads];
    int n_heads;
    float ln_eps;
    int M, d, V;
    State* partials;                       // [n_heads][gridDim.x][N]
    Control* ctrl;
    int k_blocks;                          // d / 64
    int box_rows;                          // vocabulary rows per tile (<= 128), the TMA box height
    int n_stages;
    int stage_stride;                      // bytes between ring slots: box_rows * 128 rounded up to 1 KB
    int y_bufs;                            // 1 or 2 activation buffers
};

struct SkinnyMaps {
    CUtensorMap w[kSkinnyMaxHeads];
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

// LayerNorm of one head's M rows into the swizzled tiles at y_tiles, by `n_warps` whole warps (this one being
// number `w`).  `sync` is a barrier over exactly those warps; it returns false if the barrier gave up.
// A head's LayerNorm parameters into shared memory (asynchronous copies, completed by the wait in fill_activations).
// They are weights: for the first head of a launch this runs before the dependency wait.
__device__ __forceinline__ void fill_params(const SkinnyParams& p, const SkinnyHead& hd, float* gamma_s, float* beta_s, int t, int nt) {
    for (int i = t; i < (p.d >> 2); i += nt) {
        sk_cp_async_16(reinterpret_cast<float4*>(gamma_s) + i, reinterpret_cast<const float4*>(hd.gamma) + i);
        sk_cp_async_16(reinterpret_cast<float4*>(beta_s) + i, reinterpret_cast<const float4*>(hd.beta) + i);
    }
}

template <int N, class Sync>
__device__ __forceinline__ bool fill_activations(const SkinnyParams& p, const SkinnyHead& hd, unsigned char* y_tiles,
                                                 float* gamma_s, float* beta_s, int w, int n_warps, int lane, Sync sync,
                                                 bool params_on_their_way = false) {
    const int nvec = p.d >> 3;
    const int t = w * 32 + lane, nt = n_warps * 32;
    for (int i = t; i < p.M * nvec; i += nt) {
        const int r = i / nvec, c = i - r * nvec;
        sk_cp_async_16(y_vec<N>(y_tiles, r, c), reinterpret_cast<const uint4*>(hd.h + (size_t)r * hd.ld_h) + c);
    }
    if (!params_on_their_way) fill_params(p, hd, gamma_s, beta_s, t, nt);
    sk_cp_async_wait_all();
    if (!sync()) return false;
    auto vec = [&](int r, int c) { return y_vec<N>(y_tiles, r, c); };
    for (int r = p.M + w; r < N; r += n_warps)                    // padding rows
        for (int c = lane; c < nvec; c += 32) *vec(r, c) = make_uint4(0, 0, 0, 0);
    for (int r = w; r < p.M; r += 2 * n_warps) {                  // two rows at a time
        const int rows[2] = {r, r + n_warps};
        layer_norm_rows_in_smem<2>(vec, rows, 1 + (rows[1] < p.M), nvec, p.ln_eps, gamma_s, beta_s, lane);
    }
    ptx::fence_proxy_async();                                     // y was written by threads, is read by the MMA
    return true;
}

template <int N>
__global__ void __launch_bounds__(sk_threads(N), 1)
exit_head_skinny_kernel(const __grid_constant__ SkinnyMaps maps, const __grid_constant__ SkinnyParams p) {
    constexpr int TOK = N < 32 ? N : 32;                          // tokens per epilogue thread
    constexpr int GROUPS = sk_groups(N);
    constexpr int kSkThreads = sk_threads(N);
    constexpr int kSkWarps = kSkThreads / 32;
    constexpr int kEpiWarps = 4 * GROUPS;
    constexpr int kEpiThreads = 32 * kEpiWarps;
    constexpr int ACC = 4;                                        // accumulator buffers in TMEM
    constexpr int TMEM_COLS = ACC * N;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
    const int S = p.n_stages;
    const int y_bytes = p.k_blocks * N * 128;
    // layout: W stages | y buffers | gamma, beta | per-quarter states | barriers
    unsigned char* y_all = smem + (size_t)S * p.stage_stride;
    float* gamma_s = reinterpret_cast<float*>(y_all + (size_t)p.y_bufs * y_bytes);
    float* beta_s = gamma_s + p.d;
    State* qpart = reinterpret_cast<State*>(beta_s + p.d);       // [4][N]
    unsigned char* bar_mem = reinterpret_cast<unsigned char*>(qpart + 4 * N);
    const uint32_t w_base = ptx::smem_addr(smem);
    const uint32_t y_base = ptx::smem_addr(y_all);
    const uint32_t bar_base = ptx::smem_addr(bar_mem);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kSkMaxStages + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kSkMaxStages + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kSkMaxStages + 4 + b); };
    const uint32_t drain_bar = bar_base + 8u * (2 * kSkMaxStages + 8);
    auto yready_bar = [&](int b) { return bar_base + 8u * (2 * kSkMaxStages + 9 + b); };
    const uint32_t epi_bar = bar_base + 8u * (2 * kSkMaxStages + 11);         // barrier among the epilogue threads
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(bar_mem + 8 * (2 * kSkMaxStages + 12));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * kSkMaxStages + 12) + 4);
    volatile int* last_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * kSkMaxStages + 13));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    sk_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < ACC; ++b) {
            ptx::mbar_init(tfull_bar(b), 1);
            ptx::mbar_init(tempty_bar(b), kEpiWarps);
        }
        for (int b = 0; b < 2; ++b) ptx::mbar_init(yready_bar(b), kEpiWarps);
        ptx::mbar_init(drain_bar, 1);
        ptx::mbar_init(epi_bar, kEpiThreads);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        for (int k = 0; k < p.n_heads; ++k) ptx::prefetch_tensormap(&maps.w[k]);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    // This CTA's contiguous slice of the vocabulary, in tiles of box_rows rows; the same for every head.
    const int r_begin = (int)(((long long)p.V * blockIdx.x) / gridDim.x);
    const int r_end = (int)(((long long)p.V * (blockIdx.x + 1)) / gridDim.x);
    const int n_tiles = (r_end - r_begin + p.box_rows - 1) / p.box_rows;
    const int loads_per_head = n_tiles * p.k_blocks;
    const int total_loads = loads_per_head * p.n_heads;
    const uint32_t stage_tx = (uint32_t)p.box_rows * 128u;
    auto issue_load = [&](int i) {                                // load number i of the CTA into slot i % S
        const int k = i / loads_per_head, j = i - k * loads_per_head;
        const int tile = j / p.k_blocks, kb = j - tile * p.k_blocks;
        const int stage = i % S;
        ptx::mbar_arrive_expect_tx(full_bar(stage), stage_tx);
        ptx::tma_load_2d(w_base + stage * p.stage_stride, &maps.w[k], kb * kBK, r_begin + tile * p.box_rows, full_bar(stage));
    };

    // The weights do not depend on earlier kernels of the stream: fill the ring before waiting for them.
    int preloaded = 0;
    if (threadIdx.x == 0)
        for (; preloaded < total_loads && preloaded < S; ++preloaded) issue_load(preloaded);

    // Activations of the first head: all warps (its LayerNorm parameters are requested before the wait).
    fill_params(p, p.head[0], gamma_s, beta_s, (int)threadIdx.x, kSkThreads);
    sk_grid_dependency_wait();
    fill_activations<N>(p, p.head[0], y_all, gamma_s, beta_s, warp, kSkWarps, lane, [] { __syncthreads(); return true; }, true);
    __syncthreads();

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
                issue_load(i);
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
            int i = 0, t = 0;                                     // load and tile counters over all heads
            for (int k = 0; ok && k < p.n_heads; ++k) {
                const int yb = p.y_bufs == 2 ? (k & 1) : 0;
                if (k > 0) {
                    // Activations of head k are the use number `use` (from zero) of buffer yb by a head > 0.
                    const uint32_t use = (uint32_t)(p.y_bufs == 2 ? (k - 1) >> 1 : k - 1);
                    if (!ptx::mbar_wait(yready_bar(yb), use & 1u, abort_flag)) {
                        if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                            p.ctrl->error_info = (2u << 24) | (0x40u << 16) | (unsigned)k;
                        *abort_flag = 1;
                        break;
                    }
                }
                for (int tile = 0; ok && tile < n_tiles; ++tile, ++t) {
                    const int buf = t % ACC;
                    const uint32_t acc_phase = (uint32_t)(t / ACC) & 1u;
                    if (!ptx::mbar_wait(tempty_bar(buf), acc_phase ^ 1u, abort_flag)) {
                        if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                            p.ctrl->error_info = (2u << 24) | (0x80u << 16) | ((unsigned)t & 0xffffu);
                        *abort_flag = 1;
                        ok = false;
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
                        const uint64_t adesc = ptx::smem_desc_k128(w_base + stage * p.stage_stride);
                        const uint64_t bdesc = ptx::smem_desc_k128(y_base + yb * y_bytes + kb * (N * 128));
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk)
                            ptx::mma_bf16_ss(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
                        ptx::mma_commit(empty_bar(stage));        // the slot is free once the tensor core has read it
                    }
                    if (ok) ptx::mma_commit(tfull_bar(buf));
                }
            }
            if (*abort_flag) {
                ptx::mma_commit(drain_bar);
                for (uint32_t n = 0; n < (1u << 16) && !ptx::mbar_try_wait(drain_bar, 0); ++n) __nanosleep(100);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2 ..)
        const int ew = warp - 2;                                  // epilogue warp number
        const int quarter = warp & 3;                             // TMEM lanes 32*quarter .. +31
        const int group = ew >> 2;                                // tokens group*32 .. +TOK-1
        const int row_in_tile = quarter * 32 + lane;
        const int et = ew * 32 + lane;                            // epilogue thread number
        uint32_t epi_phase = 0;
        auto epi_sync = [&]() {                                   // bounded barrier over the epilogue threads
            ptx::mbar_arrive(epi_bar);
            const bool good = ptx::mbar_wait(epi_bar, epi_phase, abort_flag);
            epi_phase ^= 1u;
            if (!good) *abort_flag = 1;
            return good;
        };
        bool ok = true;
        int t = 0;                                                // tile counter over all heads
        for (int k = 0; ok && k < p.n_heads; ++k) {
            const SkinnyHead& hd = p.head[k];
            // With two buffers, head k+1's activations are prepared while head k's first tile is on its way.
            if (p.y_bufs == 2 && k + 1 < p.n_heads) {
                ok = fill_activations<N>(p, p.head[k + 1], y_all + ((k + 1) & 1) * y_bytes, gamma_s, beta_s, ew, kEpiWarps,
                                         lane, epi_sync);
                if (!ok) break;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(yready_bar((k + 1) & 1));
            }
            State own[TOK];
#pragma unroll
            for (int q = 0; q < TOK; ++q) own[q] = state_empty();
            for (int tile = 0; tile < n_tiles; ++tile, ++t) {
                const int buf = t % ACC;
                const uint32_t acc_phase = (uint32_t)(t / ACC) & 1u;
                const bool landed = ptx::mbar_wait(tfull_bar(buf), acc_phase, abort_flag);
                if (!__all_sync(0xffffffffu, landed)) {
                    if (lane == 0) {
                        if (atomicCAS(&p.ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
                            p.ctrl->error_info = (3u << 24) | ((unsigned)buf << 16) | ((unsigned)t & 0xffffu);
                        *abort_flag = 1;
                    }
                    ok = false;
                    break;
                }
                ptx::tc_fence_after_sync();
                const int row = r_begin + tile * p.box_rows + row_in_tile;   // this lane's vocabulary row
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
            if (!ok) break;
            // Cross-lane reduction of this warp's states: per token a warp maximum, then sums of rescaled terms.
#pragma unroll
            for (int c = 0; c < TOK; ++c) {
                if (group * 32 + c >= p.M) break;                 // padding tokens: nobody reads their states
                const State a = state_reduce_lanes<1, 16>(own[c]);
                if (lane == 0) qpart[quarter * N + group * 32 + c] = a;
            }
            // Head k's MMAs are complete.  With a single buffer the next head's activations are prepared now (the
            // per-thread states have just been handed over, which frees the registers LayerNorm needs).
            if (p.y_bufs == 1 && k + 1 < p.n_heads) {
                ok = fill_activations<N>(p, p.head[k + 1], y_all, gamma_s, beta_s, ew, kEpiWarps, lane, epi_sync);
                if (!ok) break;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(yready_bar(0));
            }
            if (!(ok = epi_sync())) break;
            // Merge the four quarters; publish the CTA partial of head k.
            State* part_k = p.partials + (size_t)k * gridDim.x * N;
            if (et < p.M) {
                const State four[4] = {qpart[et], qpart[N + et], qpart[2 * N + et], qpart[3 * N + et]};
                part_k[(size_t)blockIdx.x * N + et] = state_combine<4>(four);
            }
            if (!(ok = epi_sync())) break;
            if (et == 0) *last_flag = ticket_arrive_is_last(&p.ctrl->head_ticket[k], gridDim.x) ? 1 : 0;
            if (!(ok = epi_sync())) break;
            if (*last_flag) {
                // Last CTA to finish head k: merge the partials of all CTAs and decide.
                merge_tokens(part_k, false, (int)gridDim.x, N, p.M, ew, kEpiWarps, lane, hd.tau_per_row, hd.tau, hd.argmax,
                             hd.entropy, hd.maxprob, hd.exit_mask);
                if (et == 0) p.ctrl->head_ticket[k] = 0;          // ready for the next call
            }
            if (!(ok = epi_sync())) break;                        // qpart and last_flag are reused by the next head
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

int pad_rows(int M) { return M <= 16 ? 16 : (M <= 32 ? 32 : 64); }

// Shared-memory bytes besides the W ring, with `y_bufs` activation buffers.
size_t skinny_fixed_bytes(int n, int d, int y_bufs) {
    return (size_t)y_bufs * n * d * 2 + (size_t)2 * d * sizeof(float) + (size_t)4 * n * sizeof(State) +
           (size_t)(2 * kSkMaxStages + 16) * 8 + 1024;
}

int stage_stride_bytes(int box_rows) { return (box_rows * 128 + 1023) / 1024 * 1024; }

// Ring slots that fit; the MMA reads 128 rows from a slot, so the last slot needs a full 16 KB behind it.
int skinny_stages(int n, int d, int y_bufs, int box_rows) {
    const long long room = (long long)kSkSmemBudget - (long long)skinny_fixed_bytes(n, d, y_bufs) -
                           (kTileRows * 128 - stage_stride_bytes(box_rows));
    long long s = room / stage_stride_bytes(box_rows);
    if (s > kSkMaxStages) s = kSkMaxStages;
    return s >= 4 ? (int)s : 0;
}

template <int N>
ee_status launch_skinny(const SkinnyMaps& maps, const SkinnyParams& p, int grid, int device, cudaStream_t stream) {
    const size_t smem = skinny_fixed_bytes(N, p.d, p.y_bufs) + (size_t)p.n_stages * p.stage_stride +
                        (kTileRows * 128 - p.stage_stride);
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
    return cudaLaunchKernelEx(&cfg, exit_head_skinny_kernel<N>, maps, p) == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace

bool skinny_supports(int M, int d) {
    if (M < 1 || M > kSkinnyMaxRows || (d % 64) != 0) return false;
    return skinny_stages(pad_rows(M), d, 1, kTileRows) > 0;
}

size_t skinny_workspace_bytes(int n_heads) {
    return (size_t)n_heads * kStreamMaxCtas * kSkinnyMaxRows * sizeof(State);
}

ee_status skinny_launch(const HeadArgs* heads, int n_heads) {
    const HeadArgs& a = heads[0];
    if (n_heads < 1 || n_heads > kSkinnyMaxHeads || !skinny_supports(a.M, a.d)) return EE_ERR_SHAPE;
    const int n = pad_rows(a.M);
    const int grid = a.num_sms < kStreamMaxCtas ? a.num_sms : kStreamMaxCtas;
    unsigned char* ws = static_cast<unsigned char*>(a.workspace);

    SkinnyParams p;
    SkinnyMaps maps;
    // Tile height: the CTA with the most rows splits them evenly over as few tiles of <= 128 rows as possible,
    // so that the last tile of a CTA reaches at most a few rows into its neighbour's range.
    const int rows_max = (a.V + grid - 1) / grid;
    const int tiles = (rows_max + kTileRows - 1) / kTileRows;
    int box = (rows_max + tiles - 1) / tiles;
    if (box > kTileRows) box = kTileRows;
    for (int k = 0; k < n_heads; ++k) {
        const HeadArgs& h = heads[k];
        SkinnyHead& s = p.head[k];
        s.h = static_cast<const __nv_bfloat16*>(h.h);
        s.ld_h = h.ld_h;
        s.gamma = h.gamma;
        s.beta = h.beta;
        s.tau_per_row = h.tau_per_row;
        s.tau = h.tau;
        s.argmax = h.argmax;
        s.entropy = h.entropy;
        s.maxprob = h.maxprob;
        s.exit_mask = h.exit_mask;
        // W is streamed once, front to back: 256-byte promotion fetches the next k-block's half of the line pair too.
        if (!make_tile_map(&maps.w[k], h.W, a.V, a.d, box, CU_TENSOR_MAP_L2_PROMOTION_L2_256B)) return EE_ERR_CUDA;
    }
    for (int k = n_heads; k < kSkinnyMaxHeads; ++k) {
        p.head[k] = p.head[0];
        maps.w[k] = maps.w[0];
    }
    p.n_heads = n_heads;
    p.ln_eps = a.ln_eps;
    p.M = a.M;
    p.d = a.d;
    p.V = a.V;
    p.partials = reinterpret_cast<State*>(ws + kCtrlBytes);
    p.ctrl = reinterpret_cast<Control*>(ws);
    p.k_blocks = a.d / kBK;
    p.box_rows = box;
    // A second activation buffer (the next head is normalised while this one streams) if the ring keeps >= 6 slots.
    p.y_bufs = (n_heads > 1 && skinny_stages(n, a.d, 2, box) >= 6) ? 2 : 1;
    p.n_stages = skinny_stages(n, a.d, p.y_bufs, box);
    p.stage_stride = stage_stride_bytes(box);

    if (n == 16) return launch_skinny<16>(maps, p, grid, a.device, a.stream);
    if (n == 32) return launch_skinny<32>(maps, p, grid, a.device, a.stream);
    return launch_skinny<64>(maps, p, grid, a.device, a.stream);
}

}  // namespace ee
