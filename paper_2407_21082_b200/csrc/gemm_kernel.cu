// Verify/prefill-sized exit head: LayerNorm kernel -> persistent TMA + tcgen05 GEMM whose epilogue reduces
// every 128 x BN block of logits to per-row softmax states straight out of tensor memory -> merge kernel.
// The M x V logits are never written anywhere.  The three kernels are chained by programmatic dependent
// launch, and the GEMM requests its first weight tiles before it waits for the LayerNorm kernel.
//
// GEMM kernel, one CTA per SM, 320 threads:
//   warp 0 (one lane)  TMA producer: y tile [128 x 64] and W tile [BN x 64] per k-block into a smem ring
//   warp 1 (one lane)  tcgen05.mma issuer; accumulators [128 x BN] fp32 double-buffered in TMEM
//   warps 2..9         epilogue (two warps per quarter of the TMEM lanes, even / odd 32-column chunks):
//                      tcgen05.ld 32 columns at a time, thread = row, online softmax state,
//                      one 16-byte partial state per (row, vocabulary tile)
// All mbarrier waits are bounded; a wait that gives up records an error word, raises the CTA's abort
// flag, and every role drains to the common exit where TMEM is released.
#include <string.h>

#include "common.cuh"
#include "kernels.h"
#include "layer_norm.cuh"
#include "sm100_ptx.cuh"
#include "gemm_roles.cuh"
#include "tensor_map.h"

namespace ee {

namespace {

constexpr int BM = 128;
constexpr int BK = kRoleBK;
constexpr int kGemmThreads = 320;           // producer warp, MMA warp, eight epilogue warps
constexpr int kATileBytes = BM * BK * 2;    // 16 KB

constexpr int kBarBytes = 512 + 2048 + 1024;   // barriers and flags (512 B), then 128 states and 128 (max, second) pairs
                                               // exchanged between epilogue warps
constexpr int kGemmMaxHeads = kGemmLaunchMaxHeads;
constexpr int kMaxGemmStages = 12;
constexpr size_t kGemmSmemBudget = 226 * 1024;

// BN_T = 256: the tile width is a compile-time constant (large M).  BN_T = 0: the width comes from the
// parameters (any multiple of 16 up to 256), chosen so that the tiles fill whole waves of CTAs.
template <int BN_T>
struct Cfg {
    static constexpr int kStages = 4;
    static constexpr int kPairStages = 6;                             // a CTA of a pair stages half of the W tile
    static constexpr int kBTileBytes = 256 * BK * 2;
    static constexpr int kStageBytes = kATileBytes + kBTileBytes;
    static constexpr int kTmemCols = 512;                             // two accumulator buffers of 256 columns
    static constexpr int kSmemBytes = kStages * kStageBytes + kBarBytes + 1024;   // + slack to align to 1024
};

// One launch evaluates up to kGemmMaxHeads heads that share M, d and V: the tile list runs head by head.
struct GemmMaps {
    CUtensorMap y;                     // LayerNorm outputs of all heads, each padded to whole tiles: [n_heads * m_tiles * 128, d]
    CUtensorMap w[kGemmMaxHeads];      // each head's weights [V, d]
};

struct MergeHeads {
    const float* tau_per_row[kGemmMaxHeads];
    float tau[kGemmMaxHeads];
    int* argmax[kGemmMaxHeads];
    float* entropy[kGemmMaxHeads];
    float* maxprob[kGemmMaxHeads];
    unsigned char* exit_mask[kGemmMaxHeads];
    float* top2gap[kGemmMaxHeads];           // NULL unless the caller asked for the top-2 probability gap
};

// Largest and second-largest value of a multiset kept as a pair (equal maxima count twice).
__device__ __forceinline__ void top2_merge(float& m1, float& m2, float o1, float o2) {
    m2 = fmaxf(fmaxf(m2, o2), fminf(m1, o1));
    m1 = fmaxf(m1, o1);
}

// One warp: merge of the n_tiles partial states of one row (lane-strided, twelve independent loads at a
// time -- one round trip for up to 384 tiles -- then the lanes reduce).  `second` (NULL if not asked for) holds each
// tile's second-largest logit for this row: with the tiles' maxima it gives the row's largest and second-largest
// logit t1, t2, from which the gap of the two largest probabilities is (1 - e^(t2 - t1)) / s.
__device__ __forceinline__ State merge_row(const State* partials, const float* second, int n_tiles, int lane, float& t1,
                                           float& t2) {
    constexpr int kBatch = 12;
    State v[kBatch + 1];
    v[kBatch] = state_empty();                                    // running result of this lane
    t1 = t2 = -CUDART_INF_F;
    for (int n0 = lane; n0 < n_tiles; n0 += 32 * kBatch) {
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int n = n0 + 32 * i;
            v[i] = n < n_tiles ? state_load_cg(partials + n) : state_empty();
        }
        if (second) {
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int n = n0 + 32 * i;
                if (n < n_tiles) top2_merge(t1, t2, v[i].m, __ldcg(second + n));
            }
        }
        v[kBatch] = state_combine<kBatch + 1>(v);
    }
    const State a = state_reduce_lanes<1, 16>(v[kBatch]);
    if (second) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float o1 = __shfl_xor_sync(0xffffffffu, t1, o), o2 = __shfl_xor_sync(0xffffffffu, t2, o);
            top2_merge(t1, t2, o1, o2);
        }
    }
    return a;
}
// ... and the final decision for that row, written by lane 0.
__device__ __forceinline__ void decide_row(const State& a, float t1, float t2, bool with_top2, int head, int row,
                                           const MergeHeads& hs, int lane) {
    if (lane != 0) return;
    if (with_top2) hs.top2gap[head][row] = (1.f - expf(t2 - t1)) / a.s;
    state_finish(a, hs.tau_per_row[head] ? ld_dep(hs.tau_per_row[head] + row) : hs.tau[head], hs.argmax[head], hs.entropy[head],
                 hs.maxprob[head], hs.exit_mask[head], row);
}
__device__ __forceinline__ void merge_row_and_decide(const State* partials, const float* second, int n_tiles, int head, int row,
                                                     const MergeHeads& hs, int lane) {
    float t1, t2;
    const State a = merge_row(partials, second, n_tiles, lane, t1, t2);
    decide_row(a, t1, t2, second != nullptr, head, row, hs, lane);
}

struct GemmParams {
    int M, V, d;
    int m_tiles, n_tiles, k_blocks;
    int n_heads;
    State* partials;       // [head][M][n_tiles]
    float* second;         // [head][M][n_tiles]: each tile's second-largest logit, or NULL if nobody asked
    Control* ctrl;
    int bn;                // tile width (vocabulary rows per tile), a multiple of 16, <= 256
    int n_stages;          // smem ring depth
    int mma_m;             // rows of one MMA: 128, or 64 when no head has more than 64 rows (runtime width only)
    int fused_merge;       // the kernel merges the partial states itself (few rows; runtime width only)
    int k2;                // a stage holds two k-blocks, fetched by one request per operand (runtime width; d % 64 == 0)
    int merge_looks;       // how often a row group's owner looks at the ticket before it leaves its rows to the last arriver
    MergeHeads mg;
};

// Fold 32 consecutive logits of one row (columns col0 .. col0+31, the first `nvalid` of them real).
template <bool kFull>
__device__ __forceinline__ void fold_chunk(State& st, const float (&v)[32], int col0, int nvalid) {
    float cm = v[0];
#pragma unroll
    for (int j = 1; j < 32; ++j)
        if (kFull || j < nvalid) cm = fmaxf(cm, v[j]);
    if (cm > st.m) {
        int j0 = 0;
#pragma unroll
        for (int j = 31; j >= 0; --j)
            if ((kFull || j < nvalid) && v[j] == cm) j0 = j;
        const float dl = st.m - cm;
        const bool was_empty = (st.s == 0.f);
        const float al = was_empty ? 0.f : ex2(dl * kLog2e);
        st.t = was_empty ? 0.f : al * fmaf(dl, st.s, st.t);
        st.s = al * st.s;
        st.m = cm;
        st.idx = col0 + j0;
    }
    const float neg_m2 = -st.m * kLog2e;
    float s = 0.f, t2 = 0.f;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (kFull || j < nvalid) {
            const float a = fmaf(v[j], kLog2e, neg_m2);      // (z - m) * log2(e)
            const float e = ex2(a);
            s += e;
            t2 = fmaf(e, a, t2);
        }
    }
    st.s += s;
    st.t = fmaf(t2, kLn2, st.t);
}

// Largest and second-largest of 32 consecutive logits of one row (the first `nvalid` real); equal maxima count twice.
template <bool kFull>
__device__ __forceinline__ void chunk_top2(const float (&v)[32], int nvalid, float& c1, float& c2) {
    c1 = v[0];
#pragma unroll
    for (int j = 1; j < 32; ++j)
        if (kFull || j < nvalid) c1 = fmaxf(c1, v[j]);
    int dup = 0;
    c2 = -CUDART_INF_F;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (kFull || j < nvalid) {
            const bool eq = v[j] == c1;
            dup += eq ? 1 : 0;
            c2 = fmaxf(c2, eq ? -CUDART_INF_F : v[j]);
        }
    }
    if (dup > 1) c2 = c1;
}

// kTop2: also track the second-largest logit (for the top-2 probability gap); a separate instantiation, so
// that the default kernel carries none of its registers or branches.
// kPair: the grid is made of clusters of two CTAs and each pair works on 256-row tiles (row tiles 2u and 2u + 1 of
// a head): each CTA stages its own 128 rows of y and half of the W tile's rows, rank 0 issues 256 x BN MMAs
// that read both CTAs' shared memory, and every CTA folds its own 128 rows out of its own tensor memory.  A W
// tile then crosses L2 -> shared memory once per 256 rows instead of once per 128.
template <int BN_T, bool kTop2, bool kPair>
__global__ void __launch_bounds__(kGemmThreads, 1)
exit_head_gemm_kernel(const __grid_constant__ GemmMaps maps, const GemmParams p) {
    using C = Cfg<BN_T>;
    const int BN = BN_T ? BN_T : p.bn;
    const int S = BN_T ? (kPair ? (p.k2 ? C::kPairStages / 2 : C::kPairStages) : C::kStages) : p.n_stages;
    const uint32_t rank = kPair ? ptx::cluster_cta_rank() : 0u;
    const int worker = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;        // tiles go round the CTAs / the pairs
    const int n_workers = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int b_rows = kPair ? BN / 2 : BN;                                     // rows of W this CTA stages per k-block
    const int b_tile_bytes = b_rows * BK * 2;
    // With at most 64 rows per head the MMA is issued with M = 64: half the tensor work (and power) of a
    // 128-row MMA whose lower half would be padding, and an 8 KB instead of a 16 KB y tile per stage.
    const int mma_m = BN_T ? BM : p.mma_m;
    const int a_tile_bytes = mma_m * BK * 2;
    // A stage of the ring holds one k-block of both operands, or -- when three such stages fit: narrow tiles, and
    // pairs at any width -- two.  A pair's CTAs each stage half a W tile, boxes of at most 128 rows, and requests that small stream
    // from HBM at 5.4 TB/s where one request for two k-blocks (256 bytes of every row) reaches the rate of a
    // contiguous copy; it also halves the requests and the barrier traffic per k-block, which is what a small head
    // gains from it (d = 512, 8 rows: 17.5 -> 16.8 us per call).
    constexpr bool kCanK2 = BN_T == 0 || kPair;
    const int kbs = (kCanK2 && p.k2) ? 2 : 1;                     // k-blocks per stage
    const int n_steps = (p.k_blocks + kbs - 1) / kbs;             // stages per tile
    const int a_stage_bytes = kbs * a_tile_bytes, b_stage_bytes = kbs * b_tile_bytes;
    const int stage_bytes = a_stage_bytes + b_stage_bytes;
    constexpr int kAccStride = 256;                               // TMEM columns between the two accumulators
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
    const uint32_t a_base = ptx::smem_addr(smem);
    const uint32_t b_base = a_base + S * a_stage_bytes;
    unsigned char* bar_mem = smem + S * stage_bytes;
    const uint32_t bar_base = ptx::smem_addr(bar_mem);
    // barrier slots (8 bytes each): full[S], empty[S], tmem_full[2], tmem_empty[2], drain
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * S + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * S + 2 + b); };
    const uint32_t drain_bar = bar_base + 8u * (2 * S + 4);
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(bar_mem + 8 * (2 * S + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * S + 5) + 4);
    // per quarter of the TMEM lanes: "state of the odd chunks is in the exchange slot" / "slot has been read"
    auto xfull_bar = [&](int q) { return bar_base + 8u * (2 * S + 6 + q); };
    auto xfree_bar = [&](int q) { return bar_base + 8u * (2 * S + 10 + q); };

    const int total_rows = p.n_heads * p.M;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // The runtime-width variant (launches of tens of microseconds) lets its dependents start at once; their few
    // CTAs wait beside this one.  The 256-wide variant runs for milliseconds and its merge has thousands of
    // CTAs: resident and waiting they cost it about a tenth of its speed, so it triggers them only when a CTA
    // starts its last tile (see the producer).
    if (BN_T == 0) launch_dependents();

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull_bar(b), 1);
            ptx::mbar_init(tempty_bar(b), (BN_T ? 4 : 8) * (kPair ? 2 : 1));   // a pair's epilogue warps all report to rank 0
        }
        for (int q = 0; q < 4; ++q) {
            ptx::mbar_init(xfull_bar(q), 1);
            ptx::mbar_init(xfree_bar(q), 1);
        }
        ptx::mbar_init(drain_bar, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&maps.y);
        for (int k = 0; k < p.n_heads; ++k) ptx::prefetch_tensormap(&maps.w[k]);
    }
    if (warp == 1) {
        if (kPair) {
            ptx::tmem_alloc_pair(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), C::kTmemCols);
            ptx::tmem_relinquish_pair();
        } else {
            ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), C::kTmemCols);
            ptx::tmem_relinquish();
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (kPair) ptx::cluster_sync_all();                   // the partner's barriers exist before anything signals them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    const int m_units = kPair ? p.m_tiles >> 1 : p.m_tiles;     // row tiles, or pairs of row tiles
    const int tiles_per_head = m_units * p.n_tiles;
    const int total_tiles = p.n_heads * tiles_per_head;
    // tile -> (head, m_tile, n_tile); within a head the order keeps concurrent CTAs on the same W tiles
    auto locate = [&](int tile, int& head, int& m_tile, int& n_tile) {
        head = tile / tiles_per_head;
        tile_coords(tile - head * tiles_per_head, m_units, p.n_tiles, m_tile, n_tile);
        if (kPair) m_tile = 2 * m_tile + (int)rank;
    };
    // Where a stage's loads report their bytes (rank 0's barrier) and how they are issued.
    auto load_full_bar = [&](int s) { return kPair ? ptx::map_to_cta(full_bar(s), 0) : full_bar(s); };
    auto load_tile = [&](uint32_t dst, const CUtensorMap* m, int step, int row, uint32_t bar) {   // the k-block(s) of stage `step`
        if (kCanK2 && kbs == 2) {
            if (kPair) ptx::tma_load_3d_pair(dst, m, 0, row, 2 * step, bar);
            else ptx::tma_load_3d(dst, m, 0, row, 2 * step, bar);
        }
        else if (kPair) ptx::tma_load_2d_pair(dst, m, step * BK, row, bar);
        else ptx::tma_load_2d(dst, m, step * BK, row, bar);
    };
    const uint32_t arm_bytes = (uint32_t)stage_bytes * (kPair ? 2u : 1u);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0, armed = 0, armed_parity = 0;
            bool ok = true;
            // The weights do not depend on earlier kernels of the stream: the W tiles of the first stages are
            // requested before the dependency wait, the y tiles (written by the LayerNorm kernel) after it.
            int n_pre = 0;
            if (worker < total_tiles) {
                int head, m_tile, n_tile;
                locate(worker, head, m_tile, n_tile);
                n_pre = min(S, n_steps);
                for (int kb = 0; kb < n_pre; ++kb) {
                    if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(kb), arm_bytes);
                    load_tile(b_base + kb * b_stage_bytes, &maps.w[head], kb, n_tile * BN + (int)rank * b_rows, load_full_bar(kb));
                    armed |= 1u << kb;
                }
            }
            grid_dependency_wait();
            int issued = 0;
            for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
                int head, m_tile, n_tile;
                locate(tile, head, m_tile, n_tile);
                const int y_row = (head * p.m_tiles + m_tile) * BM;   // each head's rows are padded to whole tiles
                if (BN_T != 0 && tile + n_workers >= total_tiles) launch_dependents();
                for (int kb = 0; kb < n_steps; ++kb, ++issued) {
                    if (issued < n_pre) {                 // stage `issued`, armed above, W tile on its way
                        load_tile(a_base + stage * a_stage_bytes, &maps.y, kb, y_row, load_full_bar(stage));
                        if (++stage == S) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) {
                        record_failure(p.ctrl, abort_flag, 1, stage, tile);
                        ok = false;
                        break;
                    }
                    if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(stage), arm_bytes);
                    load_tile(a_base + stage * a_stage_bytes, &maps.y, kb, y_row, load_full_bar(stage));
                    load_tile(b_base + stage * b_stage_bytes, &maps.w[head], kb, n_tile * BN + (int)rank * b_rows, load_full_bar(stage));
                    armed |= 1u << stage;
                    armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
            if (*abort_flag) producer_drain(rank, S, full_bar(0), armed, armed_parity);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = ptx::idesc_bf16_f32(kPair ? 2 * BM : mma_m, BN);
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            bool ok = true;
            for (int tile = worker; ok && tile < total_tiles; tile += n_workers, ++local) {
                const int buf = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1u;
                if (!ptx::mbar_wait(tempty_bar(buf), acc_phase ^ 1u, abort_flag)) {
                    record_failure(p.ctrl, abort_flag, 2, 0x80 | buf, tile);
                    break;
                }
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kAccStride);
                for (int kb = 0; kb < n_steps; ++kb) {
                    // with two k-blocks in a stage the second one is absent at the end of an odd number of them
                    const bool two = kCanK2 && kbs == 2 && 2 * kb + 1 < p.k_blocks;
                    if (!mma_k_block<kPair>(full_bar(stage), phase, empty_bar(stage), a_base + stage * a_stage_bytes,
                                            b_base + stage * b_stage_bytes, d_tmem, idesc, kb == 0, abort_flag,
                                            two ? (uint32_t)a_tile_bytes : 0u, (uint32_t)b_tile_bytes)) {
                        record_failure(p.ctrl, abort_flag, 2, stage, tile);
                        ok = false;
                        break;
                    }
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (ok) mma_commit_all<kPair>(tfull_bar(buf));    // accumulator complete
            }
            if (*abort_flag) mma_drain<kPair>(drain_bar);
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9)
        // Two warps share each quarter of the TMEM lanes: one folds the even 32-column chunks of a tile, the
        // other the odd ones, and the first adds the second's state to its own before it stores the partial.
        const int quarter = warp & 3;                     // TMEM lanes 32*quarter .. +31 belong to this warp
        // (The compile-time 256-wide variant is tensor-bound and its epilogue hides behind the next tile's MMAs:
        // there one warp per quarter folds all chunks and the other four warps stay out of the way.)
        constexpr bool kSplit = BN_T == 0;
        const int half = (warp - 2) >> 2;
        State* xchg = reinterpret_cast<State*>(bar_mem + 512) + quarter * 32 + lane;
        float2* xchg2 = reinterpret_cast<float2*>(bar_mem + 512 + 2048) + quarter * 32 + lane;
        constexpr bool want_top2 = kTop2;
        // M = 128: accumulator row i sits in lane i.  M = 64: rows 16q .. 16q+15 sit in the first 16 lanes of
        // quarter q, the other 16 lanes hold nothing.
        const int row_in_tile = mma_m == 64 ? (lane < 16 ? quarter * 16 + lane : BM) : quarter * 32 + lane;
        int local = 0;
        grid_dependency_wait();                           // the partial states may still be read by an earlier merge
        for (int tile = worker; (kSplit || half == 0) && tile < total_tiles; tile += n_workers, ++local) {
            int head, m_tile, n_tile;
            locate(tile, head, m_tile, n_tile);
            const int buf = local & 1;
            const uint32_t acc_phase = (local >> 1) & 1u;
            const bool landed = ptx::mbar_wait(tfull_bar(buf), acc_phase, abort_flag);
            if (!__all_sync(0xffffffffu, landed)) {       // also reconverges the warp for the aligned TMEM loads
                if (lane == 0) record_failure(p.ctrl, abort_flag, 3, buf, tile);
                break;
            }
            ptx::tc_fence_after_sync();
            const int n0 = n_tile * BN;
            const int ncols = min(BN, p.V - n0);
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * kAccStride);
            State st = state_empty();
            float z1 = -CUDART_INF_F, z2 = -CUDART_INF_F;     // largest and second-largest logit seen (only if asked for)
            const int row = m_tile * BM + row_in_tile;
            const bool live = row < p.M;                  // padding rows are neither read nor folded
            if (__any_sync(0xffffffffu, live)) {
                for (int c = kSplit ? half : 0; c * 32 < ncols; c += kSplit ? 2 : 1) {
                    float v[32];
                    ptx::tmem_ld_32x32(taddr + c * 32, v);
                    ptx::tmem_ld_wait();
                    const int nvalid = ncols - c * 32;
                    if (live) {
                        if (nvalid >= 32) fold_chunk<true>(st, v, n0 + c * 32, 32);
                        else fold_chunk<false>(st, v, n0 + c * 32, nvalid);
                        if constexpr (want_top2) {
                            float c1, c2;
                            if (nvalid >= 32) chunk_top2<true>(v, 32, c1, c2);
                            else chunk_top2<false>(v, nvalid, c1, c2);
                            top2_merge(z1, z2, c1, c2);
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (kPair) ptx::mbar_arrive_remote(ptx::map_to_cta(tempty_bar(buf), 0));
                else ptx::mbar_arrive(tempty_bar(buf));
            }
            const uint32_t x_phase = (uint32_t)local & 1u;
            if (!kSplit) {
                if (live) {
                    p.partials[((size_t)head * p.M + row) * p.n_tiles + n_tile] = st;
                    if constexpr (want_top2) p.second[((size_t)head * p.M + row) * p.n_tiles + n_tile] = z2;
                }
            } else if (half == 1) {
                // the slot is free once the partner has read the state of the tile before
                const bool free_ = local == 0 || ptx::mbar_wait(xfree_bar(quarter), x_phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, free_)) {
                    if (lane == 0) record_failure(p.ctrl, abort_flag, 5, quarter, tile);
                    break;
                }
                *xchg = st;
                if constexpr (want_top2) *xchg2 = make_float2(z1, z2);
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(xfull_bar(quarter));
            } else {
                const bool there = ptx::mbar_wait(xfull_bar(quarter), x_phase, abort_flag);
                if (!__all_sync(0xffffffffu, there)) {
                    if (lane == 0) record_failure(p.ctrl, abort_flag, 6, quarter, tile);
                    break;
                }
                const State other = *xchg;
                float2 other2 = make_float2(0.f, 0.f);
                if constexpr (want_top2) other2 = *xchg2;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(xfree_bar(quarter));
                if (live) {
                    state_merge(st, other);
                    if constexpr (want_top2) top2_merge(z1, z2, other2.x, other2.y);
                    p.partials[((size_t)head * p.M + row) * p.n_tiles + n_tile] = st;
                    if constexpr (want_top2) p.second[((size_t)head * p.M + row) * p.n_tiles + n_tile] = z2;
                }
            }
        }
        if (kSplit && p.fused_merge) {
            // With few rows the merge runs here instead of in a kernel of its own (one launch boundary less per
            // call).  Every CTA has stored its tiles' states and takes a ticket.  The rows are dealt out in groups
            // (group g: rows 8g + w for epilogue warp w, stepping by 8 * groups) to the first CTAs of the grid, which
            // also carry the most tiles and so finish among the last.  An owner looks at the ticket for a bounded
            // time and, once every CTA has published, merges its group: no further atomic on that path.  An owner
            // whose looks run out says so (a bit in merge_abandon) and leaves; the LAST arriver, whoever it is,
            // takes and merges every group so marked.  So the call completes whether or not the owners were still
            // around -- no CTA's progress depends on another CTA being scheduled, and an owner that stops looking
            // loses nothing but its share of the work.
            // An owner that gives up just as the last ticket is taken: it sets its bit, fences, and looks once more;
            // the last arriver takes its ticket, fences, and reads the bits (sequentially consistent fences: at
            // least one of the two sees the other).  If the owner's last look finds the count full, both may want
            // the group, and two bits in one word decide: the owner sets CLAIM, the last arriver TAKEN, each with an
            // atomic OR that shows it the other's bit; whoever finds the other's bit already there leaves the group
            // to the other.  Ticket and bits are zeroed by the next call's LayerNorm kernel (which starts after
            // this kernel has completed).
            // The barrier orders the epilogue threads' stores before one thread's acquire-release ticket, which is
            // cumulative: whoever sees the full count sees every CTA's states.  A CTA whose roles gave up still
            // takes its ticket (its tiles' states are missing, the error word says so).
            const int kMergeLooks = p.merge_looks;
            const int et = (warp - 2) * 32 + lane;
            const int grid = (int)gridDim.x;
            const int n_groups = min(grid, (total_rows + 7) >> 3);
            const int group = (int)blockIdx.x < n_groups ? (int)blockIdx.x : -1;
            volatile int* slot = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * S + 14));     // three words
            const bool with_top2 = kTop2 && p.second != nullptr;
            auto merge_group = [&](int g) {
                for (int r = g * 8 + (warp - 2); r < total_rows; r += 8 * n_groups) {
                    const int head = r / p.M;
                    merge_row_and_decide(p.partials + (size_t)r * p.n_tiles, with_top2 ? p.second + (size_t)r * p.n_tiles : nullptr,
                                         p.n_tiles, head, r - head * p.M, p.mg, lane);
                }
            };
            auto look = [&]() {
                unsigned int v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(&p.ctrl->ticket) : "memory");
                return v >= (unsigned)grid;
            };
            auto atom_or = [&](unsigned int* word, unsigned int bits) {
                unsigned int old;
                asm volatile("atom.acq_rel.gpu.global.or.b32 %0, [%1], %2;" : "=r"(old) : "l"(word), "r"(bits) : "memory");
                return old;
            };
            constexpr unsigned int kClaim = 1u, kTaken = 2u;          // two bits per group in merge_pair_bits
            asm volatile("bar.sync 1, 256;" ::: "memory");            // the eight epilogue warps, whatever path they took
            unsigned int arrival = 0;                                 // looked at only after the owner's work: the
            if (et == 0)                                              // ticket's round trip is off the owners' path
                asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(arrival) : "l"(&p.ctrl->ticket) : "memory");
            if (group >= 0) {
                if (et == 0) {
                    bool mine = false;
                    for (int i = 0; !mine && i < kMergeLooks; ++i) {
                        mine = look();
                        if (!mine && i >= 8) __nanosleep(i < 32 ? 100 : 1000);
                    }
                    if (!mine) {
                        atom_or(&p.ctrl->merge_abandon[group >> 5], 1u << (group & 31));
                        asm volatile("fence.sc.gpu;" ::: "memory");
                        if (look()) {                                 // the last ticket came in meanwhile
                            const int sh = 2 * (group & 15);
                            mine = ((atom_or(&p.ctrl->merge_pair_bits[group >> 4], kClaim << sh) >> sh) & kTaken) == 0;
                        }
                    }
                    slot[1] = mine ? 1 : 0;
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (slot[1]) merge_group(group);
            }
            if (et == 0) slot[2] = arrival == (unsigned)grid - 1u ? 1 : 0;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (slot[2]) {
                // The last arriver: the groups whose owners have stopped looking.
                if (et < 2) {
                    asm volatile("fence.sc.gpu;" ::: "memory");
                    unsigned int left;
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(left) : "l"(&p.ctrl->merge_abandon[et]) : "memory");
                    unsigned int won = 0;
                    for (unsigned int rest = left; rest; rest &= rest - 1) {
                        const int g = 32 * et + __ffs(rest) - 1;
                        const int sh = 2 * (g & 15);
                        if (((atom_or(&p.ctrl->merge_pair_bits[g >> 4], kTaken << sh) >> sh) & kClaim) == 0) won |= 1u << (g & 31);
                    }
                    slot[et] = (int)won;
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                for (int w2 = 0; w2 < 2; ++w2)
                    for (unsigned int won = (unsigned int)slot[w2]; won; won &= won - 1) merge_group(32 * w2 + __ffs(won) - 1);
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    // Neither CTA of a pair leaves, or gives its tensor memory back, while the other may still signal its
    // barriers, read its shared memory or write its accumulators.
    if (kPair) ptx::cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        ptx::tc_fence_after_sync();
        if (kPair) ptx::tmem_dealloc_pair(tmem_base, C::kTmemCols);
        else ptx::tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ---------------------------------------------------------------------------------------------
// LayerNorm of every head's input: h_k [M, d] (row stride ld_h) -> y [k][M, d] bf16, one warp per row,
// blockIdx.y = head.  With VPL > 0 (rows of up to 1024 columns) the row stays in registers (VPL 16-byte vectors per
// lane, d <= 256 * VPL) and is read once; VPL = 0 (rows beyond 4096 columns) re-reads it from global memory per
// pass.  No shared memory and few enough registers that a CTA fits on an SM beside a CTA of the call before (which
// holds nearly all of the shared memory) and is resident, its parameters fetched, when that call completes.
// ---------------------------------------------------------------------------------------------
// The first kernel of every call zeroes the counters of the in-kernel merge (it passes its dependency wait only
// after the call before has completed, so nobody is looking at them).
__device__ __forceinline__ void reset_merge_counters(Control* ctrl) {
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        ctrl->ticket = 0;
        ctrl->merge_abandon[0] = ctrl->merge_abandon[1] = 0;
        ctrl->merge_pair_bits[0] = ctrl->merge_pair_bits[1] = ctrl->merge_pair_bits[2] = ctrl->merge_pair_bits[3] = 0;
    }
}

struct LnHeads {
    const __nv_bfloat16* h[kGemmMaxHeads];
    long long ld_h[kGemmMaxHeads];
    const float* gamma[kGemmMaxHeads];
    const float* beta[kGemmMaxHeads];
};

// Threads per CTA: four warps when the rows are held in registers; a CTA then stays under 24 K registers, what an SM
// has left beside a CTA of the GEMM kernel.
__host__ __device__ constexpr int ln_threads(int vpl) { return vpl > 0 ? 128 : 256; }

template <int VPL>
__global__ void __launch_bounds__(ln_threads(VPL), 3)
layer_norm_rows_kernel(const __grid_constant__ LnHeads hs, float ln_eps, __nv_bfloat16* __restrict__ y_all, int M, int d,
                       Control* ctrl) {
    launch_dependents();
    const int row = blockIdx.x * (ln_threads(VPL) / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int head = blockIdx.y;
    const int m_pad = (M + BM - 1) / BM * BM;            // a head's rows are padded to whole 128-row tiles
    const int nvec = d >> 3;
    const float* gamma = hs.gamma[head];
    const float* beta = hs.beta[head];
    // The LayerNorm parameters are weights, not results of an earlier kernel: they are fetched before the wait, into
    // registers (sixteen per vector), because a load from L2 after it costs about a microsecond while the next
    // call's weight stream is running.
    float4 g[VPL > 0 ? VPL : 1][2], b[VPL > 0 ? VPL : 1][2];
    if (row >= m_pad) return;
    uint4* yrow = reinterpret_cast<uint4*>(y_all + ((size_t)head * m_pad + row) * d);
    if (row >= M) {
        // Padding row: zeros, so that the rows of a tile that carry no token cost the tensor pipe no switching.
        grid_dependency_wait();
        reset_merge_counters(ctrl);
        for (int c = lane; c < nvec; c += 32) yrow[c] = make_uint4(0, 0, 0, 0);
        return;
    }
    const uint4* hrow = reinterpret_cast<const uint4*>(hs.h[head] + (size_t)row * hs.ld_h[head]);
    if constexpr (VPL > 0) {
        const double dd = (double)d, inv_d = 1.0 / dd;       // a division: some thirty dependent operations, done before the wait
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            const int c = lane + 32 * k;
            if (c < nvec) {
                g[k][0] = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * c);
                g[k][1] = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * c + 1);
                b[k][0] = __ldg(reinterpret_cast<const float4*>(beta) + 2 * c);
                b[k][1] = __ldg(reinterpret_cast<const float4*>(beta) + 2 * c + 1);
            }
        }
        // h may be an earlier kernel's output, so it is read after the wait; asking L2 for its lines before
        // the wait is harmless (L2 is the point of coherence) and hides a DRAM round trip when h is not cached.
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            const int c = lane + 32 * k;
            if (c < nvec && (c & 7) == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(hrow + c));
        }
        grid_dependency_wait();                          // y may still be read by the GEMM of the call before
        reset_merge_counters(ctrl);
        uint4 x[VPL];
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            const int c = lane + 32 * k;
            x[k] = c < nvec ? ld_dep(hrow + c) : make_uint4(0, 0, 0, 0);
        }
        Moments m;
        m.clear();
#pragma unroll
        for (int k = 0; k < VPL; ++k) m.add(x[k], k);                     // vectors beyond the row are zero
        double s = m.sum(), q = m.sum_sq();
        warp_sum2_d(s, q);
        double mu, var;
        if (!row_variance_one_pass(s, q, dd, inv_d, mu, var)) {
            double q0 = 0.0, q1 = 0.0;
#pragma unroll
            for (int k = 0; k < VPL; ++k)
                if (lane + 32 * k < nvec) vec8_sqdev_d(x[k], mu, q0, q1);
            var = warp_sum_d(q0 + q1) * inv_d;
        }
        const RowStats st = row_stats(mu, var, ln_eps);
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            const int c = lane + 32 * k;
            if (c < nvec) yrow[c] = layer_norm_vec8(x[k], st, g[k][0], g[k][1], b[k][0], b[k][1]);
        }
    } else {
        grid_dependency_wait();
        reset_merge_counters(ctrl);
        const RowStats st = row_stats_strided([&](int c) { return ld_dep(hrow + c); }, nvec, ln_eps, lane);
        for (int c = lane; c < nvec; c += 32) yrow[c] = layer_norm_vec8(ld_dep(hrow + c), st, gamma, beta, c);
    }
}

// Rows wider than 1024 columns: one CTA of four warps per row, VPL 16-byte vectors per thread (d <= 1024 * VPL), so
// that a row's work -- 64 and more elements per lane if one warp took it -- is a quarter as long.  The warps' moments
// meet in shared memory (64 bytes; summed in a fixed order).  Parameters in registers, fetched before the wait.
// kLean (batches of thousands of rows, where the launch is bound by memory and not by a dependent chain): the
// parameters are read where they are used instead (they stay in L1), which halves the registers and lets six CTAs
// share an SM (five with four vectors per thread) instead of three -- enough rows in flight to cover the memory latency.
template <int VPL, bool kLean>
__global__ void __launch_bounds__(128, kLean ? (VPL == 4 ? 5 : 6) : 3)
layer_norm_wide_rows_kernel(const __grid_constant__ LnHeads hs, float ln_eps, __nv_bfloat16* __restrict__ y_all, int M, int d,
                            Control* ctrl) {
    __shared__ double part[2][4][2];
    launch_dependents();
    const int row = blockIdx.x, head = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m_pad = (M + BM - 1) / BM * BM;
    const int nvec = d >> 3;
    uint4* yrow = reinterpret_cast<uint4*>(y_all + ((size_t)head * m_pad + row) * d);
    if (row >= M) {                                      // padding row (the whole CTA)
        grid_dependency_wait();
        for (int c = tid; c < nvec; c += 128) yrow[c] = make_uint4(0, 0, 0, 0);
        return;
    }
    const uint4* hrow = reinterpret_cast<const uint4*>(hs.h[head] + (size_t)row * hs.ld_h[head]);
    const float* gamma = hs.gamma[head];
    const float* beta = hs.beta[head];
    const double dd = (double)d, inv_d = 1.0 / dd;
    float4 g[kLean ? 1 : VPL][2], b[kLean ? 1 : VPL][2];
#pragma unroll
    for (int k = 0; k < (kLean ? 0 : VPL); ++k) {
        const int c = tid + 128 * k;
        if (c < nvec) {
            g[k][0] = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * c);
            g[k][1] = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * c + 1);
            b[k][0] = __ldg(reinterpret_cast<const float4*>(beta) + 2 * c);
            b[k][1] = __ldg(reinterpret_cast<const float4*>(beta) + 2 * c + 1);
            if ((c & 7) == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(hrow + c));
        }
    }
    grid_dependency_wait();                              // y may still be read by the GEMM of the call before
    reset_merge_counters(ctrl);
    uint4 x[VPL];
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int c = tid + 128 * k;
        x[k] = c < nvec ? ld_dep(hrow + c) : make_uint4(0, 0, 0, 0);
    }
    Moments m;
    m.clear();
#pragma unroll
    for (int k = 0; k < VPL; ++k) m.add(x[k], k);
    double s = m.sum(), q = m.sum_sq();
    warp_sum2_d(s, q);
    if (lane == 0) { part[0][warp][0] = s; part[0][warp][1] = q; }
    __syncthreads();
    s = (part[0][0][0] + part[0][1][0]) + (part[0][2][0] + part[0][3][0]);
    q = (part[0][0][1] + part[0][1][1]) + (part[0][2][1] + part[0][3][1]);
    double mu, var;
    if (!row_variance_one_pass(s, q, dd, inv_d, mu, var)) {          // the same decision in every thread of the CTA
        double q0 = 0.0, q1 = 0.0;
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (tid + 128 * k < nvec) vec8_sqdev_d(x[k], mu, q0, q1);
        q0 = warp_sum_d(q0 + q1);
        if (lane == 0) part[1][warp][0] = q0;
        __syncthreads();
        var = ((part[1][0][0] + part[1][1][0]) + (part[1][2][0] + part[1][3][0])) * inv_d;
    }
    const RowStats st = row_stats(mu, var, ln_eps);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int c = tid + 128 * k;
        if (c < nvec) {
            if constexpr (kLean) yrow[c] = layer_norm_vec8(x[k], st, gamma, beta, c);
            else yrow[c] = layer_norm_vec8(x[k], st, g[k][0], g[k][1], b[k][0], b[k][1]);
        }
    }
}

// LayerNorm of a gathered subset of one head's rows: output row j = LayerNorm(h[row_idx[j]]) for j < *m_dev,
// zeros from there to the end of the padded tile rows.  The list and the count come from an earlier kernel of
// the stream (the cascade of heads), so everything is read after the dependency wait.  Warp per row.
__global__ void __launch_bounds__(256) layer_norm_gather_kernel(const __nv_bfloat16* h, long long ld_h,
                                                                const float* __restrict__ gamma,
                                                                const float* __restrict__ beta, float ln_eps,
                                                                const int* row_idx, const int* m_dev,
                                                                __nv_bfloat16* y, int M, int d, Control* ctrl) {
    launch_dependents();
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int m_pad = (M + BM - 1) / BM * BM;
    if (row >= m_pad) return;
    const int nvec = d >> 3;
    uint4* yrow = reinterpret_cast<uint4*>(y + (size_t)row * d);
    grid_dependency_wait();
        reset_merge_counters(ctrl);
    const int m_live = m_dev ? min(max(ld_dep(m_dev), 0), M) : M;
    if (row >= m_live) {
        for (int c = lane; c < nvec; c += 32) yrow[c] = make_uint4(0, 0, 0, 0);
        return;
    }
    const int src = row_idx ? ld_dep(row_idx + row) : row;
    const uint4* hrow = reinterpret_cast<const uint4*>(h + (size_t)src * ld_h);
    const RowStats st = row_stats_strided([&](int c) { return ld_dep(hrow + c); }, nvec, ln_eps, lane);
    for (int c = lane; c < nvec; c += 32) yrow[c] = layer_norm_vec8(ld_dep(hrow + c), st, gamma, beta, c);
}

// ---------------------------------------------------------------------------------------------
// Merge of the per-tile partial states, one warp per row, in vocabulary order; final decision.
// blockIdx.y = head.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) merge_rows_kernel(const State* partials_all, const float* second_all, int n_tiles, int M,
                                                         const __grid_constant__ MergeHeads hs) {
    launch_dependents();
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int head = blockIdx.y;
    if (row >= M) return;
    const State* partials = partials_all + ((size_t)head * M + row) * n_tiles;
    grid_dependency_wait();                              // the partial states come from the GEMM kernel
    merge_row_and_decide(partials, second_all ? second_all + ((size_t)head * M + row) * n_tiles : nullptr, n_tiles, head, row,
                         hs, lane);
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
constexpr int kMinTileN = 64;
constexpr int kFusedMergeMaxRows = 512;    // rows (over all heads of a launch) up to which the GEMM kernel merges itself
// Ring depth for a runtime tile width; b_rows = rows of W one CTA stages per k-block.
int stages_for(int b_rows, int mma_m, int kbs) {
    const size_t stage = (size_t)kbs * ((size_t)mma_m * BK * 2 + (size_t)b_rows * BK * 2);
    const size_t n = (kGemmSmemBudget - kBarBytes - 1024) / stage;
    return (int)(n < (size_t)kMaxGemmStages ? n : (size_t)kMaxGemmStages);
}

template <int BN_T, bool kTop2, bool kPair>
ee_status configure_gemm(int device) {
    static bool configured[kMaxDevices] = {};
    if (!configured[device]) {
        if (cudaFuncSetAttribute(exit_head_gemm_kernel<BN_T, kTop2, kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kGemmSmemBudget) != cudaSuccess)
            return EE_ERR_CUDA;
        configured[device] = true;
    }
    return EE_OK;
}

template <int BN_T, bool kTop2, bool kPair>
ee_status launch_gemm(const GemmMaps& maps, const GemmParams& p, int grid, int device, cudaStream_t stream) {
    if (configure_gemm<BN_T, kTop2, kPair>(device) != EE_OK) return EE_ERR_CUDA;
    const int b_rows = kPair ? p.bn / 2 : p.bn;
    const size_t smem = BN_T ? (size_t)Cfg<BN_T>::kSmemBytes
                             : (size_t)p.n_stages * (p.k2 ? 2 : 1) * ((size_t)p.mma_m * BK * 2 + (size_t)b_rows * BK * 2) + kBarBytes + 1024;
    const cudaError_t err = kPair ? launch_pdl_pairs(exit_head_gemm_kernel<BN_T, kTop2, kPair>, grid, kGemmThreads, smem, stream, maps, p)
                                  : launch_pdl(exit_head_gemm_kernel<BN_T, kTop2, kPair>, grid, kGemmThreads, smem, stream, maps, p);
    return err == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

// How many two-CTA clusters of the GEMM kernel the device runs at once (0: none, or the query failed); asked
// once per device.  All instantiations have the same footprint (one CTA per SM, the whole shared memory).
int resident_pairs(int device) {
    static int pairs[kMaxDevices];
    static bool asked[kMaxDevices] = {};
    if (!asked[device]) {
        pairs[device] = 0;
        if (configure_gemm<0, false, true>(device) == EE_OK) {
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute attr[2];
            pair_launch_config(cfg, attr, dim3(2), kGemmThreads, kGemmSmemBudget, nullptr);
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, exit_head_gemm_kernel<0, false, true>, &cfg) == cudaSuccess && n > 0)
                pairs[device] = n;
            else
                (void)cudaGetLastError();
        }
        asked[device] = true;
    }
    return pairs[device];
}

// Pairs of CTAs work on 256-row tiles when a head has an even number of 128-row tiles; EE_GEMM_PAIRS=0 in the
// environment keeps every CTA on its own 128-row tiles (for comparisons).
// Looks an owner of the in-kernel merge takes at the ticket before it hands its rows to the last arriver: 96
// (some hundred microseconds with the back-off) unless EE_MERGE_LOOKS says otherwise -- 0 makes every owner give
// up at once, which is how the tests drive the hand-over paths that otherwise need contention to occur.
int merge_looks() {
    const char* e = getenv("EE_MERGE_LOOKS");
    if (!e || !*e) return 96;
    const int v = atoi(e);
    return v < 0 ? 0 : (v > 4096 ? 4096 : v);
}

bool k2_enabled() {
    static int enabled = -1;
    if (enabled < 0) {
        const char* e = getenv("EE_GEMM_K2");
        enabled = (e && e[0] == '0') ? 0 : 1;
    }
    return enabled != 0;
}

bool pairs_enabled() {
    static int enabled = -1;
    if (enabled < 0) {
        const char* e = getenv("EE_GEMM_PAIRS");
        enabled = (e && e[0] == '0') ? 0 : 1;
    }
    return enabled != 0;
}

// Upper bound on the partial states of M rows of one head whatever tile width the launch picks.
size_t second_bytes(int M, int V);
size_t partials_bytes(int M, int V) {
    const int bn = M > 1024 ? 256 : kMinTileN;
    return align_up((size_t)M * ((V + bn - 1) / bn) * sizeof(State), 256);
}

// The stacked LayerNorm outputs, every head's rows padded to whole 128-row tiles (padding rows are written as
// zeros): each tile the GEMM loads lies inside the buffer, a plain copy for the TMA unit, which it serves
// faster than a tile it has to fill with zeros itself, and no tile holds another head's rows.
size_t y_rows(int M, int n_heads) { return (size_t)n_heads * (size_t)((M + BM - 1) / BM) * BM; }
size_t y_bytes(int M, int d, int n_heads) { return align_up(y_rows(M, n_heads) * d * sizeof(__nv_bfloat16), 256); }

// One float per partial state (the tile's second-largest logit), used when the top-2 probability gap is asked for.
size_t second_bytes(int M, int V) { return align_up(partials_bytes(M, V) / 4, 256); }

}  // namespace

// Large M: 256, the widest accumulator (two fit in tensor memory), which maximises the reuse of each y tile.
// Up to 1024 rows the weights are read about once and the launch is bound by HBM and by how evenly the
// tiles fill the SMs: the width in 64..256 (multiple of 16) that minimises waves x (width + fixed cost).
static int tile_n_for(long long m_units, int V, int n_heads, int num_sms);
int gemm_tile_n(int M, int V, int n_heads, int num_sms) {
    if (M > 1024) return 256;
    return tile_n_for((M + BM - 1) / BM, V, n_heads, num_sms);
}
// m_units row tiles (or pairs of row tiles) per head, num_sms CTAs (or pairs of CTAs) to spread the tiles over.
static int tile_n_for(long long m_tiles, int V, int n_heads, int num_sms) {
    int best = 128;
    long long best_cost = -1;
    for (int bn = kMinTileN; bn <= 256; bn += 16) {
        const long long tiles = n_heads * m_tiles * ((V + bn - 1) / bn);
        const long long waves = (tiles + num_sms - 1) / num_sms;
        const long long cost = waves * (bn + 16);
        if (best_cost < 0 || cost < best_cost || (cost == best_cost && bn > best)) {
            best = bn;
            best_cost = cost;
        }
    }
    return best;
}

// LayerNorm and GEMM; plus the merge kernel when the rows are too many for the GEMM kernel to merge itself.
int gemm_launches(int M, int n_heads) { return n_heads * M <= kFusedMergeMaxRows ? 2 : 3; }

size_t gemm_workspace_bytes(int M, int d, int V, int n_heads) {
    return (size_t)n_heads * (partials_bytes(M, V) + second_bytes(M, V)) + y_bytes(M, d, n_heads);
}

// Everything one call needs but the launches themselves: kernel arguments (tensor maps included), launch shapes and
// which instantiations to use.  Filled by gemm_plan from the heads' arguments (and, once per process, the
// environment); gemm_run launches from it on any stream.  Plain data: a caller may keep it in memory of its own.
namespace {
struct GemmPlan {
    LnHeads ln;
    const int* row_idx;
    const int* m_dev;
    unsigned char maps[sizeof(GemmMaps)];      // copied to an aligned object for the launch
    GemmParams p;
    __nv_bfloat16* y;
    float ln_eps;
    int device;
    int ln_kind;                               // 2, 4: rows in registers; -2, -3, -4: one CTA per row (-12 .. -14: lean); 0: re-read; 100: gathered rows
    int ln_grid_x, ln_threads;
    int gemm_grid;
    int pair, wide, top2;                      // GEMM instantiation
    int merge_grid_x;                          // 0: the GEMM kernel merges itself
};
static_assert(sizeof(GemmPlan) <= kGemmPlanBytes, "kGemmPlanBytes in kernels.h is too small");
static_assert(alignof(GemmPlan) <= 8, "a plan lives in caller memory aligned to 8 bytes");
}  // namespace

ee_status gemm_plan(const HeadArgs* heads, int n_heads, void* storage) {
    if (n_heads < 1 || n_heads > kGemmMaxHeads) return EE_ERR_SHAPE;
    GemmPlan& g = *static_cast<GemmPlan*>(storage);
    memset(&g, 0, sizeof(g));
    const HeadArgs& a = heads[0];
    unsigned char* ws = static_cast<unsigned char*>(a.workspace);
    State* partials = reinterpret_cast<State*>(ws + kCtrlBytes);
    float* second = reinterpret_cast<float*>(ws + kCtrlBytes + (size_t)n_heads * partials_bytes(a.M, a.V));
    __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(ws + kCtrlBytes +
                                                        (size_t)n_heads * (partials_bytes(a.M, a.V) + second_bytes(a.M, a.V)));
    const int m_tiles = (a.M + BM - 1) / BM;
    const int n_pairs = (m_tiles % 2 == 0 && pairs_enabled()) ? resident_pairs(a.device) : 0;
    const bool pair = n_pairs > 0;
    const int bn = !pair ? gemm_tile_n(a.M, a.V, n_heads, a.num_sms)
                         : (a.M > 1024 ? 256 : tile_n_for(m_tiles / 2, a.V, n_heads, n_pairs));

    MergeHeads mg = {};
    for (int k = 0; k < n_heads; ++k) {
        g.ln.h[k] = static_cast<const __nv_bfloat16*>(heads[k].h);
        g.ln.ld_h[k] = heads[k].ld_h;
        g.ln.gamma[k] = heads[k].gamma;
        g.ln.beta[k] = heads[k].beta;
        mg.tau_per_row[k] = heads[k].tau_per_row;
        mg.tau[k] = heads[k].tau;
        mg.argmax[k] = heads[k].argmax;
        mg.entropy[k] = heads[k].entropy;
        mg.maxprob[k] = heads[k].maxprob;
        mg.exit_mask[k] = heads[k].exit_mask;
        mg.top2gap[k] = heads[k].top2gap;
    }
    g.y = y;
    g.ln_eps = a.ln_eps;
    g.device = a.device;
    g.row_idx = a.row_idx;
    g.m_dev = a.m_dev;
    const int m_pad = m_tiles * BM;
    if (a.row_idx || a.m_dev) {
        if (n_heads != 1) return EE_ERR_SHAPE;
        g.ln_kind = 100; g.ln_threads = 256; g.ln_grid_x = m_pad / 8;
    } else if (a.d <= 1024) {
        g.ln_kind = a.d <= 512 ? 2 : 4; g.ln_threads = ln_threads(g.ln_kind); g.ln_grid_x = m_pad / (g.ln_threads / 32);
    } else if (a.d <= 4096) {
        g.ln_kind = a.d <= 2048 ? -2 : (a.d <= 3072 ? -3 : -4); g.ln_threads = 128; g.ln_grid_x = m_pad;
        if ((long long)m_pad * n_heads >= 2048) g.ln_kind -= 10;      // memory-bound batch: the lean variant
    } else {
        g.ln_kind = 0; g.ln_threads = ln_threads(0); g.ln_grid_x = m_pad / (g.ln_threads / 32);
    }

    // 256-byte L2 promotion for the weights while they are read about once: a tile load touches 128 bytes of
    // each row, and fetching the neighbouring 128 bytes (the next k-block's) with it lets the row-strided
    // pattern stream from HBM at the rate of a contiguous copy (measured: 6.9 against 5.5 TB/s).
    const CUtensorMapL2promotion promo = a.M <= 1024 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B;
    GemmMaps maps;
    const int mma_m = a.M <= 64 ? 64 : BM;
    // A ring slot holds two k-blocks fetched by one request per operand (see the kernel) whenever three such slots
    // fit (with the 256-wide tiles of large batches: pairs); EE_GEMM_K2=0 switches it off for comparisons.
    const int k2 = (a.d % 64 == 0 && k2_enabled() && (a.M > 1024 ? pair : stages_for(pair ? bn / 2 : bn, mma_m, 2) >= 3)) ? 1 : 0;
    if (!(k2 ? make_tile_map_k2(&maps.y, y, (int)y_rows(a.M, n_heads), a.d, mma_m)
             : make_tile_map(&maps.y, y, (int)y_rows(a.M, n_heads), a.d, mma_m)))
        return EE_ERR_CUDA;
    for (int k = 0; k < kGemmMaxHeads; ++k) {
        const void* W = heads[k < n_heads ? k : 0].W;
        if (!(k2 ? make_tile_map_k2(&maps.w[k], W, a.V, a.d, pair ? bn / 2 : bn, promo) : make_tile_map(&maps.w[k], W, a.V, a.d, pair ? bn / 2 : bn, promo)))
            return EE_ERR_CUDA;
    }
    memcpy(g.maps, &maps, sizeof(maps));

    GemmParams& p = g.p;
    p.M = a.M;
    p.V = a.V;
    p.d = a.d;
    p.m_tiles = m_tiles;
    p.n_tiles = (a.V + bn - 1) / bn;
    p.k_blocks = (a.d + BK - 1) / BK;
    p.n_heads = n_heads;
    p.partials = partials;
    p.second = nullptr;
    for (int k = 0; k < n_heads; ++k)
        if (heads[k].top2gap) p.second = second;
    for (int k = 0; k < n_heads; ++k)
        if (p.second && !heads[k].top2gap) return EE_ERR_NULL;        // all heads of a launch or none
    p.ctrl = reinterpret_cast<Control*>(ws);
    p.bn = bn;
    p.mma_m = mma_m;
    p.fused_merge = (n_heads * a.M <= kFusedMergeMaxRows) ? 1 : 0;
    p.merge_looks = merge_looks();
    p.mg = mg;
    p.k2 = k2;
    p.n_stages = stages_for(pair ? bn / 2 : bn, mma_m, k2 ? 2 : 1);
    g.pair = pair ? 1 : 0;
    g.wide = a.M > 1024 ? 1 : 0;
    g.top2 = p.second ? 1 : 0;
    if (pair) {
        const long long total = (long long)n_heads * (p.m_tiles / 2) * p.n_tiles;
        g.gemm_grid = 2 * (int)(total < n_pairs ? total : n_pairs);
    } else {
        const long long total = (long long)n_heads * p.m_tiles * p.n_tiles;
        g.gemm_grid = (int)(total < a.num_sms ? total : a.num_sms);
    }
    g.merge_grid_x = p.fused_merge ? 0 : (a.M + 7) / 8;
    // the kernels' shared-memory attributes are per device and set once: done here, so that gemm_run only launches
    ee_status st = EE_OK;
    if (g.pair) st = g.wide ? (g.top2 ? configure_gemm<256, true, true>(g.device) : configure_gemm<256, false, true>(g.device))
                            : (g.top2 ? configure_gemm<0, true, true>(g.device) : configure_gemm<0, false, true>(g.device));
    else st = g.wide ? (g.top2 ? configure_gemm<256, true, false>(g.device) : configure_gemm<256, false, false>(g.device))
                     : (g.top2 ? configure_gemm<0, true, false>(g.device) : configure_gemm<0, false, false>(g.device));
    return st;
}

ee_status gemm_run(const void* storage, cudaStream_t stream) {
    const GemmPlan& g = *static_cast<const GemmPlan*>(storage);
    const GemmParams& p = g.p;
    const dim3 ln_grid(g.ln_grid_x, p.n_heads);
    cudaError_t err;
    switch (g.ln_kind) {
        case 100: err = launch_pdl(layer_norm_gather_kernel, dim3(g.ln_grid_x), 256, 0, stream, g.ln.h[0], g.ln.ld_h[0], g.ln.gamma[0],
                                   g.ln.beta[0], g.ln_eps, g.row_idx, g.m_dev, g.y, p.M, p.d, p.ctrl); break;
        case 2: err = launch_pdl(layer_norm_rows_kernel<2>, ln_grid, g.ln_threads, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
        case 4: err = launch_pdl(layer_norm_rows_kernel<4>, ln_grid, g.ln_threads, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
        case -2: err = launch_pdl(layer_norm_wide_rows_kernel<2, false>, ln_grid, 128, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
        case -3: err = launch_pdl(layer_norm_wide_rows_kernel<3, false>, ln_grid, 128, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
        case -4: err = launch_pdl(layer_norm_wide_rows_kernel<4, false>, ln_grid, 128, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
        case -12: err = launch_pdl(layer_norm_wide_rows_kernel<2, true>, ln_grid, 128, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
        case -13: err = launch_pdl(layer_norm_wide_rows_kernel<3, true>, ln_grid, 128, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
        case -14: err = launch_pdl(layer_norm_wide_rows_kernel<4, true>, ln_grid, 128, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
        default: err = launch_pdl(layer_norm_rows_kernel<0>, ln_grid, g.ln_threads, 0, stream, g.ln, g.ln_eps, g.y, p.M, p.d, p.ctrl); break;
    }
    if (err != cudaSuccess) return EE_ERR_CUDA;
    GemmMaps maps;
    memcpy(&maps, g.maps, sizeof(maps));
    ee_status st;
    if (g.pair) st = g.wide ? (g.top2 ? launch_gemm<256, true, true>(maps, p, g.gemm_grid, g.device, stream)
                                      : launch_gemm<256, false, true>(maps, p, g.gemm_grid, g.device, stream))
                            : (g.top2 ? launch_gemm<0, true, true>(maps, p, g.gemm_grid, g.device, stream)
                                      : launch_gemm<0, false, true>(maps, p, g.gemm_grid, g.device, stream));
    else st = g.wide ? (g.top2 ? launch_gemm<256, true, false>(maps, p, g.gemm_grid, g.device, stream)
                               : launch_gemm<256, false, false>(maps, p, g.gemm_grid, g.device, stream))
                     : (g.top2 ? launch_gemm<0, true, false>(maps, p, g.gemm_grid, g.device, stream)
                               : launch_gemm<0, false, false>(maps, p, g.gemm_grid, g.device, stream));
    if (st != EE_OK || g.merge_grid_x == 0) return st;
    err = launch_pdl(merge_rows_kernel, dim3(g.merge_grid_x, p.n_heads), 256, 0, stream, (const State*)p.partials,
                     (const float*)p.second, p.n_tiles, p.M, p.mg);
    return err == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

ee_status gemm_launch(const HeadArgs* heads, int n_heads) {
    alignas(8) unsigned char storage[kGemmPlanBytes];
    const ee_status st = gemm_plan(heads, n_heads, storage);
    return st != EE_OK ? st : gemm_run(storage, heads[0].stream);
}

}  // namespace ee
