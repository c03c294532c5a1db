// Forward pass of a head's self-supervised training objective (paper section 3.3, "Losses"):
//     kl_i = sum_v p_head(v) (log p_head(v) - log p_teacher(v))       loss = mean_i kl_i
// for M tokens, from the head's hidden states and weights and the main model's final hidden states and head,
// without ever writing either M x V logit matrix.
//
// With z = head logits, w = teacher logits:  kl = -H(p_head) + logZ(w) - E_{p_head}[w], so next to the head's
// mergeable state (m, s, t, idx) a row carries the teacher's (m_w, s_w) and the cross sum u = sum e^{z - m} w.
// With labels the same pass also gives the supervised objective of that paragraph, ce_i = -log p_head(label_i)
// = logZ(z) - z[label_i]: the epilogue keeps the head's logit at the label's column.
//
// Three kernels chained by programmatic dependent launch:
//   LayerNorm of both inputs (warp per row) into one bf16 buffer, rows padded to whole 128-row tiles with zeros;
//   a persistent TMA + tcgen05 kernel, one CTA per SM: every tile of (128 rows x BN vocabulary rows) is computed
//   twice in a row -- head operands into TMEM buffer 0, teacher operands into buffer 1 -- and the eight
//   epilogue warps fold the head's statistics out of buffer 0 while the teacher's MMAs still run, then read both
//   buffers column chunk by column chunk for the cross sum and the teacher's maximum, give buffer 0 back, and
//   sum the teacher's exponentials out of buffer 1 while the next tile's head MMAs run (only the second pass
//   does not overlap MMAs; the roles and the bounded waits are those of the inference kernel); with an even number of 128-row tiles two CTAs of a cluster share 256-row tiles, each
//   staging half of every W tile (cta_group::2 MMAs), as in the inference kernel;
//   a merge kernel (warp per row) that combines the per-tile states and writes kl; its last CTA to finish adds the
//   means in a fixed order.
#include "common.cuh"
#include "layer_norm.cuh"
#include "kernels.h"
#include "sm100_ptx.cuh"
#include "gemm_roles.cuh"
#include "tensor_map.h"

namespace ee {

namespace {

constexpr int BM = 128;
constexpr int BK = kRoleBK;
constexpr int kThreads = 320;                   // producer warp, MMA warp, eight epilogue warps
constexpr int kATileBytes = BM * BK * 2;
constexpr int kBarBytes = 512 + 2048 + 2048;    // barriers, then 128 head states and 128 teacher/cross states exchanged
constexpr size_t kSmemBudget = 226 * 1024;
constexpr int kMaxStages = 12;
constexpr int kAccStride = 256;
constexpr int kTmemCols = 512;

struct KlMaps {
    CUtensorMap y;         // [2 * m_pad, d]: the head's rows, then the teacher's
    CUtensorMap w[2];      // head weights, teacher weights, each [V, d]
};

// Teacher side and cross term of a row restricted to some vocabulary range.
struct Cross {
    float mw, sw;          // running maximum of the teacher logits and sum of e^{w - mw}
    float u;               // sum of e^{z - m} w, m being the head state's maximum
    float zl;              // the head's logit at the row's label, -inf while the label's column has not been seen
};
static_assert(sizeof(Cross) == 16, "one 16-byte store per (row, tile)");

struct KlParams {
    int M, V, d;
    int m_tiles, n_tiles, k_blocks, m_pad;
    int bn, n_stages;
    int k2;                // a ring slot holds two k-blocks, fetched by one request per operand (d % 64 == 0)
    State* head_part;      // [M][n_tiles]
    Cross* cross_part;     // [M][n_tiles]
    Control* ctrl;
    const int* labels;     // [M] or NULL (no cross-entropy asked for)
};

// Fold 32 consecutive head logits of one row (the first `nvalid` real) into (m, s, t, idx); the logit at the
// row's label is picked up on the way.
template <bool kFull>
__device__ __forceinline__ void fold_head(State& st, float& zl, const float (&z)[32], int col0, int nvalid, int label) {
    float cm = z[0];
#pragma unroll
    for (int j = 1; j < 32; ++j)
        if (kFull || j < nvalid) cm = fmaxf(cm, z[j]);
    if (cm > st.m) {
        int j0 = 0;
#pragma unroll
        for (int j = 31; j >= 0; --j)
            if ((kFull || j < nvalid) && z[j] == cm) j0 = j;
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
            const float a = fmaf(z[j], kLog2e, neg_m2);      // (z - m) * log2(e)
            const float e = ex2(a);
            s += e;
            t2 = fmaf(e, a, t2);
        }
    }
    st.s += s;
    st.t = fmaf(t2, kLn2, st.t);
    if ((unsigned)(label - col0) < (unsigned)nvalid) {       // one chunk of a row at most; columns past nvalid are the next tile's
#pragma unroll
        for (int j = 0; j < 32; ++j) zl = (col0 + j == label) ? z[j] : zl;
    }
}

// Cross sum u over 32 columns once the maximum of the head logits this thread folds is final (neg_m2 =
// -m * log2(e); no rescaling of u is left), and the running maximum of the teacher logits.
template <bool kFull>
__device__ __forceinline__ void fold_cross(float& u_acc, float& mw, float neg_m2, const float (&z)[32], const float (&w)[32],
                                           int nvalid) {
    float u = 0.f, cw = w[0];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (kFull || j < nvalid) {
            u = fmaf(ex2(fmaf(z[j], kLog2e, neg_m2)), w[j], u);
            cw = fmaxf(cw, w[j]);
        }
    }
    u_acc += u;
    mw = fmaxf(mw, cw);
}

// sum of e^{w - mw} over 32 teacher logits, mw being final (neg_w2 = -mw * log2(e)).
template <bool kFull>
__device__ __forceinline__ float fold_teacher(float neg_w2, const float (&w)[32], int nvalid) {
    float sw = 0.f;
#pragma unroll
    for (int j = 0; j < 32; ++j)
        if (kFull || j < nvalid) sw += ex2(fmaf(w[j], kLog2e, neg_w2));
    return sw;
}

// (st, cr) <- merge with (so, co): two vocabulary ranges of the same row.
__device__ __forceinline__ void merge_pair(State& st, Cross& cr, const State& so, const Cross& co) {
    if (so.s != 0.f) {
        if (st.s == 0.f) {
            cr.u = co.u;
        } else {
            const float m = fmaxf(st.m, so.m);
            cr.u = ex2((st.m - m) * kLog2e) * cr.u + ex2((so.m - m) * kLog2e) * co.u;
        }
    }
    state_merge(st, so);
    cr.zl = fmaxf(cr.zl, co.zl);                            // at most one range holds the label's column
    if (co.sw != 0.f) {
        if (cr.sw == 0.f) {
            cr.mw = co.mw;
            cr.sw = co.sw;
        } else {
            const float mw = fmaxf(cr.mw, co.mw);
            cr.sw = ex2((cr.mw - mw) * kLog2e) * cr.sw + ex2((co.mw - mw) * kLog2e) * co.sw;
            cr.mw = mw;
        }
    }
}

// kPair: clusters of two CTAs share 256-row tiles (row tiles 2u and 2u + 1): each CTA stages its own 128 rows
// of y and half of the W tile's rows, rank 0 issues 256 x BN MMAs over both CTAs' shared memory, each CTA folds its
// own rows out of its own tensor memory (the protocol of the inference kernel's pair mode).
template <bool kPair>
__global__ void __launch_bounds__(kThreads, 1)
kl_pair_gemm_kernel(const __grid_constant__ KlMaps maps, const KlParams p) {
    const int BN = p.bn, S = p.n_stages;
    const uint32_t rank = kPair ? ptx::cluster_cta_rank() : 0u;
    const int worker = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int n_workers = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int b_rows = kPair ? BN / 2 : BN;
    const int b_tile_bytes = b_rows * BK * 2;
    // one k-block per ring slot, or two fetched by one request per operand (as in the inference kernel)
    const int kbs = p.k2 ? 2 : 1;
    const int n_steps = (p.k_blocks + kbs - 1) / kbs;
    const int a_stage_bytes = kbs * kATileBytes, b_stage_bytes = kbs * b_tile_bytes;
    const int stage_bytes = a_stage_bytes + b_stage_bytes;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
    const uint32_t a_base = ptx::smem_addr(smem);
    const uint32_t b_base = a_base + S * a_stage_bytes;
    unsigned char* bar_mem = smem + S * stage_bytes;
    const uint32_t bar_base = ptx::smem_addr(bar_mem);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * S + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * S + 2 + b); };
    const uint32_t drain_bar = bar_base + 8u * (2 * S + 4);
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(bar_mem + 8 * (2 * S + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 8 * (2 * S + 5) + 4);
    auto xfull_bar = [&](int q) { return bar_base + 8u * (2 * S + 6 + q); };
    auto xfree_bar = [&](int q) { return bar_base + 8u * (2 * S + 10 + q); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull_bar(b), 1);
            ptx::mbar_init(tempty_bar(b), kPair ? 16 : 8);
        }
        for (int q = 0; q < 4; ++q) {
            ptx::mbar_init(xfull_bar(q), 1);
            ptx::mbar_init(xfree_bar(q), 1);
        }
        ptx::mbar_init(drain_bar, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&maps.y);
        ptx::prefetch_tensormap(&maps.w[0]);
        ptx::prefetch_tensormap(&maps.w[1]);
    }
    if (warp == 1) {
        if (kPair) {
            ptx::tmem_alloc_pair(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), kTmemCols);
            ptx::tmem_relinquish_pair();
        } else {
            ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), kTmemCols);
            ptx::tmem_relinquish();
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (kPair) ptx::cluster_sync_all();                      // the partner's barriers exist before anything signals them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;
    const int m_units = kPair ? p.m_tiles >> 1 : p.m_tiles;
    const int total_tiles = m_units * p.n_tiles;             // each tile is computed for the head and for the teacher
    auto locate = [&](int tile, int& m_tile, int& n_tile) {
        tile_coords(tile, m_units, p.n_tiles, m_tile, n_tile);
        if (kPair) m_tile = 2 * m_tile + (int)rank;
    };
    auto load_full_bar = [&](int s) { return kPair ? ptx::map_to_cta(full_bar(s), 0) : full_bar(s); };
    auto load_tile = [&](uint32_t dst, const CUtensorMap* m, int step, int row, uint32_t bar) {   // the k-block(s) of stage `step`
        if (kbs == 2) {
            if (kPair) ptx::tma_load_3d_pair(dst, m, 0, row, 2 * step, bar);
            else ptx::tma_load_3d(dst, m, 0, row, 2 * step, bar);
        } else if (kPair) ptx::tma_load_2d_pair(dst, m, step * BK, row, bar);
        else ptx::tma_load_2d(dst, m, step * BK, row, bar);
    };
    const uint32_t arm_bytes = (uint32_t)stage_bytes * (kPair ? 2u : 1u);

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0, armed = 0, armed_parity = 0;
            bool ok = true;
            int n_pre = 0;
            if (worker < total_tiles) {                       // head weights of the first stages before the wait
                int m_tile, n_tile;
                locate(worker, m_tile, n_tile);
                n_pre = min(S, n_steps);
                for (int kb = 0; kb < n_pre; ++kb) {
                    if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(kb), arm_bytes);
                    load_tile(b_base + kb * b_stage_bytes, &maps.w[0], kb, n_tile * BN + (int)rank * b_rows, load_full_bar(kb));
                    armed |= 1u << kb;
                }
            }
            grid_dependency_wait();
            int issued = 0;
            for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
                int m_tile, n_tile;
                locate(tile, m_tile, n_tile);
                for (int which = 0; ok && which < 2; ++which) {
                    const int y_row = which * p.m_pad + m_tile * BM;
                    for (int kb = 0; kb < n_steps; ++kb, ++issued) {
                        if (issued < n_pre) {
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
                        load_tile(b_base + stage * b_stage_bytes, &maps.w[which], kb, n_tile * BN + (int)rank * b_rows,
                                  load_full_bar(stage));
                        armed |= 1u << stage;
                        armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
                        if (++stage == S) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (*abort_flag) producer_drain(rank, S, full_bar(0), armed, armed_parity);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer: buffer 0 = head, 1 = teacher
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = ptx::idesc_bf16_f32(kPair ? 2 * BM : BM, BN);
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            bool ok = true;
            for (int tile = worker; ok && tile < total_tiles; tile += n_workers, ++local) {
                const uint32_t acc_phase = (uint32_t)local & 1u;
                for (int which = 0; ok && which < 2; ++which) {
                    if (!ptx::mbar_wait(tempty_bar(which), acc_phase ^ 1u, abort_flag)) {
                        record_failure(p.ctrl, abort_flag, 2, 0x80 | which, tile);
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(which * kAccStride);
                    for (int kb = 0; kb < n_steps; ++kb) {
                        const bool two = kbs == 2 && 2 * kb + 1 < p.k_blocks;        // the second k-block of the slot exists
                        if (!mma_k_block<kPair>(full_bar(stage), phase, empty_bar(stage), a_base + stage * a_stage_bytes,
                                                b_base + stage * b_stage_bytes, d_tmem, idesc, kb == 0, abort_flag,
                                                two ? (uint32_t)kATileBytes : 0u, (uint32_t)b_tile_bytes)) {
                            record_failure(p.ctrl, abort_flag, 2, stage, tile);
                            ok = false;
                            break;
                        }
                        if (++stage == S) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) mma_commit_all<kPair>(tfull_bar(which));
                }
            }
            if (*abort_flag) mma_drain<kPair>(drain_bar);
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9)
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;                   // even / odd 32-column chunks
        State* xchg = reinterpret_cast<State*>(bar_mem + 512) + quarter * 32 + lane;
        Cross* xchg_c = reinterpret_cast<Cross*>(bar_mem + 512 + 2048) + quarter * 32 + lane;
        const int row_in_tile = quarter * 32 + lane;
        int local = 0;
        grid_dependency_wait();
        for (int tile = worker; tile < total_tiles; tile += n_workers, ++local) {
            int m_tile, n_tile;
            locate(tile, m_tile, n_tile);
            const uint32_t acc_phase = (uint32_t)local & 1u;
            // the head's statistics are folded while the teacher's MMAs of the same tile still run
            if (!__all_sync(0xffffffffu, ptx::mbar_wait(tfull_bar(0), acc_phase, abort_flag))) {
                if (lane == 0) record_failure(p.ctrl, abort_flag, 3, 0, tile);
                break;
            }
            ptx::tc_fence_after_sync();
            const int n0 = n_tile * BN;
            const int ncols = min(BN, p.V - n0);
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
            State st = state_empty();
            Cross cr = {-CUDART_INF_F, 0.f, 0.f, -CUDART_INF_F};
            const int row = m_tile * BM + row_in_tile;
            const bool live = row < p.M;
            const bool any_live = __any_sync(0xffffffffu, live);
            const int label = (live && p.labels) ? ld_dep(p.labels + row) : -1;
            if (any_live) {
                for (int c = half; c * 32 < ncols; c += 2) {
                    float z[32];
                    ptx::tmem_ld_32x32(taddr + c * 32, z);
                    ptx::tmem_ld_wait();
                    const int nvalid = ncols - c * 32;
                    if (live) {
                        if (nvalid >= 32) fold_head<true>(st, cr.zl, z, n0 + c * 32, 32, label);
                        else fold_head<false>(st, cr.zl, z, n0 + c * 32, nvalid, label);
                    }
                }
            }
            // second pass over both accumulators: the cross sum against the now final maximum and the teacher's
            // maximum; the head's accumulator is then free for the next tile's MMAs
            if (!__all_sync(0xffffffffu, ptx::mbar_wait(tfull_bar(1), acc_phase, abort_flag))) {
                if (lane == 0) record_failure(p.ctrl, abort_flag, 3, 1, tile);
                break;
            }
            ptx::tc_fence_after_sync();
            if (any_live) {
                const float neg_m2 = -st.m * kLog2e;
                for (int c = half; c * 32 < ncols; c += 2) {
                    float z[32], w[32];
                    ptx::tmem_ld_32x32(taddr + c * 32, z);
                    ptx::tmem_ld_32x32(taddr + kAccStride + c * 32, w);
                    ptx::tmem_ld_wait();
                    const int nvalid = ncols - c * 32;
                    if (live) {
                        if (nvalid >= 32) fold_cross<true>(cr.u, cr.mw, neg_m2, z, w, 32);
                        else fold_cross<false>(cr.u, cr.mw, neg_m2, z, w, nvalid);
                    }
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (kPair) ptx::mbar_arrive_remote(ptx::map_to_cta(tempty_bar(0), 0));
                else ptx::mbar_arrive(tempty_bar(0));
            }
            // third pass, over the teacher's accumulator alone (the next tile's head MMAs may run meanwhile)
            if (any_live) {
                const float neg_w2 = -cr.mw * kLog2e;
                for (int c = half; c * 32 < ncols; c += 2) {
                    float w[32];
                    ptx::tmem_ld_32x32(taddr + kAccStride + c * 32, w);
                    ptx::tmem_ld_wait();
                    const int nvalid = ncols - c * 32;
                    if (live) cr.sw += nvalid >= 32 ? fold_teacher<true>(neg_w2, w, 32) : fold_teacher<false>(neg_w2, w, nvalid);
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (kPair) ptx::mbar_arrive_remote(ptx::map_to_cta(tempty_bar(1), 0));
                else ptx::mbar_arrive(tempty_bar(1));
            }
            const uint32_t x_phase = (uint32_t)local & 1u;
            if (half == 1) {
                const bool free_ = local == 0 || ptx::mbar_wait(xfree_bar(quarter), x_phase ^ 1u, abort_flag);
                if (!__all_sync(0xffffffffu, free_)) {
                    if (lane == 0) record_failure(p.ctrl, abort_flag, 5, quarter, tile);
                    break;
                }
                *xchg = st;
                *xchg_c = cr;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(xfull_bar(quarter));
            } else {
                const bool there = ptx::mbar_wait(xfull_bar(quarter), x_phase, abort_flag);
                if (!__all_sync(0xffffffffu, there)) {
                    if (lane == 0) record_failure(p.ctrl, abort_flag, 6, quarter, tile);
                    break;
                }
                const State so = *xchg;
                const Cross co = *xchg_c;
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(xfree_bar(quarter));
                if (live) {
                    merge_pair(st, cr, so, co);
                    p.head_part[(size_t)row * p.n_tiles + n_tile] = st;
                    p.cross_part[(size_t)row * p.n_tiles + n_tile] = cr;
                }
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (kPair) ptx::cluster_sync_all();       // neither CTA leaves while the other may still signal it or write its accumulators
    if (warp == 1) {
        __syncwarp();
        ptx::tc_fence_after_sync();
        if (kPair) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
        else ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// LayerNorm of the head's rows (blockIdx.y = 0) and the teacher's (1) into y [2][m_pad][d]; zero rows above M.
struct KlLnArgs {
    const __nv_bfloat16* h[2];
    long long ld_h[2];
    const float* gamma[2];
    const float* beta[2];
    float ln_eps[2];
};

__global__ void __launch_bounds__(256) kl_layer_norm_kernel(const __grid_constant__ KlLnArgs a, __nv_bfloat16* y,
                                                            int M, int m_pad, int d) {
    launch_dependents();
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int which = blockIdx.y;
    if (row >= m_pad) return;
    const int nvec = d >> 3;
    uint4* yrow = reinterpret_cast<uint4*>(y + ((size_t)which * m_pad + row) * d);
    grid_dependency_wait();
    if (row >= M) {
        for (int c = lane; c < nvec; c += 32) yrow[c] = make_uint4(0, 0, 0, 0);
        return;
    }
    const uint4* hrow = reinterpret_cast<const uint4*>(a.h[which] + (size_t)row * a.ld_h[which]);
    const RowStats st = row_stats_strided([&](int c) { return ld_dep(hrow + c); }, nvec, a.ln_eps[which], lane);
    for (int c = lane; c < nvec; c += 32) yrow[c] = layer_norm_vec8(ld_dep(hrow + c), st, a.gamma[which], a.beta[which], c);
}

// Sum of src[0 .. M) by the 256 threads of a CTA in a fixed order (bit-identical from run to run), divided by M.
__device__ __forceinline__ float cta_mean_fixed_order(const float* src, int M, float* part) {
    float s = 0.f;
    for (int i = threadIdx.x; i < M; i += 256) s += ld_dep(src + i);
    part[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    const float mean = part[0] / (float)M;
    __syncthreads();
    return mean;
}

// One warp per row: the tiles' states in vocabulary order -> kl (and ce).  With `loss`, the CTA that finishes last
// (a ticket in the control block, taken after the CTA's rows are stored) also writes the means: loss[0] = mean of kl,
// loss[1] = mean of ce if there is one -- summed in a fixed order whichever CTA that is.
__global__ void __launch_bounds__(256) kl_merge_kernel(const State* head_part, const Cross* cross_part,
                                                       int n_tiles, int M, float* kl, float* ce, float* loss, Control* ctrl) {
    __shared__ float part[256];
    __shared__ int is_last;
    launch_dependents();
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    grid_dependency_wait();
    if (row < M) {
    State st = state_empty();
    Cross cr = {-CUDART_INF_F, 0.f, 0.f, -CUDART_INF_F};
    for (int n = lane; n < n_tiles; n += 32) {
        const State so = state_load_cg(head_part + (size_t)row * n_tiles + n);
        const float4 c4 = __ldcg(reinterpret_cast<const float4*>(cross_part + (size_t)row * n_tiles + n));
        merge_pair(st, cr, so, Cross{c4.x, c4.y, c4.z, c4.w});
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const State so = state_shfl_xor(st, o);
        Cross co;
        co.mw = __shfl_xor_sync(0xffffffffu, cr.mw, o);
        co.sw = __shfl_xor_sync(0xffffffffu, cr.sw, o);
        co.u = __shfl_xor_sync(0xffffffffu, cr.u, o);
        co.zl = __shfl_xor_sync(0xffffffffu, cr.zl, o);
        // both lanes of a pair must end with the same bits: merge in a fixed (lower lane first) order
        State a = (lane & o) ? so : st, b = (lane & o) ? st : so;
        Cross ca = (lane & o) ? co : cr, cb = (lane & o) ? cr : co;
        merge_pair(a, ca, b, cb);
        st = a;
        cr = ca;
    }
    if (lane == 0) {
        const float entropy = logf(st.s) - st.t / st.s;                 // H(p_head)
        const float log_z_teacher = cr.mw + logf(cr.sw);
        kl[row] = -entropy + log_z_teacher - cr.u / st.s;
        if (ce) ce[row] = st.m + logf(st.s) - cr.zl;                    // -log p_head(label)
    }
    }
    if (!loss) return;
    __syncthreads();                                                    // the CTA's rows are stored
    if (threadIdx.x == 0) is_last = ticket_arrive_is_last(&ctrl->head_ticket[0], gridDim.x) ? 1 : 0;
    __syncthreads();
    if (!is_last) return;
    const float mean_kl = cta_mean_fixed_order(kl, M, part);
    const float mean_ce = ce ? cta_mean_fixed_order(ce, M, part) : 0.f;
    if (threadIdx.x == 0) {
        loss[0] = mean_kl;
        if (ce) loss[1] = mean_ce;
        ctrl->head_ticket[0] = 0;                                       // ready for the next call
    }
}

int stages_for(int b_rows, int kbs) {
    const size_t stage = (size_t)kbs * (kATileBytes + (size_t)b_rows * BK * 2);
    const size_t n = (kSmemBudget - kBarBytes - 1024) / stage;
    return (int)(n < (size_t)kMaxStages ? n : (size_t)kMaxStages);
}

// How many two-CTA clusters of the pair kernel the device runs at once; 0 if the query fails or EE_GEMM_PAIRS=0
// in the environment switches pairs off.  Asked once per device.
int resident_pairs(int device) {
    static int pairs[kMaxDevices];
    static bool asked[kMaxDevices] = {};
    if (!asked[device]) {
        pairs[device] = 0;
        const char* e = getenv("EE_GEMM_PAIRS");
        if (!(e && e[0] == '0') &&
            cudaFuncSetAttribute(kl_pair_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) == cudaSuccess) {
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute attr[2];
            pair_launch_config(cfg, attr, dim3(2), kThreads, kSmemBudget, nullptr);
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kl_pair_gemm_kernel<true>, &cfg) == cudaSuccess && n > 0) pairs[device] = n;
            else (void)cudaGetLastError();
        }
        asked[device] = true;
    }
    return pairs[device];
}

// Tile width for m_units pairs of row tiles spread over n_pairs pairs of CTAs: 256 for many rows, else the multiple
// of 16 in 64..256 that minimises waves x (width + 16).
int pair_tile_n(int m_units, int V, int n_pairs) {
    if (m_units > 4) return 256;
    int best = 128;
    long long best_cost = -1;
    for (int bn = 64; bn <= 256; bn += 16) {
        const long long tiles = (long long)m_units * ((V + bn - 1) / bn);
        const long long waves = (tiles + n_pairs - 1) / n_pairs;
        const long long cost = waves * (bn + 16);
        if (best_cost < 0 || cost < best_cost || (cost == best_cost && bn > best)) {
            best = bn;
            best_cost = cost;
        }
    }
    return best;
}

int m_pad_of(int M) { return (M + BM - 1) / BM * BM; }
size_t part_bytes(int M, int V) { return align_up((size_t)M * ((V + 63) / 64) * sizeof(State), 256); }

}  // namespace

size_t kl_workspace_bytes(int M, int d, int V) {
    return kCtrlBytes + 2 * part_bytes(M, V) + align_up((size_t)2 * m_pad_of(M) * d * sizeof(__nv_bfloat16), 256);
}

ee_status kl_launch(const HeadArgs& head, const HeadArgs& teacher, const int* labels, float* kl, float* ce, float* loss) {
    const int M = head.M, d = head.d, V = head.V;
    unsigned char* ws = static_cast<unsigned char*>(head.workspace);
    State* head_part = reinterpret_cast<State*>(ws + kCtrlBytes);
    Cross* cross_part = reinterpret_cast<Cross*>(ws + kCtrlBytes + part_bytes(M, V));
    __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(ws + kCtrlBytes + 2 * part_bytes(M, V));
    const int m_pad = m_pad_of(M);
    const int n_pairs = ((m_pad / BM) % 2 == 0) ? resident_pairs(head.device) : 0;     // 0: pairs switched off or unavailable
    const bool pair = n_pairs > 0;
    const int bn = pair ? pair_tile_n(m_pad / BM / 2, V, n_pairs) : gemm_tile_n(M, V, 1, head.num_sms);
    const int b_rows = pair ? bn / 2 : bn;

    KlLnArgs ln;
    const HeadArgs* both[2] = {&head, &teacher};
    for (int k = 0; k < 2; ++k) {
        ln.h[k] = static_cast<const __nv_bfloat16*>(both[k]->h);
        ln.ld_h[k] = both[k]->ld_h;
        ln.gamma[k] = both[k]->gamma;
        ln.beta[k] = both[k]->beta;
        ln.ln_eps[k] = both[k]->ln_eps;
    }
    if (launch_pdl(kl_layer_norm_kernel, dim3(m_pad / 8, 2), 256, 0, head.stream, ln, y, M, m_pad, d) != cudaSuccess)
        return EE_ERR_CUDA;

    KlMaps maps;
    const CUtensorMapL2promotion promo = M <= 1024 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B;
    // two k-blocks per request whenever three such ring slots fit (M = 4096: 686 -> 618 us, M = 1024: 194 -> 174)
    static const bool k2_on = !(getenv("EE_GEMM_K2") && getenv("EE_GEMM_K2")[0] == '0');
    const int k2 = (d % 64 == 0 && k2_on && stages_for(b_rows, 2) >= 3) ? 1 : 0;
    if (k2 ? (!make_tile_map_k2(&maps.y, y, 2 * m_pad, d, BM) || !make_tile_map_k2(&maps.w[0], head.W, V, d, b_rows, promo) ||
              !make_tile_map_k2(&maps.w[1], teacher.W, V, d, b_rows, promo))
           : (!make_tile_map(&maps.y, y, 2 * m_pad, d, BM) || !make_tile_map(&maps.w[0], head.W, V, d, b_rows, promo) ||
              !make_tile_map(&maps.w[1], teacher.W, V, d, b_rows, promo)))
        return EE_ERR_CUDA;
    KlParams p;
    p.M = M; p.V = V; p.d = d;
    p.m_tiles = m_pad / BM;
    p.n_tiles = (V + bn - 1) / bn;
    p.k_blocks = (d + BK - 1) / BK;
    p.m_pad = m_pad;
    p.bn = bn;
    p.k2 = k2;
    p.n_stages = stages_for(b_rows, k2 ? 2 : 1);
    p.head_part = head_part;
    p.cross_part = cross_part;
    p.ctrl = reinterpret_cast<Control*>(ws);
    p.labels = ce ? labels : nullptr;
    static bool configured[kMaxDevices] = {};
    if (!configured[head.device]) {
        if (cudaFuncSetAttribute(kl_pair_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess ||
            cudaFuncSetAttribute(kl_pair_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget) != cudaSuccess)
            return EE_ERR_CUDA;
        configured[head.device] = true;
    }
    const size_t smem = (size_t)p.n_stages * (k2 ? 2 : 1) * (kATileBytes + (size_t)b_rows * BK * 2) + kBarBytes + 1024;
    if (pair) {
        const long long total = (long long)(p.m_tiles / 2) * p.n_tiles;
        const int grid = 2 * (int)(total < n_pairs ? total : n_pairs);
        if (launch_pdl_pairs(kl_pair_gemm_kernel<true>, grid, kThreads, smem, head.stream, maps, p) != cudaSuccess) return EE_ERR_CUDA;
    } else {
        const long long total = (long long)p.m_tiles * p.n_tiles;
        const int grid = (int)(total < head.num_sms ? total : head.num_sms);
        if (launch_pdl(kl_pair_gemm_kernel<false>, grid, kThreads, smem, head.stream, maps, p) != cudaSuccess) return EE_ERR_CUDA;
    }
    if (launch_pdl(kl_merge_kernel, (M + 7) / 8, 256, 0, head.stream, (const State*)head_part, (const Cross*)cross_part, p.n_tiles,
                   M, kl, ce, loss, p.ctrl) != cudaSuccess)
        return EE_ERR_CUDA;
    return EE_OK;
}

}  // namespace ee
