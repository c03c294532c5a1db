// What the two persistent TMA + tcgen05 kernels -- the exit head's (gemm_kernel.cu) and the KL loss's
// (kl_kernel.cu) -- have in common: the order in which a launch walks its tiles, how a role records a wait that
// gave up, one k-block of MMAs with its barriers, and what the producer and the MMA issuer do before the CTA may
// give its shared and tensor memory back after such a failure.  Each kernel keeps its own tile list, operands and
// epilogue; what is here is written once so that a change to the ring protocol is made once.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace ee {

constexpr int kRoleGroupM = 16;            // m-tiles per super-row of the tile order
constexpr int kRoleBK = 64;                // one k-block: 64 bf16 = one 128-byte swizzled row

// Tile number -> (m_tile, n_tile): super-rows of kRoleGroupM row tiles, inside one the row tile runs fastest, so that
// CTAs working at the same time share a weight tile in L2.
__device__ __forceinline__ void tile_coords(int tile, int m_tiles, int n_tiles, int& m_tile, int& n_tile) {
    const int per_group = kRoleGroupM * n_tiles;
    const int grp = tile / per_group;
    const int within = tile - grp * per_group;
    const int rows_in_group = min(kRoleGroupM, m_tiles - grp * kRoleGroupM);
    n_tile = within / rows_in_group;
    m_tile = grp * kRoleGroupM + (within - n_tile * rows_in_group);
}

// A bounded wait ran out: the first such event of a call is kept in the control block (role, stage or buffer,
// tile), and the CTA's other roles are told to stop.
__device__ __forceinline__ void record_failure(Control* ctrl, volatile int* abort_flag, unsigned role, unsigned stage,
                                               unsigned tile) {
    if (atomicCAS(&ctrl->error, 0u, (unsigned)EE_ERR_TIMEOUT) == 0u)
        ctrl->error_info = (role << 24) | ((stage & 0xffu) << 16) | (tile & 0xffffu);
    *abort_flag = 1;
    __threadfence_block();
}

// One stage by the MMA-issuing thread: wait until the stage's operands have landed, four MMAs of K = 16 on the
// 128-byte-swizzled tiles at a_addr / b_addr into the accumulator at d_tmem (the first MMA of a tile overwrites
// it) -- and, if the stage holds a second k-block (a_second != 0: its tiles lie a_second / b_second bytes further
// on), four more --, then a commit that frees the stage, in both CTAs of a pair, once the tensor core has read it.
// False if the wait gave up.
template <bool kPair>
__device__ __forceinline__ bool mma_k_block(uint32_t full_bar, uint32_t phase, uint32_t empty_bar, uint32_t a_addr, uint32_t b_addr,
                                            uint32_t d_tmem, uint32_t idesc, bool first_of_tile, const volatile int* abort_flag,
                                            uint32_t a_second = 0, uint32_t b_second = 0) {
    if (!ptx::mbar_wait(full_bar, phase, abort_flag)) return false;
    ptx::tc_fence_after_sync();
    const uint64_t adesc = ptx::smem_desc_k128(a_addr);
    const uint64_t bdesc = ptx::smem_desc_k128(b_addr);
#pragma unroll
    for (int k = 0; k < kRoleBK / 16; ++k) {          // 16 bf16 = 32 bytes = 2 descriptor units per step
        const uint32_t accumulate = (first_of_tile && k == 0) ? 0u : 1u;
        if (kPair) ptx::mma_bf16_ss_pair(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, accumulate);
        else ptx::mma_bf16_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, accumulate);
    }
    if (a_second != 0) {
        const uint64_t adesc2 = ptx::smem_desc_k128(a_addr + a_second);
        const uint64_t bdesc2 = ptx::smem_desc_k128(b_addr + b_second);
#pragma unroll
        for (int k = 0; k < kRoleBK / 16; ++k) {
            if (kPair) ptx::mma_bf16_ss_pair(d_tmem, adesc2 + 2u * k, bdesc2 + 2u * k, idesc, 1u);
            else ptx::mma_bf16_ss(d_tmem, adesc2 + 2u * k, bdesc2 + 2u * k, idesc, 1u);
        }
    }
    if (kPair) ptx::mma_commit_pair(empty_bar, 3);
    else ptx::mma_commit(empty_bar);
    return true;
}

// Arrival on `bar` (in both CTAs of a pair) when every MMA issued so far has completed: an accumulator is ready.
template <bool kPair>
__device__ __forceinline__ void mma_commit_all(uint32_t bar) {
    if (kPair) ptx::mma_commit_pair(bar, 3);
    else ptx::mma_commit(bar);
}

// After a failure, the MMA issuer makes sure that no MMA is still writing tensor memory when it is released.
template <bool kPair>
__device__ __forceinline__ void mma_drain(uint32_t drain_bar) {
    if (kPair) ptx::mma_commit_pair(drain_bar, 1);
    else ptx::mma_commit(drain_bar);
    for (uint32_t i = 0; i < (1u << 16) && !ptx::mbar_try_wait(drain_bar, 0); ++i) __nanosleep(100);
}

// After a failure, the producer lets the copies still in flight land before the CTA gives its shared memory back:
// `armed` names the stages with a copy outstanding, `armed_parity` the phase each reports to.  (Rank 1 of a pair
// cannot poll the barrier its copies report to -- it lives in rank 0 -- and waits out a fixed time instead.)
__device__ __forceinline__ void producer_drain(uint32_t rank, int n_stages, uint32_t full_bar0, uint32_t armed, uint32_t armed_parity) {
    if (rank != 0) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        return;
    }
    for (int s = 0; s < n_stages; ++s)
        if (armed & (1u << s)) {
            const uint32_t par = (armed_parity >> s) & 1u;
            for (uint32_t i = 0; i < (1u << 16) && !ptx::mbar_try_wait(full_bar0 + 8u * s, par); ++i) __nanosleep(100);
        }
}

}  // namespace ee
