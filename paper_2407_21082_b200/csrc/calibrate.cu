// Calibration of a head's threshold (paper section 3.4.1): joint sort of (confidence, correctness) over the
// calibration tokens, running count of correct predictions, and the most permissive threshold whose set of
// tokens is correct with proportion >= epsilon.
//
// The metric is the entropy H (smaller = surer).  Each token becomes one 64-bit word
//     word = (monotone 32-bit key of H) << 1 | t        t = [argmax_head == argmax_final]   (Eq. 3)
// and the words are sorted ascending by key with a least-significant-digit radix sort: four stable passes of
// 8 bits over the key's 32 bits (per-tile digit histogram -> per-digit exclusive scan over the tiles -> stable
// scatter); t rides along in bit 0 and is not sorted on, because tokens of equal entropy are judged as one group.  A last pass over the sorted words counts the correct predictions before each position and
// tests  correct >= epsilon * count  (fp64) at every position that closes a group of equal entropies; the
// largest such position wins (64-bit atomic max of (count << 32 | correct)).
// Integer work throughout, except that one comparison.
#include "common.cuh"
#include "kernels.h"

namespace ee {

namespace {

constexpr int kSortThreads = 256;
constexpr int kItems = 8;                               // words per thread
constexpr int kTile = kSortThreads * kItems;            // 2048 words per CTA
constexpr int kWarpChunk = 32 * kItems;                 // 256 consecutive words per warp
constexpr int kDigits = 256;
constexpr int kPasses = 4;                              // the 32 key bits; bit 0 (t) is carried, not sorted on

typedef unsigned long long u64;

// Order-preserving map of a float onto unsigned integers (negative floats reversed below the positive ones;
// the two zeros compare equal, so both take the key of +0).
__device__ __forceinline__ unsigned int float_key(float f) {
    const unsigned int b = f == 0.f ? 0u : __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(unsigned int k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__global__ void __launch_bounds__(kSortThreads) calib_pack_kernel(const float* __restrict__ entropy,
                                                                  const int* __restrict__ argmax_head,
                                                                  const int* __restrict__ argmax_final, int n,
                                                                  u64* __restrict__ words, u64* __restrict__ best) {
    const int i = blockIdx.x * kSortThreads + threadIdx.x;
    if (i == 0) *best = 0ull;
    if (i >= n) return;
    const unsigned int t = argmax_head[i] == argmax_final[i] ? 1u : 0u;
    words[i] = ((u64)float_key(entropy[i]) << 1) | t;
}

// hist[digit * n_tiles + tile] = number of words of the tile whose digit of this pass is `digit`.
__global__ void __launch_bounds__(kSortThreads) calib_hist_kernel(const u64* __restrict__ words, int n, int shift,
                                                                  unsigned int* __restrict__ hist, int n_tiles) {
    __shared__ unsigned int cnt[kDigits];
    cnt[threadIdx.x] = 0;
    __syncthreads();
    const int base = blockIdx.x * kTile;
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int i = base + r * kSortThreads + threadIdx.x;
        if (i < n) atomicAdd(&cnt[(unsigned int)(words[i] >> shift) & 255u], 1u);
    }
    __syncthreads();
    hist[(size_t)threadIdx.x * n_tiles + blockIdx.x] = cnt[threadIdx.x];
}

// One CTA per digit: in-place exclusive scan of the digit's row hist[digit][0 .. n_tiles) (where each tile's
// words of that digit start among all words of that digit) and the row total.
__global__ void __launch_bounds__(1024) calib_scan_kernel(unsigned int* __restrict__ hist, int n_tiles,
                                                          unsigned int* __restrict__ digit_total) {
    __shared__ unsigned int warp_sum[32];
    __shared__ unsigned int s_carry;
    unsigned int* row = hist + (size_t)blockIdx.x * n_tiles;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int t0 = 0; t0 < n_tiles; t0 += 1024) {
        const int t = t0 + threadIdx.x;
        const unsigned int v = t < n_tiles ? row[t] : 0u;
        unsigned int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int x = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += x;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const unsigned int w = warp_sum[lane];
            unsigned int wi = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int x = __shfl_up_sync(0xffffffffu, wi, o);
                if (lane >= o) wi += x;
            }
            warp_sum[lane] = wi - w;                     // exclusive over warps
        }
        __syncthreads();
        const unsigned int carry = s_carry;
        if (t < n_tiles) row[t] = carry + warp_sum[warp] + incl - v;
        __syncthreads();
        if (threadIdx.x == 1023) s_carry = carry + warp_sum[31] + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) digit_total[blockIdx.x] = s_carry;
}

// Stable scatter of one tile.  Warp w owns a run of 32 * kItems consecutive words of the tile and walks them 32 at a time,
// so the order of equal digits inside the tile is (warp, round, lane) = their order in memory.  The tile is
// first put in output order in shared memory, so that consecutive threads then write consecutive words of a
// digit's run to global memory.
__global__ void __launch_bounds__(kSortThreads, 4) calib_scatter_kernel(const u64* __restrict__ src, u64* __restrict__ dst,
                                                                     int n, int shift,
                                                                     const unsigned int* __restrict__ tile_start,
                                                                     const unsigned int* __restrict__ digit_total,
                                                                     int n_tiles) {
    __shared__ unsigned int cnt[kSortThreads / 32][kDigits];
    __shared__ unsigned int out_shift[kDigits];        // output position minus position inside the sorted tile, per digit
    __shared__ unsigned int warp_part[kSortThreads / 32];
    __shared__ u64 staged[kTile];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < (kSortThreads / 32) * kDigits; i += kSortThreads) (&cnt[0][0])[i] = 0;
    __syncthreads();
    const int tile_base = blockIdx.x * kTile;
    const int base = tile_base + warp * kWarpChunk;
    u64 v[kItems];
    unsigned int rank[kItems];
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int i = base + r * 32 + lane;
        const bool valid = i < n;
        v[r] = valid ? src[i] : 0ull;
        const unsigned int d = valid ? ((unsigned int)(v[r] >> shift) & 255u) : 0xffffffffu;
        const unsigned int peers = __match_any_sync(0xffffffffu, d);
        const int leader = __ffs(peers) - 1;
        unsigned int before = 0;                                             // the leader reserves the group's ranks
        if (valid && lane == leader) before = atomicAdd(&cnt[warp][d], (unsigned int)__popc(peers));
        before = __shfl_sync(0xffffffffu, before, leader);
        rank[r] = before + __popc(peers & ((1u << lane) - 1u));
    }
    __syncthreads();
    {   // thread = digit d: the tile's count of d, the exclusive scan of the counts over the digits (inside the
        // tile) and of the digit totals (over all words), and each warp's start inside the digit's run
        const unsigned int d = threadIdx.x;
        unsigned int mine = 0;
#pragma unroll
        for (int w = 0; w < kSortThreads / 32; ++w) mine += cnt[w][d];
        const unsigned int total = digit_total[d];
        unsigned int incl = mine, gincl = total;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int x = __shfl_up_sync(0xffffffffu, incl, o);
            const unsigned int g = __shfl_up_sync(0xffffffffu, gincl, o);
            if (lane >= o) { incl += x; gincl += g; }
        }
        if (lane == 31) warp_part[warp] = incl;
        __syncthreads();
        unsigned int lbase = 0;
        for (int w = 0; w < warp; ++w) lbase += warp_part[w];
        __syncthreads();
        if (lane == 31) warp_part[warp] = gincl;
        __syncthreads();
        unsigned int gbase = 0;
        for (int w = 0; w < warp; ++w) gbase += warp_part[w];
        const unsigned int lstart = lbase + incl - mine;
        out_shift[d] = gbase + gincl - total + tile_start[(size_t)d * n_tiles + blockIdx.x] - lstart;
        unsigned int run = lstart;
#pragma unroll
        for (int w = 0; w < kSortThreads / 32; ++w) {
            const unsigned int c = cnt[w][d];
            cnt[w][d] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int i = base + r * 32 + lane;
        if (i < n) staged[cnt[warp][(unsigned int)(v[r] >> shift) & 255u] + rank[r]] = v[r];
    }
    __syncthreads();
    const int in_tile = min(kTile, n - tile_base);
    for (int k = threadIdx.x; k < in_tile; k += kSortThreads) {
        const u64 w = staged[k];
        const unsigned int d = (unsigned int)(w >> shift) & 255u;
        dst[out_shift[d] + (unsigned int)k] = w;
    }
}

// Correct predictions per tile of the sorted words.
__global__ void __launch_bounds__(kSortThreads) calib_tile_sum_kernel(const u64* __restrict__ sorted, int n,
                                                                      unsigned int* __restrict__ tile_sum) {
    __shared__ unsigned int warp_part[kSortThreads / 32];
    const int base = blockIdx.x * kTile;
    unsigned int s = 0;
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int i = base + r * kSortThreads + threadIdx.x;
        if (i < n) s += (unsigned int)sorted[i] & 1u;
    }
    s = __reduce_add_sync(0xffffffffu, s);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int t = 0;
        for (int w = 0; w < kSortThreads / 32; ++w) t += warp_part[w];
        tile_sum[blockIdx.x] = t;
    }
}

// Position i (0-based, surest first) closes a group when the next word has another key.  There the set of the
// i + 1 surest tokens is tested; the largest qualifying set wins.  Warp w walks its run of 32 * kItems positions
// of the tile 32 at a time (held in registers), after the warps have exchanged their counts.
__global__ void __launch_bounds__(kSortThreads) calib_select_kernel(const u64* __restrict__ sorted, int n,
                                                                    const unsigned int* __restrict__ tile_sum,
                                                                    double epsilon, u64* __restrict__ best) {
    __shared__ unsigned int part[kSortThreads / 32];
    __shared__ unsigned int warp_total[kSortThreads / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned int before = 0;                                   // correct predictions in the tiles before this one
    for (int b = threadIdx.x; b < (int)blockIdx.x; b += kSortThreads) before += tile_sum[b];
    before = __reduce_add_sync(0xffffffffu, before);
    const int base = blockIdx.x * kTile + warp * kWarpChunk;
    u64 w[kItems];
    unsigned int mine = 0;
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int i = base + r * 32 + lane;
        w[r] = i < n ? sorted[i] : ~0ull;
        mine += i < n ? ((unsigned int)w[r] & 1u) : 0u;
    }
    mine = __reduce_add_sync(0xffffffffu, mine);
    if (lane == 0) { part[warp] = before; warp_total[warp] = mine; }
    __syncthreads();
    unsigned int run = 0;
    for (int k = 0; k < kSortThreads / 32; ++k) run += part[k] + (k < warp ? warp_total[k] : 0u);
    // the word after this warp's chunk (the first of the next warp's, or of the next tile)
    const int after = base + kWarpChunk;
    const u64 chunk_next = after < n ? sorted[after] : ~0ull;
    u64 local_best = 0;
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int i = base + r * 32 + lane;
        const unsigned int t = i < n ? ((unsigned int)w[r] & 1u) : 0u;
        unsigned int incl = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int x = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += x;
        }
        u64 next = __shfl_down_sync(0xffffffffu, w[r], 1);
        const u64 first_of_next = (r + 1 < kItems) ? w[(r + 1) % kItems] : chunk_next;   // lane 0's follows lane 31's word
        const u64 next_round = __shfl_sync(0xffffffffu, first_of_next, 0);
        if (lane == 31) next = next_round;
        if (i < n) {
            const unsigned int correct = run + incl;               // correct among the i + 1 surest
            const bool closes = (i + 1 == n) || ((next >> 1) != (w[r] >> 1));
            if (closes && (double)correct >= epsilon * (double)(i + 1)) local_best = ((u64)(i + 1) << 32) | correct;
        }
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    // one atomic per CTA: the candidates of a CTA are reduced first (positions grow with lane, round and warp)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const u64 x = __shfl_xor_sync(0xffffffffu, local_best, o);
        local_best = x > local_best ? x : local_best;
    }
    __shared__ u64 warp_best[kSortThreads / 32];
    if (lane == 0) warp_best[warp] = local_best;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 m = 0;
        for (int k = 0; k < kSortThreads / 32; ++k) m = warp_best[k] > m ? warp_best[k] : m;
        if (m) atomicMax(best, m);
    }
}

__global__ void calib_output_kernel(const u64* __restrict__ sorted, int n, const u64* __restrict__ best,
                                    float* __restrict__ tau, int* __restrict__ counts) {
    const u64 b = *best;
    const int n_exit = (int)(b >> 32);
    counts[0] = n_exit;
    counts[1] = (int)(b & 0xffffffffull);
    counts[2] = n_exit ? n - n_exit + 1 : 0;
    *tau = n_exit ? key_float((unsigned int)(sorted[n_exit - 1] >> 1)) : -CUDART_INF_F;
}

__global__ void calib_empty_kernel(float* __restrict__ tau, int* __restrict__ counts) {
    counts[0] = counts[1] = counts[2] = 0;
    *tau = -CUDART_INF_F;
}

constexpr size_t kCalibHeader = 2048;      // the result word and the 256 digit totals

size_t words_bytes(int n) { return align_up((size_t)n * sizeof(u64), 256); }
int tiles_of(int n) { return (n + kTile - 1) / kTile; }

}  // namespace

size_t calibrate_workspace_bytes(int n) {
    const int n_tiles = tiles_of(n);
    return kCalibHeader + 2 * words_bytes(n) + align_up((size_t)kDigits * n_tiles * sizeof(unsigned int), 256) +
           align_up((size_t)n_tiles * sizeof(unsigned int), 256);
}

int calibrate_launches(int n) { return n > 0 ? 1 + 3 * kPasses + 3 : 1; }

ee_status calibrate_launch(const float* entropy, const int* argmax_head, const int* argmax_final, int n, double epsilon,
                           float* tau, int* counts, void* workspace, cudaStream_t stream) {
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    u64* best = reinterpret_cast<u64*>(ws);
    u64* a = reinterpret_cast<u64*>(ws + kCalibHeader);
    u64* b = reinterpret_cast<u64*>(ws + kCalibHeader + words_bytes(n));
    const int n_tiles = tiles_of(n);
    unsigned int* hist = reinterpret_cast<unsigned int*>(ws + kCalibHeader + 2 * words_bytes(n));
    unsigned int* tile_sum = hist + align_up((size_t)kDigits * n_tiles * sizeof(unsigned int), 256) / sizeof(unsigned int);
    unsigned int* digit_total = reinterpret_cast<unsigned int*>(ws + 8);        // 256 counters inside the first 2 KB
    if (n == 0) {
        calib_empty_kernel<<<1, 1, 0, stream>>>(tau, counts);
        return cudaGetLastError() == cudaSuccess ? EE_OK : EE_ERR_CUDA;
    }
    calib_pack_kernel<<<(n + kSortThreads - 1) / kSortThreads, kSortThreads, 0, stream>>>(entropy, argmax_head,
                                                                                           argmax_final, n, a, best);
    u64 *src = a, *dst = b;
    for (int pass = 0; pass < kPasses; ++pass) {
        const int shift = 1 + 8 * pass;
        calib_hist_kernel<<<n_tiles, kSortThreads, 0, stream>>>(src, n, shift, hist, n_tiles);
        calib_scan_kernel<<<kDigits, 1024, 0, stream>>>(hist, n_tiles, digit_total);
        calib_scatter_kernel<<<n_tiles, kSortThreads, 0, stream>>>(src, dst, n, shift, hist, digit_total, n_tiles);
        u64* t = src;
        src = dst;
        dst = t;
    }
    calib_tile_sum_kernel<<<n_tiles, kSortThreads, 0, stream>>>(src, n, tile_sum);
    calib_select_kernel<<<n_tiles, kSortThreads, 0, stream>>>(src, n, tile_sum, epsilon, best);
    calib_output_kernel<<<1, 1, 0, stream>>>(src, n, best, tau, counts);
    return cudaGetLastError() == cudaSuccess ? EE_OK : EE_ERR_CUDA;
}

}  // namespace ee
