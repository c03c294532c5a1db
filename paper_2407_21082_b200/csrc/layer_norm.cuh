// LayerNorm of bf16 rows whose result, rounded to bf16, is the correctly rounded value of the exact expression
//   y_j = (x_j - mean) / sqrt(var + eps) * gamma_j + beta_j      (biased variance, eps under the root)
// and therefore the value an fp64 evaluation rounds to (an fp64 result is 2^-29 bf16 units from the exact one, so
// the two can differ only for an element that close to a bf16 midpoint).
//
// How: the row's moments (sum x, sum x^2; x^2 of a bf16 value is exact) are accumulated in fp64, which B200 runs
// at half the fp32 rate, in one pass; var = E[x^2] - mean^2 loses log2(E[x^2] / var) of fp64's 53 bits, so when
// that is more than 12 bits (|mean| above 64 standard deviations) the squared deviations are summed in a second
// pass, as the definition has it.  Every element is then normalised in fp32 together with a bound B on the error
// of that fp32 value against the exact one; if no bf16 midpoint lies within B of y, the exact value rounds to the
// bf16 value y rounds to (rounding is monotonic) and the fp32 result stands.  Otherwise -- about one element in a thousand -- the
// element is redone in fp64 and converted with a single rounding.
//
// Error bound of the fp32 path (u = 2^-24; mu, R = 1/sqrt(var + eps) exact up to fp64 rounding; mu_f = fl(mu);
// R_f = fl(R); t = (x - mu) R):
//   fl(x - mu_f)        differs from x - mu by at most u (|mu| + |x - mu|)
//   times R_f, rounded  adds 2 u |t|                      -> |t_f - t| <= u (|mu| R + 3 |t|)
//   fma(t_f, g, b)      adds u |y|                        -> |y_f - y| <= u ((|mu| R + 3 |t|) |g| + |y|) =: u Q
// to first order.  B = 2 u Q' with Q' = (|mu| R + 4 |t|) |g| + |y| leaves room for the second-order terms, for Q'
// being evaluated in fp32 from the computed quantities.
#pragma once

#include "common.cuh"

namespace ee {

// Four LayerNorm parameters through the read-only path.  An ordered (volatile) load on purpose: a plain __ldg is
// free to move, and in a loop over a row's vectors the compiler lifts all of them to the top, sixteen registers
// per vector.
__device__ __forceinline__ float4 ld_param4(const float* p) {
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

struct RowStats {
    double mu, rstd;          // mean and 1 / sqrt(var + eps) in fp64
    float mu_f, rstd_f;       // their fp32 roundings
    float c0;                 // |mu_f| * rstd_f, the row-constant part of the error bound
};

// (Measured, 64 elements per lane, one warp per scheduler: conversion instruction + tree of fp64 operations 1180
// cycles; doubles assembled with integer instructions and a branch for zero / subnormal / infinite values 4630;
// fp32 arithmetic alone 690.  The conversion instruction is not what costs.)
__device__ __forceinline__ double bf16_lo_d(uint32_t v) { return (double)bf16_lo(v); }
__device__ __forceinline__ double bf16_hi_d(uint32_t v) { return (double)bf16_hi(v); }

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ void warp_sum2_d(double& a, double& b) {      // two sums whose shuffles overlap
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double oa = __shfl_xor_sync(0xffffffffu, a, o), ob = __shfl_xor_sync(0xffffffffu, b, o);
        a += oa;
        b += ob;
    }
}

// Running moments of a lane's share of a row.  An fp64 operation has a latency of some sixty cycles on this part
// (its throughput, half of fp32, shows only with dozens of operations in flight), so nothing here is a long
// dependent chain: the eight elements of a vector are summed as a tree, and a vector adds one operation to each
// of two alternating accumulators.
struct Moments {
    double s[2], q[2];
    __device__ __forceinline__ void clear() { s[0] = s[1] = q[0] = q[1] = 0.0; }
    __device__ __forceinline__ void add(uint4 v, int k) {             // the eight elements of vector number k of the lane
        const double x0 = bf16_lo_d(v.x), x1 = bf16_hi_d(v.x), x2 = bf16_lo_d(v.y), x3 = bf16_hi_d(v.y);
        const double x4 = bf16_lo_d(v.z), x5 = bf16_hi_d(v.z), x6 = bf16_lo_d(v.w), x7 = bf16_hi_d(v.w);
        const double sa = (x0 + x1) + (x2 + x3), sb = (x4 + x5) + (x6 + x7);
        const double qa = fma(x1, x1, x0 * x0) + fma(x3, x3, x2 * x2), qb = fma(x5, x5, x4 * x4) + fma(x7, x7, x6 * x6);
        s[k & 1] += sa + sb;
        q[k & 1] += qa + qb;
    }
    __device__ __forceinline__ double sum() const { return s[0] + s[1]; }
    __device__ __forceinline__ double sum_sq() const { return q[0] + q[1]; }
};

// Sum of the squared deviations from mu of the eight elements, added to acc (the second pass, when it is needed).
__device__ __forceinline__ void vec8_sqdev_d(uint4 v, double mu, double& acc0, double& acc1) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const double a = bf16_lo_d(w[i]) - mu, b = bf16_hi_d(w[i]) - mu;
        acc0 = fma(a, a, acc0);
        acc1 = fma(b, b, acc1);
    }
}

// From the warp-wide moments: mean and E[x^2] - mean^2, with multiplications by 1/d instead of divisions (a
// division is a chain of some thirty dependent operations).  The mean gets one correction step, r = sum - mean d
// exactly (fused), mean += r / d, after which a row of equal values has exactly that value as its mean, as it has
// with a true division (and, after the second pass, a variance of exactly zero).  False if the subtraction cancels
// more than 12 bits: the caller then sums the squared deviations.
__device__ __forceinline__ bool row_variance_one_pass(double sum, double sum_sq, double d, double inv_d, double& mu, double& var) {
    const double m0 = sum * inv_d;
    mu = fma(fma(-m0, d, sum), inv_d, m0);
    const double ex2 = sum_sq * inv_d;
    var = fma(-mu, mu, ex2);
    return var * 4096.0 >= ex2;
}

// 1 / sqrt(v) in fp64 from the fp32 estimate and one Newton step: relative error about 2^-43, a thousand times
// finer than the doubtful elements need, in four dependent operations (the library routine takes some fifteen).
__device__ __forceinline__ double rsqrt_newton(double v) {
    const float vf = (float)v;
    if (!(vf < 3e38f) || vf < 1e-37f) return rsqrt(v);                // outside fp32's comfortable range (or NaN)
    const double r = (double)rsqrtf(vf);
    const double h = 0.5 * r;
    return fma(fma(-v * r, r, 1.0), h, r);                            // r + r (1 - v r^2) / 2
}

__device__ __forceinline__ RowStats row_stats(double mu, double var, float ln_eps) {
    RowStats st;
    st.mu = mu;
    st.rstd = rsqrt_newton(fmax(var, 0.0) + (double)ln_eps);
    st.mu_f = (float)mu;
    st.rstd_f = (float)st.rstd;
    st.c0 = fabsf(st.mu_f) * st.rstd_f;
    return st;
}

// fp64 -> bf16 with one rounding (to nearest, ties to even): truncate to fp32, make the last bit sticky
// (round to odd), then round the 24-bit value to 8 bits.
__device__ __forceinline__ uint32_t bf16_from_double(double v) {
    float f = __double2float_rz(v);
    if ((double)f != v) f = __uint_as_float(__float_as_uint(f) | 1u);
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// One element on the fp32 path: y, and whether the exact value may round to another bf16 value than y does
// (`doubt`): that is the case when the bf16 midpoint nearest to y -- y's bits with the low half replaced by 0x8000 --
// lies within B of y (y - mid is exact in fp32: the two share their upper sixteen bits).
__device__ __forceinline__ float layer_norm_elem_fast(float x, const RowStats& st, float g, float b, uint32_t& doubt) {
    const float t = (x - st.mu_f) * st.rstd_f;
    const float y = fmaf(t, g, b);
    const float q = fmaf(fmaf(4.f, fabsf(t), st.c0), fabsf(g), fabsf(y));
    const float mid = __uint_as_float((__float_as_uint(y) & 0xffff0000u) | 0x8000u);
    const float B = 1.2e-7f * q;                                   // 2 u Q'
    // (second test: a bound so coarse that midpoints other than the nearest come into reach -- everything is doubtful)
    doubt = (fabsf(y - mid) <= B || B * 2048.f >= fabsf(y)) ? 1u : 0u;
    return y;
}

// Eight consecutive elements (one 16-byte vector of bf16) on the fp32 path; bit e of `doubts` is set if element e
// has to be redone in fp64.
__device__ __forceinline__ uint4 layer_norm_vec8_fast(uint4 v, const RowStats& st, float4 g0, float4 g1, float4 b0, float4 b1,
                                                      uint32_t& doubts) {
    uint32_t d0, d1, d2, d3, d4, d5, d6, d7;
    uint4 o;
    o.x = pack_bf16(layer_norm_elem_fast(bf16_lo(v.x), st, g0.x, b0.x, d0), layer_norm_elem_fast(bf16_hi(v.x), st, g0.y, b0.y, d1));
    o.y = pack_bf16(layer_norm_elem_fast(bf16_lo(v.y), st, g0.z, b0.z, d2), layer_norm_elem_fast(bf16_hi(v.y), st, g0.w, b0.w, d3));
    o.z = pack_bf16(layer_norm_elem_fast(bf16_lo(v.z), st, g1.x, b1.x, d4), layer_norm_elem_fast(bf16_hi(v.z), st, g1.y, b1.y, d5));
    o.w = pack_bf16(layer_norm_elem_fast(bf16_lo(v.w), st, g1.z, b1.z, d6), layer_norm_elem_fast(bf16_hi(v.w), st, g1.w, b1.w, d7));
    doubts = d0 | (d1 << 1) | (d2 << 2) | (d3 << 3) | (d4 << 4) | (d5 << 5) | (d6 << 6) | (d7 << 7);
    return o;
}

// The elements of a vector named in `doubts` (about one element in two thousand), decided in fp64 and put into y.
__device__ __forceinline__ uint4 layer_norm_vec8_redo_inline(uint4 v, uint4 y, double mu, double rstd, float4 g0, float4 g1,
                                                             float4 b0, float4 b1, uint32_t doubts) {
    const uint32_t xw[4] = {v.x, v.y, v.z, v.w};
    uint32_t yw[4] = {y.x, y.y, y.z, y.w};
    const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        if ((doubts >> e) & 1u) {
            const float x = (e & 1) ? bf16_hi(xw[e >> 1]) : bf16_lo(xw[e >> 1]);
            const uint32_t r = bf16_from_double(fma(((double)x - mu) * rstd, (double)g[e], (double)b[e]));
            yw[e >> 1] = (e & 1) ? ((yw[e >> 1] & 0x0000ffffu) | (r << 16)) : ((yw[e >> 1] & 0xffff0000u) | r);
        }
    }
    return make_uint4(yw[0], yw[1], yw[2], yw[3]);
}
// Out of line, for loops that are not unrolled over a row's vectors: it runs rarely and would otherwise be
// replicated, with its registers, at every call site.
static __device__ __noinline__ uint4 layer_norm_vec8_redo(uint4 v, uint4 y, double mu, double rstd, float4 g0, float4 g1, float4 b0,
                                                          float4 b1, uint32_t doubts) {
    return layer_norm_vec8_redo_inline(v, y, mu, rstd, g0, g1, b0, b1, doubts);
}

// Eight consecutive elements -> eight correctly rounded bf16, given the gammas / betas of these columns.
__device__ __forceinline__ uint4 layer_norm_vec8(uint4 v, const RowStats& st, float4 g0, float4 g1, float4 b0, float4 b1) {
    uint32_t doubts;
    uint4 o = layer_norm_vec8_fast(v, st, g0, g1, b0, b1, doubts);
    if (doubts) o = layer_norm_vec8_redo(v, o, st.mu, st.rstd, g0, g1, b0, b1, doubts);
    return o;
}

// Same, reading gamma and beta of vector c (columns 8c .. 8c+7) from global memory (weights: read-only path).
__device__ __forceinline__ uint4 layer_norm_vec8(uint4 v, const RowStats& st, const float* gamma, const float* beta, int c) {
    const float4 g0 = ld_param4(gamma + 8 * c);
    const float4 g1 = ld_param4(gamma + 8 * c + 4);
    const float4 b0 = ld_param4(beta + 8 * c);
    const float4 b1 = ld_param4(beta + 8 * c + 4);
    return layer_norm_vec8(v, st, g0, g1, b0, b1);
}

// For a caller that keeps a row's vectors in registers: the fp32 path alone, with the doubts handed back, so that
// the unrolled loop over its vectors stays short; it redoes the doubtful vectors afterwards (layer_norm_vec8_redo_at).
__device__ __forceinline__ uint4 layer_norm_vec8_fast(uint4 v, const RowStats& st, const float* gamma, const float* beta, int c,
                                                      uint32_t& doubts) {
    const float4 g0 = ld_param4(gamma + 8 * c);
    const float4 g1 = ld_param4(gamma + 8 * c + 4);
    const float4 b0 = ld_param4(beta + 8 * c);
    const float4 b1 = ld_param4(beta + 8 * c + 4);
    return layer_norm_vec8_fast(v, st, g0, g1, b0, b1, doubts);
}
__device__ __forceinline__ void layer_norm_vec8_redo_at(uint4 x, uint4* y_vec, const RowStats& st, const float* gamma,
                                                        const float* beta, int c, uint32_t doubts) {
    const float4 g0 = ld_param4(gamma + 8 * c);
    const float4 g1 = ld_param4(gamma + 8 * c + 4);
    const float4 b0 = ld_param4(beta + 8 * c);
    const float4 b1 = ld_param4(beta + 8 * c + 4);
    *y_vec = layer_norm_vec8_redo_inline(x, *y_vec, st.mu, st.rstd, g0, g1, b0, b1, doubts);
}

// Statistics of a row that one warp holds lane-strided: `load(c)` returns vector c (columns 8c .. 8c+7) for
// c < nvec.
template <class LoadFn>
__device__ __forceinline__ RowStats row_stats_strided(LoadFn load, int nvec, float ln_eps, int lane) {
    const double d = (double)(nvec * 8), inv_d = 1.0 / d;
    Moments m;
    m.clear();
    int k = 0;
    for (int c = lane; c < nvec; c += 32, ++k) m.add(load(c), k);
    double s = m.sum(), q = m.sum_sq();
    warp_sum2_d(s, q);
    double mu, var;
    if (!row_variance_one_pass(s, q, d, inv_d, mu, var)) {
        double q0 = 0.0, q1 = 0.0;
        for (int c = lane; c < nvec; c += 32) vec8_sqdev_d(load(c), mu, q0, q1);
        var = warp_sum_d(q0 + q1) * inv_d;
    }
    return row_stats(mu, var, ln_eps);
}

// ---------------------------------------------------------------------------------------------
// LayerNorm of rows that already sit in shared memory as raw bf16 (16-byte vectors reached through
// vec(row, c)), in place.  A warp works on R rows at a time so that their dependency chains (two warp
// reductions each) overlap; every pass re-reads the rows from shared memory, which keeps the register count low.
// ---------------------------------------------------------------------------------------------
template <int R, class VecFn>
__device__ __forceinline__ void layer_norm_rows_in_smem(VecFn vec, const int (&rows)[R], int n_rows, int nvec, float ln_eps,
                                                        const float* gamma_s, const float* beta_s, int lane) {
    const double d = (double)(nvec * 8), inv_d = 1.0 / d;
    Moments m[R];
#pragma unroll
    for (int i = 0; i < R; ++i) m[i].clear();
    int k = 0;
    for (int c = lane; c < nvec; c += 32, ++k) {
#pragma unroll
        for (int i = 0; i < R; ++i)
            if (i < n_rows) m[i].add(*vec(rows[i], c), k);
    }
    RowStats st[R];
#pragma unroll
    for (int i = 0; i < R; ++i) {
        double s = m[i].sum(), q = m[i].sum_sq();
        warp_sum2_d(s, q);
        double mu, var;
        if (!row_variance_one_pass(s, q, d, inv_d, mu, var) && i < n_rows) {
            double q0 = 0.0, q1 = 0.0;
            for (int c = lane; c < nvec; c += 32) vec8_sqdev_d(*vec(rows[i], c), mu, q0, q1);
            var = warp_sum_d(q0 + q1) * inv_d;
        }
        st[i] = row_stats(mu, var, ln_eps);
    }
    for (int c = lane; c < nvec; c += 32) {
        const float4* g4 = reinterpret_cast<const float4*>(gamma_s) + 2 * c;
        const float4* b4 = reinterpret_cast<const float4*>(beta_s) + 2 * c;
        const float4 g0 = g4[0], g1 = g4[1], b0 = b4[0], b1 = b4[1];
#pragma unroll
        for (int i = 0; i < R; ++i)
            if (i < n_rows) {
                uint4* v = vec(rows[i], c);
                *v = layer_norm_vec8(*v, st[i], g0, g1, b0, b1);
            }
    }
}

}  // namespace ee
