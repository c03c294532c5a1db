// LayerNorm of bf16 rows whose result, rounded to bf16, is the correctly rounded value of the exact expression
//   y_j = (x_j - mean) / sqrt(var + eps) * gamma_j + beta_j      (biased variance, eps under the root)
// and therefore the value an fp64 evaluation rounds to (an fp64 result is 2^-29 bf16 units from the exact one, so
// the two can differ only for an element that close to a bf16 midpoint).
//
// How: the row statistics are accumulated in fp64 (three fp64 operations per element; B200 runs them at half the
// fp32 rate).  Every element is then normalised in fp32 together with a bound B on the error of that fp32 value
// against the exact one; if y - B and y + B round to the same bf16 value, so does the exact y (rounding is
// monotonic) and the fp32 result stands.  Otherwise -- about one element in a thousand -- the element is redone
// in fp64 and converted with a single rounding.
//
// Error bound of the fp32 path (u = 2^-24; mu, R = 1/sqrt(var + eps) exact up to fp64 rounding; mu_f, R_f their
// fp32 roundings; t = (x - mu) R):
//   fl(x - mu_f)        differs from x - mu by at most u (|mu| + |x - mu|)
//   times R_f, rounded  adds 2 u |t|                      -> |t_f - t| <= u (|mu| R + 3 |t|)
//   fma(t_f, g, b)      adds u |y|                        -> |y_f - y| <= u ((|mu| R + 3 |t|) |g| + |y|) =: u Q
// to first order.  B = 3 u Q leaves room for the second-order terms, for Q being evaluated in fp32 from the
// computed quantities, and for the roundings of y - B and y + B themselves (each at most u |y| <= u Q).
#pragma once

#include "common.cuh"

namespace ee {

struct RowStats {
    double mu, rstd;          // mean and 1 / sqrt(var + eps)
    float mu_f, rstd_f;       // their fp32 roundings
    float c0;                 // |mu_f| * rstd_f, the row-constant part of the error bound
};

__device__ __forceinline__ double bf16_lo_d(uint32_t v) { return (double)bf16_lo(v); }
__device__ __forceinline__ double bf16_hi_d(uint32_t v) { return (double)bf16_hi(v); }

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum of the eight elements of a 16-byte vector, added to acc (two chains, so that the additions pipeline).
__device__ __forceinline__ void vec8_sum_d(uint4 v, double& acc0, double& acc1) {
    acc0 += bf16_lo_d(v.x);
    acc1 += bf16_hi_d(v.x);
    acc0 += bf16_lo_d(v.y);
    acc1 += bf16_hi_d(v.y);
    acc0 += bf16_lo_d(v.z);
    acc1 += bf16_hi_d(v.z);
    acc0 += bf16_lo_d(v.w);
    acc1 += bf16_hi_d(v.w);
}

// Sum of the squared deviations from mu of the eight elements, added to acc.
__device__ __forceinline__ void vec8_sqdev_d(uint4 v, double mu, double& acc0, double& acc1) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const double a = bf16_lo_d(w[i]) - mu, b = bf16_hi_d(w[i]) - mu;
        acc0 = fma(a, a, acc0);
        acc1 = fma(b, b, acc1);
    }
}

__device__ __forceinline__ RowStats row_stats(double mu, double sum_sqdev, double inv_d, float ln_eps) {
    RowStats st;
    st.mu = mu;
    st.rstd = 1.0 / sqrt(sum_sqdev * inv_d + (double)ln_eps);
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

// One element: bf16 bits (low 16 bits of the result) of the correctly rounded LayerNorm output.
__device__ __forceinline__ uint32_t layer_norm_elem(float x, const RowStats& st, float g, float b) {
    const float t = (x - st.mu_f) * st.rstd_f;
    const float y = fmaf(t, g, b);
    const float q = fmaf(fmaf(3.f, fabsf(t), st.c0), fabsf(g), fabsf(y));
    const float B = 1.8e-7f * q;                                   // 3 u Q
    const uint32_t both = pack_bf16(y - B, y + B);                 // low half: y - B, high half: y + B
    const uint32_t lo = both & 0xffffu, hi = both >> 16;
    if (lo == hi) return lo;
    // The interval straddles a bf16 midpoint: decide in fp64.
    return bf16_from_double(fma(((double)x - st.mu) * st.rstd, (double)g, (double)b));
}

// Eight consecutive elements (one 16-byte vector of bf16) -> eight bf16, given the gammas / betas of these columns.
__device__ __forceinline__ uint4 layer_norm_vec8(uint4 v, const RowStats& st, float4 g0, float4 g1, float4 b0, float4 b1) {
    uint4 o;
    o.x = layer_norm_elem(bf16_lo(v.x), st, g0.x, b0.x) | (layer_norm_elem(bf16_hi(v.x), st, g0.y, b0.y) << 16);
    o.y = layer_norm_elem(bf16_lo(v.y), st, g0.z, b0.z) | (layer_norm_elem(bf16_hi(v.y), st, g0.w, b0.w) << 16);
    o.z = layer_norm_elem(bf16_lo(v.z), st, g1.x, b1.x) | (layer_norm_elem(bf16_hi(v.z), st, g1.y, b1.y) << 16);
    o.w = layer_norm_elem(bf16_lo(v.w), st, g1.z, b1.z) | (layer_norm_elem(bf16_hi(v.w), st, g1.w, b1.w) << 16);
    return o;
}

// Same, reading gamma and beta of vector c (columns 8c .. 8c+7) from global memory (weights: read-only path).
__device__ __forceinline__ uint4 layer_norm_vec8(uint4 v, const RowStats& st, const float* gamma, const float* beta, int c) {
    const float4 g0 = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * c);
    const float4 g1 = __ldg(reinterpret_cast<const float4*>(gamma) + 2 * c + 1);
    const float4 b0 = __ldg(reinterpret_cast<const float4*>(beta) + 2 * c);
    const float4 b1 = __ldg(reinterpret_cast<const float4*>(beta) + 2 * c + 1);
    return layer_norm_vec8(v, st, g0, g1, b0, b1);
}

// Statistics of a row that one warp holds lane-strided: `load(c)` returns vector c (columns 8c .. 8c+7) for
// c < nvec.  Two passes over the row (mean, then squared deviations -- the definition, which does not cancel).
template <class LoadFn>
__device__ __forceinline__ RowStats row_stats_strided(LoadFn load, int nvec, double inv_d, float ln_eps, int lane) {
    double s0 = 0.0, s1 = 0.0;
    for (int c = lane; c < nvec; c += 32) vec8_sum_d(load(c), s0, s1);
    const double mu = warp_sum_d(s0 + s1) * inv_d;
    double q0 = 0.0, q1 = 0.0;
    for (int c = lane; c < nvec; c += 32) vec8_sqdev_d(load(c), mu, q0, q1);
    return row_stats(mu, warp_sum_d(q0 + q1), inv_d, ln_eps);
}

// ---------------------------------------------------------------------------------------------
// LayerNorm of rows that already sit in shared memory as raw bf16 (16-byte vectors reached through
// vec(row, c)), in place.  A warp keeps R whole rows in registers (up to VPL vectors per lane), so each row is
// read once and the R dependency chains (two warp reductions each) overlap.  Requires nvec <= 32 * VPL.
// ---------------------------------------------------------------------------------------------
template <int R, int VPL, class VecFn>
__device__ __forceinline__ void layer_norm_rows_in_regs(VecFn vec, const int (&rows)[R], int n_rows, int nvec, float ln_eps,
                                                        const float* gamma_s, const float* beta_s, int lane) {
    uint4 x[R][VPL];
    double mu[R], sq[R];
    const double inv_d = 1.0 / (double)(nvec * 8);
#pragma unroll
    for (int i = 0; i < R; ++i) {
        double s0 = 0.0, s1 = 0.0;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            const int c = lane + 32 * k;
            x[i][k] = (i < n_rows && c < nvec) ? *vec(rows[i], c) : make_uint4(0, 0, 0, 0);
            vec8_sum_d(x[i][k], s0, s1);
        }
        mu[i] = s0 + s1;
    }
#pragma unroll
    for (int i = 0; i < R; ++i) mu[i] = warp_sum_d(mu[i]) * inv_d;
#pragma unroll
    for (int i = 0; i < R; ++i) {
        double q0 = 0.0, q1 = 0.0;
#pragma unroll
        for (int k = 0; k < VPL; ++k)
            if (lane + 32 * k < nvec) vec8_sqdev_d(x[i][k], mu[i], q0, q1);
        sq[i] = q0 + q1;
    }
    RowStats st[R];
#pragma unroll
    for (int i = 0; i < R; ++i) st[i] = row_stats(mu[i], warp_sum_d(sq[i]), inv_d, ln_eps);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        const int c = lane + 32 * k;
        if (c < nvec) {
            const float4* g4 = reinterpret_cast<const float4*>(gamma_s) + 2 * c;
            const float4* b4 = reinterpret_cast<const float4*>(beta_s) + 2 * c;
            const float4 g0 = g4[0], g1 = g4[1], b0 = b4[0], b1 = b4[1];
#pragma unroll
            for (int i = 0; i < R; ++i)
                if (i < n_rows) *vec(rows[i], c) = layer_norm_vec8(x[i][k], st[i], g0, g1, b0, b1);
        }
    }
}

}  // namespace ee
