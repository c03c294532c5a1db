"""Pins for the oracle's bf16 rounding and LayerNorm (step A1)."""
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import torch

import oracle
from gen import bf16_bits_from_f32


def _finite_patterns():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    with np.errstate(invalid="ignore"):      # signalling-NaN patterns warn when widened
        vals = oracle.bf16_decode(bits)
    keep = np.isfinite(vals)
    return bits[keep], vals[keep]


def test_bf16_round_trip_is_identity_on_every_pattern():
    _, vals = _finite_patterns()
    assert np.array_equal(oracle.bf16_rne(vals), vals)


def test_bf16_midpoints_go_to_even_and_neighbours_go_to_nearest():
    bits, vals = _finite_patterns()
    pos = vals >= 0
    order = np.argsort(vals[pos])
    v = vals[pos][order]
    b = bits[pos][order].astype(np.int64)
    lo, hi = v[:-1], v[1:]
    mid = (lo + hi) / 2            # exact in fp64
    even_is_lo = (b[:-1] % 2) == 0
    want = np.where(even_is_lo, lo, hi)
    assert np.array_equal(oracle.bf16_rne(mid), want)
    assert np.array_equal(oracle.bf16_rne(-mid), -want)
    # a hair above / below the midpoint must not be treated as a tie (no double rounding through fp32)
    above = np.nextafter(mid, np.inf)
    below = np.nextafter(mid, -np.inf)
    assert np.array_equal(oracle.bf16_rne(above), hi)
    assert np.array_equal(oracle.bf16_rne(below[1:]), lo[1:])


def test_bf16_matches_an_independent_converter_on_fp32_inputs():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(200000).astype(np.float32) * 3,
                        (rng.standard_normal(1000) * 1e-39).astype(np.float32),
                        np.float32([0.0, -0.0, 1.0, 3.3895314e38, 1e-45])])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = oracle.bf16_rne(x.astype(np.float64))
    assert np.array_equal(got, want)
    # and the input packer used by the generators agrees with both
    assert np.array_equal(oracle.bf16_decode(bf16_bits_from_f32(x)), want)


def test_bf16_overflow_and_specials():
    big = 2.0 ** 128 * (1 - 2.0 ** -9)          # exactly half-way between bf16 max and 2^128 -> rounds to inf (even)
    assert oracle.bf16_rne(np.array([big]))[0] == np.inf
    assert oracle.bf16_rne(np.array([2.0 ** 127 * 1.99]))[0] == 2.0 ** 127 * (2 - 2.0 ** -7)
    out = oracle.bf16_rne(np.array([np.inf, -np.inf, np.nan, 0.0]))
    assert out[0] == np.inf and out[1] == -np.inf and np.isnan(out[2]) and out[3] == 0.0


def _bits(x):
    return bf16_bits_from_f32(np.asarray(x, dtype=np.float32))


def test_layer_norm_alternating_signs_gives_exactly_plus_minus_one():
    d = 64
    x = np.tile([1.0, -1.0], d // 2)[None, :]
    y = oracle.layer_norm(_bits(x), np.ones(d, np.float32), np.zeros(d, np.float32), 1e-5)
    # mean 0, variance 1, 1/sqrt(1+1e-5) = 0.999995 which rounds to 1 in bf16
    assert np.array_equal(y, x)
    y_exact = oracle.layer_norm(_bits(x), np.ones(d, np.float32), np.zeros(d, np.float32), 1e-5, round_to_bf16=False)
    assert np.allclose(np.abs(y_exact), 1 / np.sqrt(1 + 1e-5), rtol=0, atol=1e-15)


def test_layer_norm_constant_row_returns_beta():
    d = 40
    beta = np.linspace(-1, 1, d).astype(np.float32)
    gamma = np.full(d, 3.0, np.float32)
    y = oracle.layer_norm(_bits(np.full((2, d), 2.5)), gamma, beta, 1e-5)
    assert np.array_equal(y, np.tile(oracle.bf16_rne(beta.astype(np.float64)), (2, 1)))


def test_layer_norm_against_50_digit_decimal_arithmetic():
    getcontext().prec = 50
    rng = np.random.default_rng(7)
    d = 12
    h = _bits(rng.standard_normal((3, d)) * 2 + 0.7)
    gamma = (1 + 0.1 * rng.standard_normal(d)).astype(np.float32)
    beta = (0.02 * rng.standard_normal(d)).astype(np.float32)
    eps = 1e-5
    y = oracle.layer_norm(h, gamma, beta, eps, round_to_bf16=False)
    x = oracle.bf16_decode(h)
    for i in range(3):
        xs = [Decimal(float(v)) for v in x[i]]
        mu = sum(xs) / d
        var = sum((v - mu) ** 2 for v in xs) / d            # biased: divide by d
        inv = 1 / (var + Decimal(eps)).sqrt()                # eps under the root
        for j in range(d):
            want = (xs[j] - mu) * inv * Decimal(float(gamma[j])) + Decimal(float(beta[j]))
            assert abs(Decimal(float(y[i, j])) - want) < Decimal("1e-14")


def test_layer_norm_invariants_before_affine():
    rng = np.random.default_rng(3)
    d = 256
    h = _bits(rng.standard_normal((5, d)) * 4 - 1)
    y = oracle.layer_norm(h, np.ones(d, np.float32), np.zeros(d, np.float32), 1e-5, round_to_bf16=False)
    x = oracle.bf16_decode(h)
    var = x.var(axis=1)
    assert np.allclose(y.mean(axis=1), 0, atol=1e-14)
    assert np.allclose((y * y).mean(axis=1), var / (var + 1e-5), rtol=1e-13)
    # rows are independent and a row is unchanged by what else is in the batch
    y0 = oracle.layer_norm(h[2:3], np.ones(d, np.float32), np.zeros(d, np.float32), 1e-5, round_to_bf16=False)
    assert np.array_equal(y0[0], y[2])


def test_layer_norm_exact_rational_case_d4():
    # x = (0, 0, 0, 4): mu = 1, var = 3, so with eps = 0 y = (-1, -1, -1, 3)/sqrt(3)
    y = oracle.layer_norm(_bits([[0, 0, 0, 4]]), np.ones(4, np.float32), np.zeros(4, np.float32), 0.0,
                          round_to_bf16=False)[0]
    assert np.allclose(y * y, [float(Fraction(1, 3))] * 3 + [3.0], rtol=4e-16, atol=0)
    assert (y[:3] < 0).all() and y[3] > 0
