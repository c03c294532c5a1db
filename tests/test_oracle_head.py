"""Pins for the oracle's projection, softmax statistics and exit decision (steps A2-A4)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from gen import bf16_bits_from_f32, make_config


def _bits(x):
    return bf16_bits_from_f32(np.asarray(x, dtype=np.float32))


def _closed_forms(golden_dir):
    rows = []
    for line in open(os.path.join(golden_dir, "closed_forms.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, V, n, a, H, p = [f.strip() for f in line.split(";")]
        rows.append((name, int(V), int(n), float(a), float(H), float(p)))
    return rows


# ------------------------------------------------------------------ A2 projection

def test_projection_exact_rationals_brute_force():
    rng = np.random.default_rng(11)
    M, d, V = 3, 7, 5                        # V != d so a transposed operand cannot even multiply
    y = oracle.bf16_rne(rng.standard_normal((M, d)))
    Wb = _bits(rng.standard_normal((V, d)))
    z = oracle.logits(y, Wb)
    Wv = oracle.bf16_decode(Wb)
    for i in range(M):
        for v in range(V):
            want = sum(Fraction(float(Wv[v, j])) * Fraction(float(y[i, j])) for j in range(d))
            assert abs(Fraction(float(z[i, v])) - want) <= abs(want) * Fraction(1, 2 ** 48) + Fraction(1, 2 ** 60)


def test_projection_plus_minus_one_rows_sum_dyadic_weights_exactly():
    d, V = 16, 6
    y = np.tile([1.0, -1.0], d // 2)[None, :]
    Wv = (np.arange(V * d).reshape(V, d) % 13 - 6) / 8.0          # small dyadic rationals, exact in bf16
    z = oracle.logits(y, _bits(Wv))
    want = Wv[:, 0::2].sum(axis=1) - Wv[:, 1::2].sum(axis=1)
    assert np.array_equal(z[0], want)


def test_projection_indexing_picks_the_right_row_and_column():
    d, V = 8, 11
    Wv = np.zeros((V, d)); Wv[4, 2] = 2.0; Wv[9, 7] = -3.0
    y = np.zeros((2, d)); y[0, 2] = 1.5; y[1, 7] = 0.5
    z = oracle.logits(y, _bits(Wv))
    want = np.zeros((2, V)); want[0, 4] = 3.0; want[1, 9] = -1.5
    assert np.array_equal(z, want)


# ------------------------------------------------------------------ A3 softmax statistics

def test_closed_form_entropies(golden_dir):
    for name, V, n, a, H, p in _closed_forms(golden_dir):
        z = np.zeros((1, V)); z[0, 5 % V:5 % V + n] = a
        if n:
            assert z.sum() == n * a
        st = oracle.softmax_stats(z)
        assert st["entropy"][0] == pytest.approx(H, rel=1e-9, abs=1e-13), name
        assert st["maxprob"][0] == pytest.approx(p, rel=1e-12), name
        assert st["argmax"][0] == (5 % V if n else 0), name
    assert _closed_forms(golden_dir)[0][4] == pytest.approx(math.log(50304), rel=1e-15)


def test_entropy_equals_minus_sum_p_ln_p_and_logZ_minus_mean_logit():
    rng = np.random.default_rng(5)
    z = rng.standard_normal((4, 37)) * np.array([[0.1], [1.0], [5.0], [30.0]]) + 100.0
    st = oracle.softmax_stats(z)
    for i in range(4):
        zi = [float(v) for v in z[i]]
        mx = max(zi)
        Z = math.fsum(math.exp(v - mx) for v in zi)
        p = [math.exp(v - mx) / Z for v in zi]
        H1 = -math.fsum(pi * math.log(pi) for pi in p if pi > 0)
        H2 = (mx + math.log(Z)) - math.fsum(pi * v for pi, v in zip(p, zi))
        assert st["entropy"][i] == pytest.approx(H1, abs=1e-12)
        assert st["entropy"][i] == pytest.approx(H2, abs=1e-11)
        assert st["maxprob"][i] == pytest.approx(max(p), rel=1e-13)
        assert st["logZ"][i] == pytest.approx(mx + math.log(Z), rel=1e-14)
        assert st["argmax"][i] == zi.index(mx)


def test_shift_invariance_and_tie_break_and_gap():
    rng = np.random.default_rng(6)
    z = rng.standard_normal((3, 50))
    a, b = oracle.softmax_stats(z), oracle.softmax_stats(z + 123.25)
    assert np.allclose(a["entropy"], b["entropy"], atol=1e-12) and np.array_equal(a["argmax"], b["argmax"])
    t = np.zeros((1, 9)); t[0, [6, 2, 8]] = 1.0
    st = oracle.softmax_stats(t)
    assert st["argmax"][0] == 2 and st["top2_gap"][0] == 0.0
    u = np.array([[0.0, 3.0, 1.0, 2.5]])
    assert oracle.softmax_stats(u)["top2_gap"][0] == 0.5


def test_partition_merge_of_partial_states_reproduces_unsplit_result():
    # the (m, s, t, idx) state of a vocabulary subset merges associatively; written here independently
    rng = np.random.default_rng(8)
    z = rng.standard_normal(1000) * 3
    full = oracle.softmax_stats(z[None, :])

    def state(lo, hi):
        seg = z[lo:hi]; m = seg.max()
        return m, np.exp(seg - m).sum(), (np.exp(seg - m) * (seg - m)).sum(), lo + int(np.argmax(seg))

    def merge(A, B):
        m = max(A[0], B[0]); aA, aB = math.exp(A[0] - m), math.exp(B[0] - m)
        s = aA * A[1] + aB * B[1]
        t = aA * (A[2] + (A[0] - m) * A[1]) + aB * (B[2] + (B[0] - m) * B[1])
        idx = A[3] if (A[0] > B[0] or (A[0] == B[0] and A[3] < B[3])) else B[3]
        return m, s, t, idx

    cuts = [0, 1, 17, 400, 401, 999, 1000]
    acc = state(cuts[0], cuts[1])
    for lo, hi in zip(cuts[1:-1], cuts[2:]):
        acc = merge(acc, state(lo, hi))
    m, s, t, idx = acc
    assert math.log(s) - t / s == pytest.approx(full["entropy"][0], abs=1e-12)
    assert 1 / s == pytest.approx(full["maxprob"][0], rel=1e-13) and idx == full["argmax"][0]


def test_gaussian_logits_entropy_is_about_lnV_minus_half_variance():
    rng = np.random.default_rng(9)
    V, sig = 50304, 0.45
    H = oracle.softmax_stats(rng.standard_normal((4, V)) * sig)["entropy"]
    assert np.allclose(H, math.log(V) - sig ** 2 / 2, atol=0.01)


# ------------------------------------------------------------------ A1-A4 whole head on tiny shapes

def _brute_head(h_bits, gamma, beta, eps, W_bits, tau):
    """Pure-python loops: LayerNorm, bf16 rounding by exhaustive nearest search, dot products, entropy."""
    grid_bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    with np.errstate(invalid="ignore"):
        grid = oracle.bf16_decode(grid_bits)
    grid = np.unique(grid[np.isfinite(grid)])
    x = oracle.bf16_decode(h_bits); W = oracle.bf16_decode(W_bits)
    out = []
    for row in x:
        d = len(row)
        mu = math.fsum(row) / d
        var = math.fsum((v - mu) ** 2 for v in row) / d
        y = []
        for j in range(d):
            val = (row[j] - mu) / math.sqrt(var + eps) * float(gamma[j]) + float(beta[j])
            k = int(np.searchsorted(grid, val))
            cands = grid[max(k - 1, 0):k + 1]
            y.append(float(cands[np.argmin(np.abs(cands - val))]))
        zs = [math.fsum(float(W[v, j]) * y[j] for j in range(d)) for v in range(W.shape[0])]
        mx = max(zs); Z = math.fsum(math.exp(v - mx) for v in zs)
        H = -math.fsum((math.exp(v - mx) / Z) * ((v - mx) - math.log(Z)) for v in zs)
        out.append((zs.index(mx), H, 1 / Z, int(H < tau)))
    return out


@pytest.mark.parametrize("M,d,V", [(3, 8, 5), (2, 16, 7), (1, 8, 1)])
def test_exit_head_against_pure_python_brute_force(M, d, V):
    rng = np.random.default_rng(100 + V)
    h = _bits(rng.standard_normal((M, d)) * 2)
    gamma = (1 + 0.1 * rng.standard_normal(d)).astype(np.float32)
    beta = (0.02 * rng.standard_normal(d)).astype(np.float32)
    W = _bits(rng.standard_normal((V, d)))
    tau = 1.0
    got = oracle.exit_head(h, gamma, beta, 1e-5, W, tau)
    for i, (am, H, p, ex) in enumerate(_brute_head(h, gamma, beta, 1e-5, W, tau)):
        assert got["argmax"][i] == am
        assert got["entropy"][i] == pytest.approx(H, abs=1e-12)
        assert got["maxprob"][i] == pytest.approx(p, rel=1e-12)
        assert got["exit_mask"][i] == ex


def test_exit_head_row_blocking_does_not_change_results():
    c = make_config("c0", seed=3, planted=True, M=9, V=257, d=64)
    hd = c["heads"][0]
    a = oracle.exit_head(c["h"], hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, rows_per_block=64)
    b = oracle.exit_head(c["h"], hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, rows_per_block=2)
    for k in ("argmax", "entropy", "maxprob", "exit_mask"):
        assert np.array_equal(a[k], b[k])


# ------------------------------------------------------------------ A4 decision

def test_exit_rule_is_strict_and_per_row():
    H = np.array([0.5, 1.0, np.nextafter(1.0, 0), np.nextafter(1.0, 2), np.nan, 0.0])
    assert oracle.exit_decision(H, 1.0).tolist() == [1, 0, 1, 0, 0, 1]
    tau = np.array([0.4, 2.0, 0.1, 5.0, 5.0, 0.0])
    assert oracle.exit_decision(H, tau).tolist() == [0, 1, 0, 1, 0, 0]


def test_decisive_rows_lists_near_ties():
    ref = dict(top2_gap=np.array([0.5, 5e-4, 1e-3]), tau_margin=np.array([2e-4, 0.3, 1e-3]))
    keep = oracle.decisive_rows(ref)
    assert keep["argmax"].tolist() == [True, False, True] and keep["exit_mask"].tolist() == [False, True, True]


def test_top2_probability_gap_closed_forms_and_brute_force():
    """Section 3.4.1's third metric: p(1st) - p(2nd)."""
    import math
    V = 1000
    st = oracle.softmax_stats(np.zeros((1, V)))
    assert st["top2_prob_gap"][0] == 0.0                                        # uniform: no gap
    a = 3.0
    z = np.zeros((1, V)); z[0, 17] = a
    want = (math.exp(a) - 1.0) / (math.exp(a) + V - 1)                          # one raised logit
    assert abs(oracle.softmax_stats(z)["top2_prob_gap"][0] - want) < 1e-15
    z[0, 400] = a                                                                # two equal maxima: gap 0
    assert oracle.softmax_stats(z)["top2_prob_gap"][0] == 0.0
    z[0, 400] = a - 1.0
    want = (math.exp(a) - math.exp(a - 1.0)) / (math.exp(a) + math.exp(a - 1.0) + V - 2)
    assert abs(oracle.softmax_stats(z)["top2_prob_gap"][0] - want) < 1e-15
    assert oracle.softmax_stats(np.array([[2.5]]))["top2_prob_gap"][0] == 1.0   # a single class
    rng = np.random.default_rng(5)
    z = rng.normal(0, 2, size=(7, 50))
    got = oracle.softmax_stats(z)
    for i in range(7):
        p = sorted((math.exp(x - z[i].max()) for x in z[i]), reverse=True)
        tot = math.fsum(p)
        assert abs(got["top2_prob_gap"][i] - (p[0] - p[1]) / tot) < 1e-14
        assert 0.0 <= got["top2_prob_gap"][i] <= got["maxprob"][i]
    assert np.all(np.diff(np.sort(z, axis=1)[:, -2:], axis=1)[:, 0] == got["top2_gap"])
