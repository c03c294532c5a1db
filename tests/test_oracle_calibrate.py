"""Pins of the calibration oracle (paper section 3.4.1): hand-worked cases, the paper's index-by-index
definition on tie-free inputs, and the properties the threshold must have."""
import math

import numpy as np
import pytest

import oracle


def paper_definition(conf, t, eps):
    """The two equations after Eq. 3, literally: sort ascending by confidence, smallest 1-based index j whose
    suffix accuracy is >= eps, tau = c_j.  Only meaningful without ties (the order of equal values is open)."""
    order = np.argsort(conf, kind="stable")
    c, tt = np.asarray(conf, float)[order], np.asarray(t)[order]
    n = c.size
    for j in range(1, n + 1):
        if tt[j - 1:].sum() / (n - j + 1) >= eps:
            return c[j - 1], j
    return None, 0


def test_hand_worked_cases():
    # confidences 0.1 .. 0.4 (entropy = -confidence), correctness 0 1 1 1
    H = -np.array([0.1, 0.2, 0.3, 0.4])
    t = np.array([0, 1, 1, 1])
    r = oracle.calibrate_threshold(H, t, 0.75)           # whole set: 3/4 correct
    assert (r["tau"], r["n_exit"], r["n_correct"], r["j_hat"]) == (-0.1, 4, 3, 1)
    r = oracle.calibrate_threshold(H, t, 0.76)           # must drop the wrong one
    assert (r["tau"], r["n_exit"], r["n_correct"], r["j_hat"]) == (-0.2, 3, 3, 2)
    r = oracle.calibrate_threshold(H, t, 1.0)
    assert (r["tau"], r["j_hat"]) == (-0.2, 2)
    r = oracle.calibrate_threshold(H, t, 0.0)            # anything qualifies: the whole set
    assert (r["tau"], r["n_exit"]) == (-0.1, 4)
    # the surest token is wrong and epsilon = 1: nothing qualifies, the head never answers
    r = oracle.calibrate_threshold(-np.array([0.1, 0.2, 0.3]), np.array([1, 1, 0]), 1.0)
    assert r == dict(tau=float("-inf"), n_exit=0, n_correct=0, j_hat=0)
    # non-monotone suffix accuracy: the SMALLEST index wins even if a later one fails
    H = -np.array([1., 2., 3., 4., 5., 6.])
    t = np.array([1, 1, 0, 0, 1, 1])                     # suffix accuracies 4/6 3/5 2/4 2/3 1 1
    assert oracle.calibrate_threshold(H, t, 0.66)["j_hat"] == 1
    assert oracle.calibrate_threshold(H, t, 0.67)["j_hat"] == 5
    assert oracle.calibrate_threshold(np.array([]), np.array([]), 0.5)["n_exit"] == 0
    for eps in (0.0, 0.66, 0.67, 1.0):
        assert oracle.calibrate_threshold_bruteforce(H, t, eps) == oracle.calibrate_threshold(H, t, eps)


def test_ties_are_taken_as_a_group():
    # three tokens share the lowest confidence; one of them is wrong.  Splitting the group is not allowed:
    # either all three are inside the set or none.
    H = np.array([2.0, 2.0, 2.0, 1.0, 0.5])
    for perm in ([0, 1, 1, 1, 1], [1, 0, 1, 1, 1], [1, 1, 0, 1, 1]):
        r = oracle.calibrate_threshold(H, np.array(perm), 0.8)
        assert (r["tau"], r["n_exit"], r["n_correct"]) == (2.0, 5, 4)
        r = oracle.calibrate_threshold(H, np.array(perm), 0.9)
        assert (r["tau"], r["n_exit"], r["n_correct"]) == (1.0, 2, 2)


@pytest.mark.parametrize("seed", range(6))
def test_matches_the_papers_index_by_index_definition_without_ties(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 300))
    conf = rng.permutation(n).astype(np.float64) / 7.0 + 0.25          # distinct values
    p_correct = 1 / (1 + np.exp(-(conf - conf.mean()) / (conf.std() + 1e-9)))
    t = (rng.random(n) < p_correct).astype(np.uint8)
    for eps in (0.0, 0.3, 0.5, 0.8, 0.95, 1.0):
        tau_c, j = paper_definition(conf, t, eps)
        r = oracle.calibrate_threshold(-conf, t, eps)
        assert r["j_hat"] == j
        if j:
            assert r["tau"] == -tau_c and r["n_exit"] == n - j + 1
        else:
            assert r["tau"] == float("-inf")


@pytest.mark.parametrize("seed", range(4))
def test_properties_with_ties(seed):
    rng = np.random.default_rng(100 + seed)
    n = 500
    H = rng.integers(0, 40, size=n).astype(np.float64) / 8.0           # many ties
    t = (rng.random(n) < np.clip(1.0 - H / 6.0, 0, 1)).astype(np.uint8)
    for eps in (0.2, 0.5, 0.7, 0.9, 1.0):
        r = oracle.calibrate_threshold(H, t, eps)
        perm = rng.permutation(n)
        assert oracle.calibrate_threshold(H[perm], t[perm], eps) == r    # no dependence on the input order
        if r["n_exit"]:
            inside = H <= r["tau"]
            assert inside.sum() == r["n_exit"] and t[inside].sum() == r["n_correct"]
            assert r["n_correct"] >= eps * r["n_exit"]                  # the guarantee
            assert r["tau"] in H
        for v in np.unique(H):                                          # maximality: no larger set qualifies
            if v > r["tau"]:
                inside = H <= v
                assert t[inside].sum() < eps * inside.sum()


@pytest.mark.parametrize("seed", range(5))
def test_sorted_version_equals_the_candidate_by_candidate_definition(seed):
    rng = np.random.default_rng(200 + seed)
    n = int(rng.integers(1, 400))
    H = np.round(rng.gamma(2.0, 1.5, size=n), 1 if seed % 2 else 6)       # with and without many ties
    t = (rng.random(n) < np.exp(-H / 3)).astype(np.uint8)
    for eps in (0.0, 0.25, 0.5, 0.75, 0.9, 1.0):
        assert oracle.calibrate_threshold(H, t, eps) == oracle.calibrate_threshold_bruteforce(H, t, eps)


def test_correctness_indicator():
    a = np.array([3, 5, 7, 7], np.int32)
    b = np.array([3, 4, 7, 0], np.int32)
    assert oracle.correctness(a, b).tolist() == [1, 0, 1, 0]
    assert not math.isnan(oracle.calibrate_threshold(np.array([0.5]), oracle.correctness(a[:1], b[:1]), 1.0)["tau"])
