"""fp64 CPU oracle for the calibration of a head's confidence threshold (paper section 3.4.1,
"Calibration of Confidence Thresholds": Eq. 3 defines the correctness indicator, the two unnumbered
equations after it define the index j-hat and the threshold tau_k = c_{k, j-hat}).

TEST INFRASTRUCTURE ONLY (see oracle/exit_head.py).  Shares no code with the CUDA sources.

The paper's procedure, in its notation: c_k holds the confidence of head k on each of the M_cal calibration
tokens (larger = surer), t_k whether the head's prediction equals the full model's.  Sort both by c
ascending; j-hat is the smallest index whose suffix has accuracy >= epsilon; tau = c at j-hat; at inference
the head answers when c >= tau.

With the entropy H as the metric, c = -H: "c >= tau_c" is "H <= tau" with tau = -tau_c, the entropy at j-hat.
Readings where the text is silent:
  * ties: the suffix condition is evaluated on whole groups of equal confidence (the paper's prose counts every
    sample whose metric is at least the candidate value), so the result does not depend on how a sort orders
    equal values;
  * no index qualifies (the surest group is already below epsilon): the head never answers, tau = -inf;
  * the threshold returned is the paper's (a sample AT the threshold is inside the set); a caller whose rule
    is the strict H < tau passes the next float above it.
Everything is integer counting except the comparison  correct >= epsilon * count,  done in fp64.

Pins (tests/test_oracle_calibrate.py): hand-worked examples, the definition enumerated index by index on the
paper's own formula for inputs without ties, permutation invariance, the guarantee (accuracy of the chosen set
>= epsilon) and its maximality (every larger candidate set that qualifies would have been chosen).
"""
from __future__ import annotations

import numpy as np


def correctness(argmax_head: np.ndarray, argmax_final: np.ndarray) -> np.ndarray:
    """Eq. 3: t_j = 1 iff the head's prediction equals the full model's prediction on token j."""
    return (np.asarray(argmax_head) == np.asarray(argmax_final)).astype(np.uint8)


def calibrate_threshold_bruteforce(entropy: np.ndarray, correct: np.ndarray, epsilon: float) -> dict:
    """The definition candidate by candidate (quadratic; for small inputs and for pinning the sorted version)."""
    H = np.asarray(entropy, dtype=np.float64)
    t = np.asarray(correct).astype(np.int64)
    n = H.size
    if np.isnan(H).any():
        raise ValueError("calibration entropies must not be NaN")
    best = None
    # candidate thresholds are the distinct entropies; the set of a candidate v is {j : H_j <= v}
    for v in np.unique(H):                      # ascending entropy = descending confidence
        inside = H <= v
        count = int(inside.sum())
        hits = int(t[inside].sum())
        if float(hits) >= float(epsilon) * float(count):
            best = (float(v), count, hits)      # keep the largest qualifying entropy = the smallest index j-hat
    if best is None:
        return dict(tau=float("-inf"), n_exit=0, n_correct=0, j_hat=0)
    tau, count, hits = best
    return dict(tau=tau, n_exit=count, n_correct=hits, j_hat=n - count + 1)


def calibrate_threshold(entropy: np.ndarray, correct: np.ndarray, epsilon: float) -> dict:
    """tau (entropy at j-hat), the number of calibration tokens with H <= tau, how many of those are correct,
    and j-hat itself (1-based index in the ascending-confidence order, 0 if no index qualifies).

    The paper's steps: sort jointly by the metric, running count of correct predictions, the condition at every
    index that closes a group of equal values, the most permissive index that satisfies it."""
    H = np.asarray(entropy, dtype=np.float64)
    t = np.asarray(correct).astype(np.int64)
    n = H.size
    if n == 0:
        return dict(tau=float("-inf"), n_exit=0, n_correct=0, j_hat=0)
    if np.isnan(H).any():
        raise ValueError("calibration entropies must not be NaN")
    order = np.argsort(H, kind="stable")        # ascending entropy: surest first
    Hs, ts = H[order], t[order]
    hits = np.cumsum(ts)                         # correct among the i+1 surest
    count = np.arange(1, n + 1, dtype=np.int64)
    group_end = np.ones(n, dtype=bool)
    group_end[:-1] = Hs[1:] != Hs[:-1]
    ok = group_end & (hits.astype(np.float64) >= float(epsilon) * count.astype(np.float64))
    idx = np.flatnonzero(ok)
    if idx.size == 0:
        return dict(tau=float("-inf"), n_exit=0, n_correct=0, j_hat=0)
    i = int(idx[-1])
    return dict(tau=float(Hs[i]), n_exit=i + 1, n_correct=int(hits[i]), j_hat=n - i)
