"""fp64 CPU oracle for the early-exit decision and the DSSD verify step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the CUDA library is compared
against.  Only the test-suite, the smoke check and the CPU-baseline leg of the benchmark may import it;
the product never does, and it shares no code with the CUDA sources.

What is computed, per hidden-state row (paper section 3.2 "Implementation Details": a head is a
classifier shaped like the model's final head on the hidden features of a block; section 3.4.1: the
confidence metric is the entropy of the predicted distribution; Eq. 2: the prediction is the argmax;
section 3.4.2 and the DSSD drafting paragraph of section 4.3.1: exit when H < tau; section 4.3.1
verification paragraph: accept the matching prefix, rewrite the first mismatch):

  A1  LayerNorm in fp64 (biased variance, eps under the root), result rounded to bf16
  A2  logits z = y @ W^T in fp64
  A3  m = max z, argmax = lowest index of m, s = sum exp(z-m), H = ln s - sum exp(z-m)(z-m) / s,
      p_max = 1/s
  A4  exit = H < tau
  A5  order-preserving list of rows that did not exit, and a copy of their input rows
  A6  draft length  = number of leading confident draft rows of a sequence
  A7  accept length = number of leading drafted tokens equal to the verifier's tokens;
      next token    = verifier's token at that position (or -1 past the verifier's last row)

Pins (tests/test_oracle_*.py): exhaustive bf16 round trip, ties-to-even midpoints and a second bf16
converter; 50-digit decimal LayerNorm; exact-rational projections; closed-form entropies (uniform,
one-hot, two-level), -sum p ln p by compensated summation, shift invariance; hand-worked compaction and
acceptance cases plus brute force.  The end-to-end pipeline on the full-size synthetic workloads has no
external reference: parity unpinned beyond those parts.
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------- bf16 <-> fp64


def bf16_decode(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp64 values (exact)."""
    u32 = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def bf16_rne(x: np.ndarray) -> np.ndarray:
    """Round fp64 values to the nearest bf16 value (ties to even), returned as fp64.

    bf16 has 8 significant bits and fp32's exponent range.  For |x| in [2^e, 2^(e+1)) the bf16 grid has
    spacing 2^(e-7); below 2^-126 the spacing stays 2^-133 (subnormals).  Dividing by the spacing is an
    exact power-of-two scaling, rint() rounds half to even, so there is a single rounding.
    """
    x = np.asarray(x, dtype=np.float64)
    out = x.copy()
    fin = np.isfinite(x) & (x != 0.0)
    xf = x[fin]
    _, e = np.frexp(xf)                      # xf = mant * 2^e with mant in [0.5, 1)
    e = np.maximum(e - 1, -126)              # floor(log2 |x|), clamped at the smallest normal exponent
    q = np.ldexp(xf, 7 - e)                  # |q| < 2^8, exact
    r = np.ldexp(np.rint(q), e - 7)
    r = np.where(np.abs(r) >= 2.0 ** 128, np.copysign(np.inf, r), r)
    out[fin] = r
    return out


# ----------------------------------------------------------------------------- A1 .. A4


def layer_norm(h_bits: np.ndarray, gamma: np.ndarray, beta: np.ndarray, ln_eps: float,
               round_to_bf16: bool = True) -> np.ndarray:
    """A1.  h_bits uint16 [M, d]; gamma, beta fp32 [d].  Returns fp64 [M, d]."""
    x = bf16_decode(h_bits)
    d = x.shape[1]
    mu = x.sum(axis=1, keepdims=True) / d
    xc = x - mu
    var = (xc * xc).sum(axis=1, keepdims=True) / d
    y = xc / np.sqrt(var + float(ln_eps)) * gamma.astype(np.float64) + beta.astype(np.float64)
    return bf16_rne(y) if round_to_bf16 else y


def logits(y: np.ndarray, W_bits: np.ndarray) -> np.ndarray:
    """A2.  z[i, v] = sum_j W[v, j] * y[i, j] in fp64."""
    return y @ bf16_decode(W_bits).T


def softmax_stats(z: np.ndarray) -> dict:
    """A3.  Entropy (nats), max probability, argmax (lowest index), the top-2 logit gap, and the difference
    between the two largest probabilities (the third confidence metric of section 3.4.1, the tie-breaking one)."""
    m = z.max(axis=1, keepdims=True)
    argmax = np.argmax(z, axis=1).astype(np.int32)           # numpy returns the first maximum
    zc = z - m
    e = np.exp(zc)
    s = e.sum(axis=1)
    t = (e * zc).sum(axis=1)
    p = e / s[:, None]
    if z.shape[1] > 1:
        top2 = np.partition(z, -2, axis=1)[:, -2:]
        gap = top2[:, 1] - top2[:, 0]
        top2p = np.partition(p, -2, axis=1)[:, -2:]          # the two largest probabilities (equal maxima count twice)
        prob_gap = top2p[:, 1] - top2p[:, 0]
    else:
        gap = np.full(z.shape[0], np.inf)
        prob_gap = p[:, 0].copy()                            # a single class: nothing to subtract
    return dict(argmax=argmax, entropy=np.log(s) - t / s, maxprob=1.0 / s, logZ=m[:, 0] + np.log(s),
                top2_gap=gap, top2_prob_gap=prob_gap)


def exit_decision(entropy: np.ndarray, tau) -> np.ndarray:
    """A4.  1 where H < tau (tau scalar or per row), else 0.  NaN entropy never exits."""
    return (entropy < np.asarray(tau, dtype=np.float64)).astype(np.uint8)


def exit_head(h_bits, gamma, beta, ln_eps, W_bits, tau, rows_per_block: int = 64,
              round_to_bf16: bool = True) -> dict:
    """A1-A4 over all rows.  tau is a scalar or an array [M] (nats)."""
    M = h_bits.shape[0]
    Wd = bf16_decode(W_bits).T.copy()        # [d, V] fp64, decoded once
    keys = ("argmax", "entropy", "maxprob", "logZ", "top2_gap", "top2_prob_gap")
    parts = {k: [] for k in keys}
    for r0 in range(0, M, rows_per_block):
        y = layer_norm(h_bits[r0:r0 + rows_per_block], gamma, beta, ln_eps, round_to_bf16)
        st = softmax_stats(y @ Wd)
        for k in keys:
            parts[k].append(st[k])
    out = {k: (np.concatenate(v) if v else np.zeros(0)) for k, v in parts.items()}
    out["argmax"] = out["argmax"].astype(np.int32)
    tau_arr = np.broadcast_to(np.asarray(tau, dtype=np.float64), (M,))
    out["exit_mask"] = exit_decision(out["entropy"], tau_arr)
    out["tau_margin"] = np.abs(out["entropy"] - tau_arr)
    return out


# ----------------------------------------------------------------------------- A5


def compact(exit_mask: np.ndarray, h_bits: np.ndarray | None = None) -> dict:
    """A5.  Rows with exit_mask == 0 continue: ascending indices, their count, their input rows."""
    kept_idx = np.flatnonzero(np.asarray(exit_mask) == 0).astype(np.int32)
    out = dict(kept_idx=kept_idx, kept_count=int(kept_idx.size))
    if h_bits is not None:
        out["h_out"] = h_bits[kept_idx].copy()
    return out


# ----------------------------------------------------------------------------- A6, A7


def dssd_accept(draft_tok: np.ndarray, draft_exit_mask: np.ndarray | None, verify_tok: np.ndarray) -> dict:
    """A6/A7.  draft_tok [S, k], draft_exit_mask [S, k] or None (all confident), verify_tok [S, kv >= k]."""
    S, k = draft_tok.shape
    kv = verify_tok.shape[1]
    draft_len = np.zeros(S, dtype=np.int32)
    accept_len = np.zeros(S, dtype=np.int32)
    next_tok = np.zeros(S, dtype=np.int32)
    for s in range(S):
        n = 0
        while n < k and (draft_exit_mask is None or draft_exit_mask[s, n] != 0):
            n += 1
        a = 0
        while a < n and draft_tok[s, a] == verify_tok[s, a]:
            a += 1
        draft_len[s], accept_len[s] = n, a
        next_tok[s] = verify_tok[s, a] if a < kv else -1
    return dict(draft_len=draft_len, accept_len=accept_len, next_tok=next_tok)


# ----------------------------------------------------------------------------- comparison rule


def decisive_rows(ref: dict, gap_min: float = 1e-3, margin_min: float = 1e-3) -> dict:
    """Rows on which integer outputs must match bit for bit.

    A row is listed and excluded from the argmax comparison when its two largest logits are closer
    than gap_min, and from the exit-mask comparison when |H - tau| < margin_min.
    """
    return dict(argmax=ref["top2_gap"] >= gap_min, exit_mask=ref["tau_margin"] >= margin_min)
