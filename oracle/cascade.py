"""fp64 CPU oracle for the inference-time cascade of exit heads (paper section 3.4.2, "Inference Process":
each input goes through the heads in order, head k answers when its confidence passes tau_k, and an input that
no head answers is left to the full model).

TEST INFRASTRUCTURE ONLY (see oracle/exit_head.py).  Shares no code with the CUDA sources.

Data-parallel form: K heads in depth order, head k reading its own hidden states h_k [M, d] (the rows of
the batch at head k's layer); a row stops at the first head whose entropy is below that head's threshold
(the exit rule of oracle.exit_head: H < tau, strict), later heads never see it.

Outputs per row: exit_head (index of the answering head, K if none), token (that head's argmax, -1 if none),
entropy (that head's entropy, NaN if none); per head: rows_in (rows it was evaluated on), the head-usage
count of the paper's Fig. 3 being rows_in[k] - rows_in[k+1].

Pins (tests/test_oracle_cascade.py): the same result from evaluating every head on every row independently
(no survivor bookkeeping), hand-built cases with known exits, conservation (every row is answered by exactly
one head or by none; rows_in is non-increasing and starts at M).
"""
from __future__ import annotations

import numpy as np

from .exit_head import exit_head


def cascade(h_list, heads, taus) -> dict:
    """h_list[k]: bf16 bit patterns [M, d] for head k; heads[k]: dict(gamma, beta, ln_eps, W); taus[k]: scalar."""
    K = len(heads)
    M = h_list[0].shape[0]
    exit_at = np.full(M, K, dtype=np.int32)
    token = np.full(M, -1, dtype=np.int32)
    entropy = np.full(M, np.nan, dtype=np.float64)
    rows_in = np.zeros(K, dtype=np.int32)
    alive = np.arange(M, dtype=np.int64)                 # rows no head has answered yet, in batch order
    per_head = []
    for k in range(K):
        rows_in[k] = alive.size
        hd = heads[k]
        out = exit_head(h_list[k][alive], hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], taus[k])
        per_head.append(dict(rows=alive.copy(), **out))
        done = out["exit_mask"] != 0
        exit_at[alive[done]] = k
        token[alive[done]] = out["argmax"][done]
        entropy[alive[done]] = out["entropy"][done]
        alive = alive[~done]
    return dict(exit_head=exit_at, token=token, entropy=entropy, rows_in=rows_in, per_head=per_head)
