"""CPU oracle for the commit step of one DSSD round (paper section 4.3.1: the three stop conditions of the
drafting phase and the atomic commit of the verification phase), for S sequences that each keep a buffer of
committed tokens.

TEST INFRASTRUCTURE ONLY (see oracle/exit_head.py).  Shares no code with the CUDA sources.  Integer work only.

Per sequence that is not finished:
  draft length n   = leading draft slots that are confident (stop iii), at most k (stop i), and not beyond the
                     first end-of-sequence token drafted (stop ii: that token is the last one drafted)
  accept length a  = leading j < n with draft_tok[j] == verify_tok[j]
  committed        = draft_tok[0 .. a) followed by verify_tok[a] when a < kv (the full model's token: the rewrite
                     of the first mismatch, the fallback after an early stop, or the bonus row), cut after the
                     first end-of-sequence token and at the buffer's capacity
  finished         = an end-of-sequence token was committed, or the buffer is full
Readings where the paper is silent: an accepted end-of-sequence token ends the sequence and no further token
follows it; a sequence that is finished is left untouched by later rounds; eos < 0 switches the stop off.
Statistics (the paper's acceptance rate and wasted tokens are ratios / differences of these): tokens drafted,
accepted, committed, and sequences that took part.

Pins (tests/test_oracle_dssd_round.py): hand-worked rounds, equality with oracle.dssd_accept when no
end-of-sequence token occurs, multi-round invariants.
"""
from __future__ import annotations

import numpy as np


def dssd_commit(draft_tok, draft_exit_mask, verify_tok, eos: int, out_tok, seq_len, finished, stats) -> dict:
    """Updates out_tok [S, cap], seq_len [S], finished [S], stats [4] in place; returns draft_len, accept_len, next_tok."""
    S, k = draft_tok.shape
    kv = verify_tok.shape[1]
    cap = out_tok.shape[1]
    draft_len = np.zeros(S, np.int32)
    accept_len = np.zeros(S, np.int32)
    next_tok = np.full(S, -1, np.int32)
    for s in range(S):
        if finished[s]:
            continue
        n = 0
        while n < k and (draft_exit_mask is None or draft_exit_mask[s, n] != 0):
            n += 1
            if eos >= 0 and draft_tok[s, n - 1] == eos:
                break
        a = 0
        while a < n and draft_tok[s, a] == verify_tok[s, a]:
            a += 1
        commit = [int(t) for t in draft_tok[s, :a]]
        ended = eos >= 0 and a > 0 and commit[-1] == eos
        if not ended and a < kv:
            next_tok[s] = verify_tok[s, a]
            commit.append(int(verify_tok[s, a]))
        room = cap - int(seq_len[s])
        commit = commit[:room]
        out_tok[s, seq_len[s]:seq_len[s] + len(commit)] = commit
        seq_len[s] += len(commit)
        if (eos >= 0 and eos in commit) or seq_len[s] >= cap:
            finished[s] = 1
        draft_len[s], accept_len[s] = n, a
        stats += np.array([n, a, len(commit), 1], dtype=stats.dtype)
    return dict(draft_len=draft_len, accept_len=accept_len, next_tok=next_tok)
