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


def dssd_round(E_draft, E_verify, draft_head, verify_head, tau: float, eos: int, k: int, last_tok, out_tok, seq_len,
               finished, stats) -> dict:
    """One whole DSSD round (drafting phase, verification phase, commit) for S sequences, with the hidden state of
    a position given by a table row of the previous token (the tests' stand-in for the transformer).

    Drafting: k steps; step j evaluates the draft head on E_draft[previous token] (the last committed token for
    j = 0, the token drafted at j - 1 after that); its argmax is the drafted token, its exit decision the
    confidence.  Verification: the full model's head on E_verify[previous token] for the k draft positions and
    one bonus position, all at once.  Then dssd_commit.  last_tok is updated to each sequence's last committed
    token.  Every sequence goes through all k steps (what lies beyond its stop is ignored by the commit)."""
    from .exit_head import exit_head
    S = last_tok.size
    cur = last_tok.astype(np.int64).copy()
    draft = np.zeros((S, k), np.int32)
    mask = np.zeros((S, k), np.uint8)
    steps = []
    for j in range(k):
        o = exit_head(E_draft[cur], draft_head["gamma"], draft_head["beta"], draft_head["ln_eps"], draft_head["W"], tau)
        draft[:, j], mask[:, j] = o["argmax"], o["exit_mask"]
        cur = o["argmax"].astype(np.int64)
        steps.append(o)
    prev_all = np.concatenate([last_tok.astype(np.int64)[:, None], draft.astype(np.int64)], axis=1)      # [S, k + 1]
    v = exit_head(E_verify[prev_all.reshape(-1)], verify_head["gamma"], verify_head["beta"], verify_head["ln_eps"],
                  verify_head["W"], np.inf)
    verify = v["argmax"].reshape(S, k + 1).astype(np.int32)
    was_finished = finished.copy()
    r = dssd_commit(draft, mask, verify, eos, out_tok, seq_len, finished, stats)
    for s in range(S):
        if not was_finished[s] and seq_len[s] > 0:
            last_tok[s] = out_tok[s, seq_len[s] - 1]
    return dict(draft_tok=draft, draft_mask=mask, verify_tok=verify, steps=steps, verify_out=v, **r)



def dssd_round_multi(E_drafts, E_verify, draft_heads, verify_head, taus, eos: int, k: int, last_tok, out_tok, seq_len,
                     finished, stats, head_use) -> dict:
    """One whole DSSD round with K draft heads (paper section 4.3.1, drafting phase: at every position the heads
    are tried from the shallowest to the deepest and the first one whose entropy is below its threshold supplies
    the token; a position that no head is sure of ends the draft -- stop (iii), the fallback to the full model).

    E_drafts[h] is the table of hidden states at head h's layer (row = previous token), draft_heads[h] that head,
    taus[h] its threshold.  Step j runs oracle.cascade on the S rows of the step: a sequence's token and
    confidence at position j are those of the answering head; where no head answers the slot is not confident and
    carries the deepest head's argmax (never committed: the draft stopped before it; it only feeds the later,
    ignored steps).  Verification and commit as in dssd_round.  head_use [K] (int64) accumulates, over the sequences
    that took part, the positions inside the draft (j < draft_len) supplied by each head: the head-usage figure of
    the paper's DSSD experiments; the mean exit head is sum(h * head_use[h]) / sum(head_use).
    """
    from .cascade import cascade
    from .exit_head import exit_head
    K = len(draft_heads)
    S = last_tok.size
    cur = last_tok.astype(np.int64).copy()
    draft = np.zeros((S, k), np.int32)
    mask = np.zeros((S, k), np.uint8)
    which = np.full((S, k), K, np.int32)
    steps = []
    for j in range(k):
        c = cascade([E[cur] for E in E_drafts], draft_heads, taus)
        tok = c["token"].copy()
        none = c["exit_head"] == K
        if none.any():                                   # the deepest head saw exactly the rows nobody answered before it
            last = c["per_head"][K - 1]
            pos = {int(r): i for i, r in enumerate(last["rows"])}
            for s in np.flatnonzero(none):
                tok[s] = last["argmax"][pos[int(s)]]
        draft[:, j], mask[:, j], which[:, j] = tok, (~none).astype(np.uint8), c["exit_head"]
        cur = tok.astype(np.int64)
        steps.append(c)
    prev_all = np.concatenate([last_tok.astype(np.int64)[:, None], draft.astype(np.int64)], axis=1)
    v = exit_head(E_verify[prev_all.reshape(-1)], verify_head["gamma"], verify_head["beta"], verify_head["ln_eps"],
                  verify_head["W"], np.inf)
    verify = v["argmax"].reshape(S, k + 1).astype(np.int32)
    was_finished = finished.copy()
    r = dssd_commit(draft, mask, verify, eos, out_tok, seq_len, finished, stats)
    for s in range(S):
        if was_finished[s]:
            continue
        if seq_len[s] > 0:
            last_tok[s] = out_tok[s, seq_len[s] - 1]
        for j in range(int(r["draft_len"][s])):
            head_use[which[s, j]] += 1
    return dict(draft_tok=draft, draft_mask=mask, draft_head=which, verify_tok=verify, steps=steps, verify_out=v, **r)
