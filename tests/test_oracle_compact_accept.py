"""Pins for compaction (A5) and the DSSD draft/accept lengths (A6, A7)."""
import os

import numpy as np
import pytest

import oracle
from gen import random_token_case


def _cases(golden_dir):
    out = []
    for line in open(os.path.join(golden_dir, "dssd_accept_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, d, c, v, want = [f.strip() for f in line.split(";")]
        out.append((name, [int(x) for x in d.split()], [int(x) for x in c.split()], [int(x) for x in v.split()],
                    [int(x) for x in want.split()]))
    return out


def test_hand_worked_accept_cases(golden_dir):
    cases = _cases(golden_dir)
    assert len(cases) >= 9
    for name, d, c, v, (n, a, nxt) in cases:
        got = oracle.dssd_accept(np.array([d], np.int32), np.array([c], np.uint8), np.array([v], np.int32))
        assert (got["draft_len"][0], got["accept_len"][0], got["next_tok"][0]) == (n, a, nxt), name


def test_accept_without_mask_means_all_confident(golden_dir):
    name, d, c, v, (n, a, nxt) = _cases(golden_dir)[0]
    got = oracle.dssd_accept(np.array([d], np.int32), None, np.array([v], np.int32))
    assert (got["draft_len"][0], got["accept_len"][0], got["next_tok"][0]) == (8, 8, -1)


@pytest.mark.parametrize("S,k,kv", [(64, 8, 8), (33, 5, 6), (7, 40, 41), (1, 1, 1)])
def test_accept_against_definition_by_enumeration(S, k, kv):
    c = random_token_case(2, S, k, kv)
    got = oracle.dssd_accept(c["draft_tok"], c["draft_exit_mask"], c["verify_tok"])
    lens = set()
    for s in range(S):
        conf = c["draft_exit_mask"][s] != 0
        n = next((j for j in range(k) if not conf[j]), k)
        same = c["draft_tok"][s] == c["verify_tok"][s, :k]
        a = max(j for j in range(n + 1) if same[:j].all())
        assert got["draft_len"][s] == n and got["accept_len"][s] == a
        assert got["next_tok"][s] == (c["verify_tok"][s, a] if a < kv else -1)
        assert 0 <= a <= n <= k
        lens.add(a)
    if S >= 33 and k >= 5:
        assert len(lens) >= 4          # the inputs exercise many prefix lengths


@pytest.mark.parametrize("mask", [
    [0, 0, 0, 0], [1, 1, 1, 1], [1, 0, 1, 0, 1, 0, 1], [0] + [1] * 40, [1] * 40 + [0], [0], [1],
    [1, 1, 0] * 11,
])
def test_compaction_hand_masks(mask):
    mask = np.array(mask, np.uint8)
    M = mask.size
    h = (np.arange(M * 6, dtype=np.uint16).reshape(M, 6) * 7 + 1).astype(np.uint16)
    got = oracle.compact(mask, h)
    want = [i for i in range(M) if mask[i] == 0]
    assert got["kept_idx"].tolist() == want and got["kept_count"] == len(want) == M - int(mask.sum())
    assert np.all(np.diff(got["kept_idx"]) > 0)
    for r, i in enumerate(want):
        assert np.array_equal(got["h_out"][r], h[i])


def test_compaction_treats_any_nonzero_byte_as_exited():
    got = oracle.compact(np.array([0, 2, 0, 255], np.uint8))
    assert got["kept_idx"].tolist() == [0, 2] and got["kept_count"] == 2
