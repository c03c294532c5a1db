"""Pins of the DSSD commit oracle (paper section 4.3.1)."""
import numpy as np

import gen
import oracle


def _state(S, cap):
    return (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))


def _one(draft, conf, verify, eos, cap=16, seq0=0):
    out, sl, fin, st = _state(1, cap)
    sl[0] = seq0
    r = oracle.dssd_commit(np.array([draft], np.int32), np.array([conf], np.uint8), np.array([verify], np.int32), eos, out, sl, fin, st)
    return out[0], int(sl[0]), int(fin[0]), st.tolist(), {k: int(v[0]) for k, v in r.items()}


def test_hand_worked_rounds():
    # all four confident and matching, a bonus row from the verifier: 4 accepted + the bonus token
    out, n, fin, st, r = _one([5, 6, 7, 8], [1, 1, 1, 1], [5, 6, 7, 8, 9], eos=0)
    assert out[:5].tolist() == [5, 6, 7, 8, 9] and n == 5 and fin == 0 and st == [4, 4, 5, 1] and r["next_tok"] == 9
    # mismatch at slot 2: two accepted, the verifier's token rewrites slot 2
    out, n, fin, st, r = _one([5, 6, 7, 8], [1, 1, 1, 1], [5, 6, 1, 8, 9], eos=0)
    assert out[:3].tolist() == [5, 6, 1] and n == 3 and st == [4, 2, 3, 1] and (r["draft_len"], r["accept_len"]) == (4, 2)
    # the head loses confidence at slot 1: one token drafted, accepted, then the full model's token
    out, n, fin, st, r = _one([5, 6, 7, 8], [1, 0, 1, 1], [5, 3, 7, 8, 9], eos=0)
    assert out[:2].tolist() == [5, 3] and st == [1, 1, 2, 1]
    # end of sequence drafted at slot 1 and accepted: drafting stops there, nothing follows it, finished
    out, n, fin, st, r = _one([5, 0, 7, 8], [1, 1, 1, 1], [5, 0, 7, 8, 9], eos=0)
    assert out[:2].tolist() == [5, 0] and n == 2 and fin == 1 and st == [2, 2, 2, 1] and r["next_tok"] == -1
    # end of sequence drafted but the verifier disagrees: rewritten, not finished
    out, n, fin, st, r = _one([5, 0, 7, 8], [1, 1, 1, 1], [5, 4, 7, 8, 9], eos=0)
    assert out[:2].tolist() == [5, 4] and fin == 0 and st == [2, 1, 2, 1]
    # the verifier's own token is the end of sequence
    out, n, fin, st, r = _one([5, 6, 7, 8], [1, 1, 1, 1], [5, 0, 7, 8, 9], eos=0)
    assert out[:2].tolist() == [5, 0] and fin == 1 and st == [4, 1, 2, 1]
    # buffer nearly full: the commit is cut at the capacity and the sequence is finished
    out, n, fin, st, r = _one([5, 6, 7, 8], [1, 1, 1, 1], [5, 6, 7, 8, 9], eos=0, cap=6, seq0=3)
    assert out[3:6].tolist() == [5, 6, 7] and n == 6 and fin == 1 and st == [4, 4, 3, 1]
    # kv == k and everything accepted: no row left for a next token
    out, n, fin, st, r = _one([5, 6], [1, 1], [5, 6], eos=-1)
    assert out[:2].tolist() == [5, 6] and n == 2 and r["next_tok"] == -1 and st == [2, 2, 2, 1]


def test_without_end_of_sequence_it_is_dssd_accept():
    for seed in range(5):
        case = gen.random_token_case(seed, S=60, k=8, kv=9, alphabet=4)
        out, sl, fin, st = _state(60, 64)
        r = oracle.dssd_commit(case["draft_tok"], case["draft_exit_mask"], case["verify_tok"], -1, out, sl, fin, st)
        ref = oracle.dssd_accept(case["draft_tok"], case["draft_exit_mask"], case["verify_tok"])
        for key in ("draft_len", "accept_len", "next_tok"):
            assert np.array_equal(r[key], ref[key]), key
        assert np.array_equal(sl, ref["accept_len"] + (ref["next_tok"] >= 0))
        assert st.tolist() == [ref["draft_len"].sum(), ref["accept_len"].sum(), sl.sum(), 60]


def test_rounds_accumulate_and_finished_sequences_are_left_alone():
    S, k, kv, cap, eos = 40, 6, 7, 20, 2
    out, sl, fin, st = _state(S, cap)
    for rnd in range(8):
        case = gen.random_token_case(100 + rnd, S=S, k=k, kv=kv, alphabet=5)
        before = (out.copy(), sl.copy(), fin.copy())
        oracle.dssd_commit(case["draft_tok"], case["draft_exit_mask"], case["verify_tok"], eos, out, sl, fin, st)
        was = before[2] != 0
        assert np.array_equal(out[was], before[0][was]) and np.array_equal(sl[was], before[1][was]) and fin[was].all()
        assert (sl <= cap).all() and (sl >= before[1]).all()
        for s in range(S):
            row = out[s, :sl[s]]
            assert (row != -9).all() and (out[s, sl[s]:] == -9).all()
            if eos in row:
                assert fin[s] and row[-1] == eos and (row[:-1] != eos).all()     # nothing after the end of sequence
            assert fin[s] == (eos in row or sl[s] >= cap)
    assert fin.sum() > 0 and st[2] == sl.sum() and st[1] <= st[0]


def _model(seed=0, V=400, d=64):
    cfg = gen.make_config("c1", seed=seed, planted=True, M=4, d=d, V=V, heads=2)
    planting = gen.make_planting(seed, f"c1/planted/d{d}/V{V}", d, V)
    mm = gen.make_markov_model(seed, V, d, planting, sigma=0.4)
    return cfg, mm


def _greedy(mm, head, start, n):
    """Plain autoregressive decoding with the full model's head: token after t = argmax head(E_verify[t])."""
    out, cur = [], start.astype(np.int64)
    for _ in range(n):
        o = oracle.exit_head(mm["E_verify"][cur], head["gamma"], head["beta"], head["ln_eps"], head["W"], np.inf)
        cur = o["argmax"].astype(np.int64)
        out.append(cur.copy())
    return np.stack(out, axis=1)


def test_round_reduces_to_greedy_decoding_in_the_two_limits():
    cfg, mm = _model()
    S, k, cap = 6, 4, 64
    start = np.arange(S, dtype=np.int32) * 7 % 400
    want = _greedy(mm, cfg["heads"][1], start, 12)
    # (a) the draft head is never confident: every round commits exactly the full model's next token
    st = (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))
    last = start.copy()
    for _ in range(5):
        oracle.dssd_round(mm["E_draft"], mm["E_verify"], cfg["heads"][0], cfg["heads"][1], -1.0, -1, k, last, *st)
    assert np.array_equal(st[0][:, :5], want[:, :5]) and (st[1] == 5).all() and st[3].tolist() == [0, 0, 5 * S, 5 * S]
    # (b) the draft is the full model itself and always confident: every round commits k + 1 tokens of the same chain
    st = (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))
    last = start.copy()
    for _ in range(2):
        oracle.dssd_round(mm["E_verify"], mm["E_verify"], cfg["heads"][1], cfg["heads"][1], np.inf, -1, k, last, *st)
    assert (st[1] == 2 * (k + 1)).all() and np.array_equal(st[0][:, :10], want[:, :10])
    assert st[3].tolist() == [2 * k * S, 2 * k * S, 2 * (k + 1) * S, 2 * S]
    # (c) any threshold in between: the committed text is still the full model's greedy chain (speculation never
    #     changes the output), only the number of rounds needed differs
    st = (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))
    last = start.copy()
    for _ in range(3):
        oracle.dssd_round(mm["E_draft"], mm["E_verify"], cfg["heads"][0], cfg["heads"][1], 1.0, -1, k, last, *st)
    for s in range(S):
        assert np.array_equal(st[0][s, :st[1][s]], want[s, :st[1][s]])
    assert 3 * S <= st[1].sum() <= 3 * (k + 1) * S and st[3][1] <= st[3][0]
