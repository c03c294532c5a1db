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


def _model3(seed=0, V=400, d=64, sigmas=(1.2, 0.6)):
    """Three heads on three tables: two noisy drafting layers (the shallower one noisier) and the full model."""
    cfg = gen.make_config("c1", seed=seed, planted=True, M=4, d=d, V=V, heads=3)
    planting = gen.make_planting(seed, f"c1/planted/d{d}/V{V}", d, V)
    tables = [gen.make_markov_model(seed + 10 * i, V, d, planting, sigma=sg) for i, sg in enumerate(sigmas)]
    return cfg, [t["E_draft"] for t in tables], tables[0]["E_verify"], tables


def _fresh(S, cap):
    return (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))


def test_round_with_one_draft_head_is_the_single_head_round():
    cfg, mm = _model()
    S, k, cap = 9, 5, 40
    start = np.arange(S, dtype=np.int32) * 11 % 400
    a, b = _fresh(S, cap), _fresh(S, cap)
    la, lb = start.copy(), start.copy()
    use = np.zeros(1, np.int64)
    for _ in range(3):
        ra = oracle.dssd_round(mm["E_draft"], mm["E_verify"], cfg["heads"][0], cfg["heads"][1], 1.0, -1, k, la, *a)
        rb = oracle.dssd_round_multi([mm["E_draft"]], mm["E_verify"], [cfg["heads"][0]], cfg["heads"][1], [1.0], -1, k, lb, *b, use)
        for key in ("draft_len", "accept_len", "next_tok", "draft_mask"):
            assert np.array_equal(ra[key], rb[key]), key
        live = rb["draft_mask"] != 0                                    # tokens of confident slots are the head's own
        assert np.array_equal(ra["draft_tok"][live], rb["draft_tok"][live])
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
    assert np.array_equal(la, lb) and use[0] == a[3][0]                 # every drafted position came from the one head


def test_multi_head_round_position_by_position_is_the_cascade():
    cfg, E_drafts, E_verify, _ = _model3()
    S, k, cap = 24, 4, 40
    start = (np.arange(S, dtype=np.int32) * 7 + 3) % 400
    st, last, use = _fresh(S, cap), start.copy(), np.zeros(2, np.int64)
    taus = [0.5, 1.5]
    r = oracle.dssd_round_multi(E_drafts, E_verify, cfg["heads"][:2], cfg["heads"][2], taus, -1, k, last, *st, use)
    cur = start.astype(np.int64)
    for j in range(k):
        c = oracle.cascade([E[cur] for E in E_drafts], cfg["heads"][:2], taus)       # the same rows, evaluated independently
        assert np.array_equal(r["draft_head"][:, j], c["exit_head"])
        answered = c["exit_head"] < 2
        assert np.array_equal(r["draft_mask"][:, j], answered.astype(np.uint8))
        assert np.array_equal(r["draft_tok"][answered, j], c["token"][answered])
        # first head whose entropy is below its threshold, checked from every head's own evaluation
        H = [oracle.exit_head(E[cur], hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], t)["entropy"]
             for E, hd, t in zip(E_drafts, cfg["heads"][:2], taus)]
        first = np.where(H[0] < taus[0], 0, np.where(H[1] < taus[1], 1, 2))
        assert np.array_equal(first, c["exit_head"])
        cur = r["draft_tok"][:, j].astype(np.int64)
    # usage counts only positions inside the draft, of sequences that took part
    want = np.zeros(2, np.int64)
    for s in range(S):
        for j in range(r["draft_len"][s]):
            want[r["draft_head"][s, j]] += 1
    assert np.array_equal(use, want) and use.sum() == st[3][0] and (r["draft_head"][r["draft_mask"] == 0] == 2).all()
    assert use[0] > 0 and use[1] > 0                                    # both heads supply tokens in this case


def test_multi_head_round_commits_the_full_models_greedy_chain():
    cfg, E_drafts, E_verify, tables = _model3(seed=2)
    S, k, cap = 8, 6, 80
    start = np.arange(S, dtype=np.int32) * 13 % 400
    want = _greedy(dict(E_verify=E_verify), cfg["heads"][2], start, 30)
    st, last, use = _fresh(S, cap), start.copy(), np.zeros(2, np.int64)
    for _ in range(4):
        oracle.dssd_round_multi(E_drafts, E_verify, cfg["heads"][:2], cfg["heads"][2], [1.0, 2.0], -1, k, last, *st, use)
    for s in range(S):
        assert np.array_equal(st[0][s, :st[1][s]], want[s, :st[1][s]])
    assert st[1].sum() > 4 * S                                          # drafts were accepted somewhere
    # thresholds that nothing passes: one token per round, no head ever used
    st, last, use = _fresh(S, cap), start.copy(), np.zeros(2, np.int64)
    for _ in range(3):
        oracle.dssd_round_multi(E_drafts, E_verify, cfg["heads"][:2], cfg["heads"][2], [-1.0, -1.0], -1, k, last, *st, use)
    assert (st[1] == 3).all() and use.sum() == 0 and np.array_equal(st[0][:, :3], want[:, :3])
