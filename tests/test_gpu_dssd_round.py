"""dssd_commit against the oracle over several rounds: buffers, lengths, flags and statistics bit for bit."""
import numpy as np
import pytest
import torch

import gen
import oracle
from _util import dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ee():
    import paper_2407_21082_b200 as ee
    return ee


@pytest.mark.parametrize("S,k,kv,cap,eos,alphabet", [(40, 6, 7, 20, 2, 5), (1, 1, 1, 3, 0, 2), (130, 32, 33, 70, 1, 6),
                                                     (17, 8, 8, 1000, -1, 3), (9, 32, 32, 33, 3, 4)])
def test_rounds_match_oracle(ee, S, k, kv, cap, eos, alphabet):
    ref_state = (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))
    state = dict(out_tok=dev(ref_state[0]), seq_len=dev(ref_state[1]), finished=dev(ref_state[2]), stats=dev(ref_state[3]))
    for rnd in range(7):
        case = gen.random_token_case(1000 * S + rnd, S=S, k=k, kv=kv, alphabet=alphabet, p_confident=0.9, p_mismatch=0.1)
        mask = case["draft_exit_mask"] if rnd % 3 else None          # every third round: no mask = all confident
        ref = oracle.dssd_commit(case["draft_tok"], mask, case["verify_tok"], eos, *ref_state)
        got = ee.dssd_commit(dev(case["draft_tok"]), dev(mask) if mask is not None else None, dev(case["verify_tok"]), eos, state)
        torch.cuda.synchronize()
        for key in ("draft_len", "accept_len", "next_tok"):
            assert np.array_equal(got[key].cpu().numpy(), ref[key]), (rnd, key)
        assert np.array_equal(state["out_tok"].cpu().numpy(), ref_state[0]), rnd
        assert np.array_equal(state["seq_len"].cpu().numpy(), ref_state[1]), rnd
        assert np.array_equal(state["finished"].cpu().numpy(), ref_state[2]), rnd
        assert state["stats"].cpu().numpy().tolist() == ref_state[3].tolist(), rnd
    assert ref_state[3][0] > 0


def test_argument_errors(ee):
    t = torch.zeros((2, 40), dtype=torch.int32, device="cuda")
    state = dict(out_tok=torch.zeros((2, 8), dtype=torch.int32, device="cuda"), seq_len=torch.zeros(2, dtype=torch.int32, device="cuda"),
                 finished=torch.zeros(2, dtype=torch.uint8, device="cuda"), stats=torch.zeros(4, dtype=torch.int64, device="cuda"))
    with pytest.raises(ee.EExitError) as e:
        ee.dssd_commit(t, None, t, 0, state)                         # k = 40 > 32
    assert e.value.code == 2


def _model(seed, V, d):
    cfg = gen.make_config("c1", seed=seed, planted=True, M=4, d=d, V=V, heads=2)
    planting = gen.make_planting(seed, f"c1/planted/d{d}/V{V}", d, V)
    return cfg, gen.make_markov_model(seed, V, d, planting, sigma=0.4)


@pytest.mark.parametrize("S,k,V,d,tau,eos", [(12, 4, 400, 64, 1.0, -1), (40, 8, 1000, 128, 0.7, 5), (3, 1, 300, 64, 5.0, -1),
                                              (70, 6, 640, 256, 1.5, 17)])
@pytest.mark.parametrize("model", ["python callback", "library table model", "chained table model"])
def test_whole_rounds_match_oracle(ee, S, k, V, d, tau, eos, model):
    """Drafting steps, verification pass and commit, several rounds in a row, against the oracle's round.  A
    sequence drops out of the comparison from the round in which one of its decisions falls inside the tolerance
    band (near-tied argmax, |H - tau| < 1e-3), because everything it does afterwards may legitimately differ."""
    from _util import GAP_MIN, MARGIN_MIN, dev_bf16, head_to_dev
    cfg, mm = _model(S + k, V, d)
    if eos >= 0:
        eos = int(gen.make_planting(S + k, f"c1/planted/d{d}/V{V}", d, V)["tokens"][eos % 64])   # a token the chain can reach
    cap = 3 * (k + 1) + 2
    start = (np.arange(S, dtype=np.int32) * 13) % V
    ref_state = (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))
    ref_last = start.copy()
    state = dict(last_tok=dev(start), out_tok=dev(ref_state[0]), seq_len=dev(ref_state[1]), finished=dev(ref_state[2]),
                 stats=dev(ref_state[3]))
    E = [dev_bf16(mm["E_draft"]), dev_bf16(mm["E_verify"])]
    calls = []

    def hidden(tokens, which, h_out):
        calls.append((which, tokens.numel()))
        torch.index_select(E[which], 0, tokens.long(), out=h_out)

    hd, hv = head_to_dev(cfg["heads"][0]), head_to_dev(cfg["heads"][1])
    rnd = ee.DssdRound(dict(gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=tau), dict(gamma=hv["gamma"], beta=hv["beta"], W=hv["W"]),
                       1e-5, k, eos, hidden if model == "python callback" else ee.TableModel(E[0], E[1], chained=model.startswith("chained")), state)
    clean = np.ones(S, bool)
    for r in range(4):
        ref = oracle.dssd_round(mm["E_draft"], mm["E_verify"], cfg["heads"][0], cfg["heads"][1], tau, eos, k, ref_last, *ref_state)
        for o in ref["steps"]:
            keep = oracle.decisive_rows(o, GAP_MIN, MARGIN_MIN)
            clean &= keep["argmax"] & keep["exit_mask"]
        clean &= oracle.decisive_rows(ref["verify_out"], GAP_MIN, MARGIN_MIN)["argmax"].reshape(S, k + 1).all(axis=1)
        got = rnd()
        torch.cuda.synchronize()
        assert ee.ee_query_async_error(rnd.workspace) == 0
        for key in ("draft_len", "accept_len", "next_tok"):
            assert np.array_equal(got[key].cpu().numpy()[clean], ref[key][clean]), (r, key)
        assert np.array_equal(state["out_tok"].cpu().numpy()[clean], ref_state[0][clean]), r
        assert np.array_equal(state["seq_len"].cpu().numpy()[clean], ref_state[1][clean]), r
        assert np.array_equal(state["finished"].cpu().numpy()[clean], ref_state[2][clean]), r
        assert np.array_equal(state["last_tok"].cpu().numpy()[clean], ref_last[clean]), r
        if clean.all():
            assert state["stats"].cpu().numpy().tolist() == ref_state[3].tolist(), r
    if model == "python callback":
        assert calls[:k + 1] == [(0, S)] * k + [(1, S * (k + 1))] and len(calls) == 4 * (k + 1)
    else:
        assert not calls
    assert clean.sum() >= S // 2                        # the case is not dominated by near-ties
    assert ref_state[1].sum() > 4 * S or tau < 0        # speculation committed more than one token per round somewhere


@pytest.mark.parametrize("S,k,V,d,taus,eos", [(12, 4, 400, 64, (1.0,), -1), (40, 8, 1000, 128, (0.4, 0.8, 1.5), 5),
                                               (3, 1, 300, 64, (0.5, 5.0, 5.0), -1), (70, 6, 640, 256, (0.6, 1.0, 2.0), 17),
                                               (33, 5, 500, 64, (0.5, 1.0, 1.0, 1.5, 2.0), -1)])
@pytest.mark.parametrize("model", ["python callback", "python callback, one call per step", "chained table model",
                                   "chained table model, one call per layer"])
def test_whole_rounds_with_several_draft_heads_match_oracle(ee, S, k, V, d, taus, eos, model):
    """K draft heads, shallowest first, each on its own layer's hidden states: per position the first confident head
    supplies the token (section 4.3.1).  State, outputs and the per-head usage counts against oracle.dssd_round_multi
    over several rounds; a sequence drops out of the comparison from the round in which one of the decisions it
    depends on falls inside the tolerance band."""
    from _util import GAP_MIN, MARGIN_MIN, dev_bf16, head_to_dev
    K = len(taus)
    seed = S + k
    cfg = gen.make_config("c1", seed=seed, planted=True, M=4, d=d, V=V, heads=K + 1)
    planting = gen.make_planting(seed, f"c1/planted/d{d}/V{V}", d, V)
    sigmas = np.linspace(1.2, 0.4, K)                                   # shallower layers are noisier
    tables = [gen.make_markov_model(seed + 10 * i, V, d, planting, sigma=float(sg)) for i, sg in enumerate(sigmas)]
    E_drafts, E_verify = [t["E_draft"] for t in tables], tables[0]["E_verify"]
    if eos >= 0:
        eos = int(planting["tokens"][eos % 64])
    cap = 3 * (k + 1) + 2
    start = (np.arange(S, dtype=np.int32) * 13) % V
    ref_state = (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))
    ref_last, ref_use = start.copy(), np.zeros(K, np.int64)
    state = dict(last_tok=dev(start), out_tok=dev(ref_state[0]), seq_len=dev(ref_state[1]), finished=dev(ref_state[2]),
                 stats=dev(ref_state[3]))
    E = [dev_bf16(t) for t in E_drafts] + [dev_bf16(E_verify)]
    calls = []

    def hidden(tokens, which, h_out):
        calls.append((which, tokens.numel()))
        if which < 0:                                                   # one forward pass: every drafting layer's states
            for layer in range(K):
                torch.index_select(E[layer], 0, tokens.long(), out=h_out[layer])
        else:
            torch.index_select(E[which], 0, tokens.long(), out=h_out)

    devs = [head_to_dev(hd) for hd in cfg["heads"]]
    drafts = [dict(gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=float(t)) for hd, t in zip(devs[:K], taus)]
    verify = dict(gamma=devs[K]["gamma"], beta=devs[K]["beta"], W=devs[K]["W"])
    if model.startswith("python callback"):
        rnd = ee.DssdRound(drafts, verify, 1e-5, k, eos, hidden, state, all_layers=model.endswith("one call per step"))
    else:
        rnd = ee.DssdRound(drafts, verify, 1e-5, k, eos, ee.TableModel(E[:K], E[K], chained=True), state,
                           all_layers=not model.endswith("one call per layer"))
    clean = np.ones(S, bool)
    for r in range(3):
        ref = oracle.dssd_round_multi(E_drafts, E_verify, cfg["heads"][:K], cfg["heads"][K], list(taus), eos, k, ref_last, *ref_state, ref_use)
        for c in ref["steps"]:                                          # every head evaluation a sequence went through
            for o in c["per_head"]:
                keep = oracle.decisive_rows(o, GAP_MIN, MARGIN_MIN)
                bad = ~(keep["argmax"] & keep["exit_mask"])
                clean[o["rows"][bad]] = False
        clean &= oracle.decisive_rows(ref["verify_out"], GAP_MIN, MARGIN_MIN)["argmax"].reshape(S, k + 1).all(axis=1)
        got = rnd()
        torch.cuda.synchronize()
        assert ee.ee_query_async_error(rnd.workspace) == 0
        for key in ("draft_len", "accept_len", "next_tok"):
            assert np.array_equal(got[key].cpu().numpy()[clean], ref[key][clean]), (r, key)
        assert np.array_equal(state["out_tok"].cpu().numpy()[clean], ref_state[0][clean]), r
        assert np.array_equal(state["seq_len"].cpu().numpy()[clean], ref_state[1][clean]), r
        assert np.array_equal(state["finished"].cpu().numpy()[clean], ref_state[2][clean]), r
        assert np.array_equal(state["last_tok"].cpu().numpy()[clean], ref_last[clean]), r
        if clean.all():
            assert state["stats"].cpu().numpy().tolist() == ref_state[3].tolist(), r
            assert rnd.head_use.cpu().numpy().tolist() == ref_use.tolist(), r
    if model == "python callback":
        assert calls[:K * k + 1] == [(h, S) for _ in range(k) for h in range(K)] + [(K, S * (k + 1))]
    if model == "python callback, one call per step":
        assert calls[:k + 1] == [(-1, S)] * k + [(K, S * (k + 1))]
    assert clean.sum() >= S // 2
    if K > 1 and clean.all():
        assert ref_use.sum() == ref_state[3][0]                         # every drafted position has its head
