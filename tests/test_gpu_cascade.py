"""ee_cascade against the oracle: which head answers each row, its token and entropy, rows per head."""
import numpy as np
import pytest
import torch

import gen
import oracle
from _util import ENTROPY_TOL, GAP_MIN, MARGIN_MIN, dev_bf16, head_to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ee():
    import paper_2407_21082_b200 as ee
    return ee


def _case(seed, M, d, V, K):
    cfg = gen.make_config("c1", seed=seed, planted=True, M=M, d=d, V=V, heads=K)
    rng = np.random.default_rng(seed)
    h_list = []
    for k in range(K):                                   # another layer's hidden states for every head
        x = gen.f32_from_bf16_bits(cfg["h"]) + rng.normal(0, 0.3 * k, size=cfg["h"].shape).astype(np.float32)
        h_list.append(gen.bf16_bits_from_f32(x))
    return cfg, h_list


def _fragile_rows(ref, taus):
    """Rows whose path through the cascade hangs on a decision inside the tolerance band (|H - tau| < 1e-3 at a
    head they reached) or whose reported token has a near-tied runner-up: excluded from the exact comparison."""
    M = ref["exit_head"].size
    margin_bad, token_bad = np.zeros(M, bool), np.zeros(M, bool)
    for k, ph in enumerate(ref["per_head"]):
        keep = oracle.decisive_rows(ph, GAP_MIN, MARGIN_MIN)
        margin_bad[ph["rows"][~keep["exit_mask"]]] = True
        answered = ph["exit_mask"] != 0
        token_bad[ph["rows"][answered & ~keep["argmax"]]] = True
    return margin_bad, token_bad


@pytest.mark.parametrize("M,d,V,K", [(24, 64, 300, 3), (1, 64, 129, 2), (100, 256, 1000, 4), (600, 128, 700, 3), (1100, 64, 520, 2),
                                     (128, 64, 700, 6), (37, 128, 515, 9), (129, 64, 300, 5), (512, 64, 520, 5), (513, 64, 520, 3)])
# up to 512 rows: every head on every row, in groups of four; above: head by head on the open rows
def test_cascade_matches_oracle(ee, M, d, V, K):
    cfg, h_list = _case(3 + M, M, d, V, K)
    taus = [0.6 + 0.7 * k for k in range(K)]
    hds = [head_to_dev(cfg["heads"][k]) for k in range(K)]
    heads = [dict(h=dev_bf16(h_list[k]), gamma=hds[k]["gamma"], beta=hds[k]["beta"], W=hds[k]["W"], tau=taus[k]) for k in range(K)]
    ref = oracle.cascade(h_list, cfg["heads"], taus)
    margin_bad, token_bad = _fragile_rows(ref, taus)
    for _ in range(2):                                   # the workspace and the counters are reusable
        out = ee.ee_cascade(heads, 1e-5)
        torch.cuda.synchronize()
        got = {k: v.cpu().numpy() for k, v in out.items()}
        ok = ~margin_bad
        assert np.array_equal(got["exit_head"][ok], ref["exit_head"][ok])
        tok_ok = ok & ~token_bad
        assert np.array_equal(got["token"][tok_ok], ref["token"][tok_ok])
        answered = ok & (ref["exit_head"] < K)
        assert np.abs(got["entropy"][answered] - ref["entropy"][answered]).max(initial=0.0) <= ENTROPY_TOL
        assert np.isnan(got["entropy"][ok & (ref["exit_head"] == K)]).all()
        if not margin_bad.any():
            assert got["rows_in"].tolist() == ref["rows_in"].tolist()
        assert got["rows_in"][0] == M and np.all(np.diff(got["rows_in"]) <= 0)
    assert (ref["exit_head"] == K).sum() + sum((ref["exit_head"] == k).sum() for k in range(K)) == M


def test_cascade_extreme_thresholds_and_errors(ee):
    cfg, h_list = _case(9, 40, 64, 257, 3)
    hds = [head_to_dev(cfg["heads"][k]) for k in range(3)]

    def heads(taus):
        return [dict(h=dev_bf16(h_list[k]), gamma=hds[k]["gamma"], beta=hds[k]["beta"], W=hds[k]["W"], tau=taus[k]) for k in range(3)]

    out = ee.ee_cascade(heads([-1.0, -1.0, -1.0]), 1e-5)           # nobody answers
    assert (out["exit_head"] == 3).all() and (out["token"] == -1).all() and out["rows_in"].tolist() == [40, 40, 40]
    assert torch.isnan(out["entropy"]).all()
    out = ee.ee_cascade(heads([1e9, 1e9, 1e9]), 1e-5)              # the first head answers everything
    assert (out["exit_head"] == 0).all() and out["rows_in"].tolist() == [40, 0, 0]
    out = ee.ee_cascade(heads([-1.0, -1.0, float("inf")]), 1e-5)   # a last head that plays the full model
    ref = oracle.exit_head(h_list[2], cfg["heads"][2]["gamma"], cfg["heads"][2]["beta"], 1e-5, cfg["heads"][2]["W"], 1e9)
    keep = oracle.decisive_rows(ref, GAP_MIN, MARGIN_MIN)["argmax"]
    assert (out["exit_head"] == 2).all() and np.array_equal(out["token"].cpu().numpy()[keep], ref["argmax"][keep])
    with pytest.raises(ee.EExitError) as e:
        ee.ee_cascade(heads([1.0, 1.0, 1.0]), 1e-5, workspace=torch.zeros(512, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 4
