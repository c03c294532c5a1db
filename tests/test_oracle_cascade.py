"""Pins of the cascade oracle (paper section 3.4.2)."""
import numpy as np

import gen
import oracle


def _case(seed, M=24, d=64, V=300, K=3):
    cfg = gen.make_config("c1", seed=seed, planted=True, M=M, d=d, V=V, heads=K)
    rng = np.random.default_rng(seed)
    # every head reads different hidden states (another layer of the model): perturb the batch per head
    h_list = []
    for k in range(K):
        x = gen.f32_from_bf16_bits(cfg["h"]) + rng.normal(0, 0.3 * k, size=cfg["h"].shape).astype(np.float32)
        h_list.append(gen.bf16_bits_from_f32(x))
    return cfg, h_list


def test_equals_independent_evaluation_of_every_head_on_every_row():
    for seed in range(4):
        cfg, h_list = _case(seed)
        taus = [0.8, 1.5, 3.0]
        got = oracle.cascade(h_list, cfg["heads"], taus)
        full = [oracle.exit_head(h_list[k], hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], taus[k])
                for k, hd in enumerate(cfg["heads"])]
        M, K = h_list[0].shape[0], len(taus)
        for i in range(M):
            first = next((k for k in range(K) if full[k]["exit_mask"][i]), K)
            assert got["exit_head"][i] == first
            if first < K:
                assert got["token"][i] == full[first]["argmax"][i]
                assert got["entropy"][i] == full[first]["entropy"][i]
            else:
                assert got["token"][i] == -1 and np.isnan(got["entropy"][i])
        answered = np.array([(got["exit_head"] == k).sum() for k in range(K)])
        assert got["rows_in"][0] == M
        assert np.array_equal(got["rows_in"][1:], M - np.cumsum(answered)[:-1])
        assert answered.sum() + (got["exit_head"] == K).sum() == M
        assert 0 < answered[0] < M                                   # the case exercises both outcomes


def test_thresholds_at_the_extremes():
    cfg, h_list = _case(7, M=10)
    K = 3
    never = oracle.cascade(h_list, cfg["heads"], [-1.0] * K)          # H < -1 never holds
    assert (never["exit_head"] == K).all() and (never["token"] == -1).all() and (never["rows_in"] == 10).all()
    always = oracle.cascade(h_list, cfg["heads"], [1e9] * K)          # the first head answers everything
    assert (always["exit_head"] == 0).all() and always["rows_in"].tolist() == [10, 0, 0]
    last = oracle.cascade(h_list, cfg["heads"], [-1.0, -1.0, 1e9])    # a final head that always answers
    assert (last["exit_head"] == 2).all() and last["rows_in"].tolist() == [10, 10, 10]
    ref = oracle.exit_head(h_list[2], cfg["heads"][2]["gamma"], cfg["heads"][2]["beta"], 1e-5, cfg["heads"][2]["W"], 1e9)
    assert np.array_equal(last["token"], ref["argmax"])
