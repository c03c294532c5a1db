"""Pins of the KL-to-teacher oracle (paper section 3.3, "Losses")."""
import math

import numpy as np

import gen
import oracle


def test_closed_forms_and_term_by_term_definition():
    # two classes: p = (a, 1-a), q = (b, 1-b)
    a, b = 0.8, 0.3
    z_p = np.log(np.array([[a, 1 - a]]))
    z_q = np.log(np.array([[b, 1 - b]])) + 5.0                       # a shift of the logits changes nothing
    want = a * math.log(a / b) + (1 - a) * math.log((1 - a) / (1 - b))
    assert abs(oracle.kl_from_logits(z_p, z_q)[0] - want) < 1e-14
    assert abs(oracle.kl_from_logits(z_p - 3.0, z_q)[0] - want) < 1e-14
    # uniform head against a one-raised-logit teacher over V classes
    V, c = 1000, 2.5
    zq = np.zeros((1, V)); zq[0, 3] = c
    want = math.log(math.exp(c) + V - 1) - math.log(V) - c / V       # sum 1/V (log 1/V - log q_v)
    assert abs(oracle.kl_from_logits(np.zeros((1, V)), zq)[0] - want) < 1e-13
    # the definition, term by term, with compensated summation
    rng = np.random.default_rng(1)
    zp, zq = rng.normal(0, 2, (6, 40)), rng.normal(0, 2, (6, 40))
    got = oracle.kl_from_logits(zp, zq)
    for i in range(6):
        p = np.exp(zp[i] - zp[i].max()); p /= math.fsum(p)
        q = np.exp(zq[i] - zq[i].max()); q /= math.fsum(q)
        assert abs(got[i] - math.fsum(pi * math.log(pi / qi) for pi, qi in zip(p, q))) < 1e-13
    assert (got > 0).all() and np.all(oracle.kl_from_logits(zp, zp) == 0.0)


def test_whole_path_is_zero_for_identical_models_and_positive_otherwise():
    cfg = gen.make_config("c1", seed=2, planted=True, M=10, d=64, V=300, heads=2)
    same = oracle.kl_to_teacher(cfg["h"], cfg["heads"][0], cfg["h"], cfg["heads"][0])
    assert np.all(same["kl"] == 0.0) and same["loss"] == 0.0
    diff = oracle.kl_to_teacher(cfg["h"], cfg["heads"][0], cfg["h"], cfg["heads"][1])
    assert (diff["kl"] > 0).all() and abs(diff["loss"] - diff["kl"].mean()) < 1e-15
    # against the pieces oracle.exit_head already pins: KL = -H_head + logZ_teacher - E_head[z_teacher]
    out_h = oracle.exit_head(cfg["h"], cfg["heads"][0]["gamma"], cfg["heads"][0]["beta"], 1e-5, cfg["heads"][0]["W"], 1.0)
    out_t = oracle.exit_head(cfg["h"], cfg["heads"][1]["gamma"], cfg["heads"][1]["beta"], 1e-5, cfg["heads"][1]["W"], 1.0)
    yh = oracle.layer_norm(cfg["h"], cfg["heads"][0]["gamma"], cfg["heads"][0]["beta"], 1e-5)
    yt = oracle.layer_norm(cfg["h"], cfg["heads"][1]["gamma"], cfg["heads"][1]["beta"], 1e-5)
    zh, zt = yh @ oracle.bf16_decode(cfg["heads"][0]["W"]).T, yt @ oracle.bf16_decode(cfg["heads"][1]["W"]).T
    ph = np.exp(zh - out_h["logZ"][:, None])
    assert np.abs(diff["kl"] - (-out_h["entropy"] + out_t["logZ"] - (ph * zt).sum(axis=1))).max() < 1e-11


def test_cross_entropy_closed_forms():
    V = 500
    assert abs(oracle.ce_from_logits(np.zeros((1, V)), np.array([7]))[0] - math.log(V)) < 1e-14          # uniform
    z = np.zeros((1, V)); z[0, 3] = 4.0
    assert abs(oracle.ce_from_logits(z, np.array([3]))[0] - (math.log(math.exp(4.0) + V - 1) - 4.0)) < 1e-13
    assert abs(oracle.ce_from_logits(z, np.array([9]))[0] - math.log(math.exp(4.0) + V - 1)) < 1e-13
    rng = np.random.default_rng(2)
    z = rng.normal(0, 3, (5, 30)); lab = rng.integers(0, 30, 5)
    got = oracle.ce_from_logits(z, lab)
    for i in range(5):
        p = np.exp(z[i] - z[i].max()); p /= math.fsum(p)
        assert abs(got[i] + math.log(p[lab[i]])) < 1e-13
    assert np.allclose(oracle.ce_from_logits(z + 11.0, lab), got, atol=1e-13)                            # shift invariance
    cfg = gen.make_config("c1", seed=2, planted=True, M=6, d=64, V=300, heads=2)
    out = oracle.kl_to_teacher(cfg["h"], cfg["heads"][0], cfg["h"], cfg["heads"][1], labels=np.arange(6) * 7)
    full = oracle.exit_head(cfg["h"], cfg["heads"][0]["gamma"], cfg["heads"][0]["beta"], 1e-5, cfg["heads"][0]["W"], 1.0)
    own = oracle.kl_to_teacher(cfg["h"], cfg["heads"][0], cfg["h"], cfg["heads"][1], labels=full["argmax"])
    assert np.abs(own["ce"] + np.log(full["maxprob"])).max() < 1e-12      # CE at the head's own prediction = -log p_max
    assert abs(out["ce_loss"] - out["ce"].mean()) < 1e-15 and (out["ce"] >= own["ce"] - 1e-12).all()
