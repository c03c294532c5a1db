"""ee_head_kl against the oracle: per-token KL of the head's distribution from the teacher's, and their mean."""
import numpy as np
import pytest
import torch

import gen
import oracle
from _util import dev_bf16, head_to_dev

pytestmark = pytest.mark.gpu
KL_TOL = 2e-3          # absolute, nats: the tolerance of the entropy it contains


@pytest.fixture(scope="module")
def ee():
    import paper_2407_21082_b200 as ee
    return ee


def _run(ee, cfg, h_head, h_teacher, labels=None):
    hd, tc = head_to_dev(cfg["heads"][0]), head_to_dev(cfg["heads"][1])
    out = ee.ee_head_kl(dict(h=dev_bf16(h_head), gamma=hd["gamma"], beta=hd["beta"], W=hd["W"]),
                        dict(h=dev_bf16(h_teacher), gamma=tc["gamma"], beta=tc["beta"], W=tc["W"]), 1e-5,
                        labels=None if labels is None else torch.from_numpy(labels).cuda())
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("M,d,V", [(1, 64, 1), (5, 72, 257), (64, 128, 400), (129, 320, 515), (300, 64, 2049), (16, 1024, 50304),
                                   (129, 320, 515), (256, 136, 1000), (700, 64, 2049), (1500, 72, 300)])   # even numbers of row tiles: CTA pairs
def test_kl_matches_oracle(ee, M, d, V):
    # Planted rows of W are about fifty times the workloads' weight scale at small d, where one element of the
    # LayerNorm output on the wrong side of a bf16 midpoint would move the cross-entropy by several 1e-3.
    for planted in (False, True):
        cfg = gen.make_config("c1", seed=31, planted=planted, M=M, d=d, V=V, heads=2)
        rng = np.random.default_rng(M)
        h_t = gen.bf16_bits_from_f32(gen.f32_from_bf16_bits(cfg["h"]) + rng.normal(0, 0.5, cfg["h"].shape).astype(np.float32))
        labels = rng.integers(0, V, size=M).astype(np.int32)
        labels[0] = V - 1                                               # the last column of the ragged last tile
        ref = oracle.kl_to_teacher(cfg["h"], cfg["heads"][0], h_t, cfg["heads"][1], labels=labels)
        out = _run(ee, cfg, cfg["h"], h_t, labels)
        again = _run(ee, cfg, cfg["h"], h_t, labels)
        ce = out["ce"].cpu().numpy().astype(np.float64)
        assert np.abs(ce - ref["ce"]).max() <= KL_TOL, (planted, np.abs(ce - ref["ce"]).max())
        assert abs(float(out["loss"][1].item()) - ref["ce_loss"]) <= KL_TOL
        assert torch.equal(out["ce"], again["ce"])
        no_labels = _run(ee, cfg, cfg["h"], h_t)
        assert torch.equal(no_labels["kl"], out["kl"]) and "ce" not in no_labels
        kl = out["kl"].cpu().numpy().astype(np.float64)
        assert np.isfinite(kl).all()
        assert np.abs(kl - ref["kl"]).max() <= KL_TOL, (planted, np.abs(kl - ref["kl"]).max())
        assert abs(float(out["loss"][0].item()) - ref["loss"]) <= KL_TOL
        assert torch.equal(out["kl"], again["kl"]) and torch.equal(out["loss"], again["loss"])     # fixed reduction order
        assert (kl > -1e-4).all()


def test_kl_full_size_on_a_row_sample(ee):
    """The benchmark's training-sized call (c1 shape, M = 4096: CTA pairs on 256-row tiles, 256 columns wide): the
    oracle checks two rows of every 128-row tile plus the tiles' edges; properties that hold for every row."""
    M, d, V = 4096, 1024, 50304
    cfg = gen.make_config("c1", seed=0, planted=False, M=M, heads=2)
    rng = np.random.default_rng(0)
    h_t = gen.bf16_bits_from_f32(gen.f32_from_bf16_bits(cfg["h"]) + rng.normal(0, 0.5, cfg["h"].shape).astype(np.float32))
    labels = rng.integers(0, V, size=M).astype(np.int32)
    labels[:4] = [0, 255, 256, V - 1]                                   # tile edges of the vocabulary
    out = _run(ee, cfg, cfg["h"], h_t, labels)
    rows = np.unique(np.concatenate([[0, 1, 2, 3, 127, 128, 255, 256, 4095],
                                     [t * 128 + (37 * t + 64 * i) % 128 for t in range(32) for i in range(2)]]))
    ref = oracle.kl_to_teacher(cfg["h"][rows], cfg["heads"][0], h_t[rows], cfg["heads"][1], labels=labels[rows])
    kl = out["kl"].cpu().numpy().astype(np.float64)
    ce = out["ce"].cpu().numpy().astype(np.float64)
    assert np.abs(kl[rows] - ref["kl"]).max() <= KL_TOL
    assert np.abs(ce[rows] - ref["ce"]).max() <= KL_TOL
    assert len(set(rows // 128)) == 32
    assert np.isfinite(kl).all() and (kl > -1e-4).all()                 # a divergence
    assert np.isfinite(ce).all() and (ce > 0).all()                     # -log of a probability below one
    assert abs(float(out["loss"][0].item()) - kl.mean()) <= 1e-4 and abs(float(out["loss"][1].item()) - ce.mean()) <= 1e-4


def test_kl_of_a_model_from_itself_is_zero(ee):
    cfg = gen.make_config("c1", seed=3, planted=True, M=40, d=128, V=900, heads=2)
    cfg["heads"][1] = cfg["heads"][0]
    out = _run(ee, cfg, cfg["h"], cfg["h"])
    assert float(out["kl"].abs().max()) <= 1e-5 and abs(float(out["loss"][0].item())) <= 1e-5


def test_kl_argument_errors(ee):
    cfg = gen.make_config("c1", seed=3, planted=False, M=4, d=64, V=100, heads=2)
    hd = head_to_dev(cfg["heads"][0])
    h = dev_bf16(cfg["h"])
    with pytest.raises(ee.EExitError) as e:
        ee.ee_head_kl(dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"]), dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"]),
                      1e-5, workspace=torch.zeros(512, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 4
