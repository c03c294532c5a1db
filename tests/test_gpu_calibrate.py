"""ee_calibrate against the oracle: bit-exact threshold and counts (the one floating-point comparison is made in
fp64 on both sides)."""
import numpy as np
import pytest
import torch

import gen
import oracle
from _util import dev, dev_bf16, head_to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ee():
    import paper_2407_21082_b200 as ee
    return ee


def _check(ee, H, a_head, a_final, eps):
    out = ee.ee_calibrate(dev(H.astype(np.float32)), dev(a_head.astype(np.int32)), dev(a_final.astype(np.int32)), eps)
    torch.cuda.synchronize()
    ref = oracle.calibrate_threshold(H.astype(np.float32), oracle.correctness(a_head, a_final), eps)
    tau = float(out["tau"].item())
    counts = out["counts"].cpu().numpy().tolist()
    assert counts == [ref["n_exit"], ref["n_correct"], ref["j_hat"]], (eps, counts, ref)
    assert tau == np.float32(ref["tau"]) or (np.isinf(tau) and np.isinf(ref["tau"]) and tau < 0), (eps, tau, ref)


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 511, 512, 513, 4095, 4096, 4097, 10000, 70001])
def test_random_sets_with_and_without_ties(ee, n):
    rng = np.random.default_rng(n)
    for ties in (False, True):
        H = rng.gamma(2.0, 1.5, size=n).astype(np.float32)
        if ties:
            H = np.round(H, 1)
        p = np.exp(-H / 3.0)
        a_final = rng.integers(0, 50304, size=n).astype(np.int32)
        a_head = np.where(rng.random(n) < p, a_final, (a_final + 1) % 50304).astype(np.int32)
        for eps in (0.0, 0.3, 0.6, 0.8, 0.95, 1.0):
            _check(ee, H, a_head, a_final, eps)


def test_hand_cases_special_values_and_empty(ee):
    H = -np.array([0.1, 0.2, 0.3, 0.4], np.float32)                 # negative entropies sort below positive ones
    t1 = np.array([1, 2, 3, 4], np.int32)
    _check(ee, H, np.array([0, 2, 3, 4], np.int32), t1, 0.75)
    _check(ee, H, np.array([0, 2, 3, 4], np.int32), t1, 0.76)
    _check(ee, -np.array([0.1, 0.2, 0.3], np.float32), np.array([1, 1, 0], np.int32), np.array([1, 1, 9], np.int32), 1.0)
    H = np.array([0.0, -0.0, np.inf, 1e-45, 3.0, -1e-45, 2.0], np.float32)      # zeros of both signs, denormals, inf
    for eps in (0.0, 0.5, 1.0):
        _check(ee, H, np.array([1, 0, 1, 1, 0, 1, 1], np.int32), np.ones(7, np.int32), eps)
    _check(ee, np.array([-0.0, 0.0], np.float32), np.array([1, 0], np.int32), np.array([1, 1], np.int32), 1.0)   # one group
    _check(ee, np.array([0.0, -0.0, 1.0], np.float32), np.array([0, 1, 1], np.int32), np.array([1, 1, 1], np.int32), 0.5)
    H = np.full(5000, 1.25, np.float32)                              # one big group
    a = np.arange(5000, dtype=np.int32)
    _check(ee, H, a, np.where(a % 4 == 0, -1, a).astype(np.int32), 0.75)
    _check(ee, H, a, np.where(a % 4 == 0, -1, a).astype(np.int32), 0.76)
    out = ee.ee_calibrate(torch.empty(0, dtype=torch.float32, device="cuda"), torch.empty(0, dtype=torch.int32, device="cuda"),
                          torch.empty(0, dtype=torch.int32, device="cuda"), 0.5)
    assert out["counts"].cpu().tolist() == [0, 0, 0] and float(out["tau"].item()) == float("-inf")


def test_argument_errors(ee):
    H, a = torch.zeros(4, device="cuda"), torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(ee.EExitError) as e:
        ee.ee_calibrate(H, a, a, 1.5)
    assert e.value.code == 2
    with pytest.raises(ee.EExitError) as e:
        ee.ee_calibrate(H, a, a, 0.5, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 4


def test_calibration_from_the_heads_own_outputs(ee):
    """The whole calibration pass of section 3.4.1 on a planted workload: an exit head and the final head on
    the same tokens (ee_exit_head_multi), then the threshold; the guarantee holds on the calibration set."""
    cfg = gen.make_config("c1", seed=5, planted=True, M=2048, d=256, V=4096, heads=2)
    h = dev_bf16(cfg["h"])
    hds = [head_to_dev(cfg["heads"][k]) for k in range(2)]
    outs = ee.ee_exit_head_multi([dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=1.0) for hd in hds], 1e-5)
    for eps in (0.5, 0.9, 0.99):
        res = ee.ee_calibrate(outs[0]["entropy"], outs[0]["argmax"], outs[1]["argmax"], eps)
        torch.cuda.synchronize()
        H = outs[0]["entropy"].cpu().numpy()
        t = oracle.correctness(outs[0]["argmax"].cpu().numpy(), outs[1]["argmax"].cpu().numpy())
        ref = oracle.calibrate_threshold(H, t, eps)
        assert res["counts"].cpu().tolist() == [ref["n_exit"], ref["n_correct"], ref["j_hat"]]
        tau = float(res["tau"].item())
        assert tau == np.float32(ref["tau"])
        if ref["n_exit"]:
            inside = H <= tau
            assert t[inside].mean() >= eps
