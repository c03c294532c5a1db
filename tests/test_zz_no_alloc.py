"""ee_exit_head_static: the entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: inside a serving process that gave all
device memory to its own pool at start-up, inside a plug-in whose host owns the allocator, or in a
latency-critical loop where an allocation (which stalls the device) is not acceptable.  For them the
library carries its scratch in a fixed device array.  This test drives that entry point through the C ABI
and checks it against the ordinary ee_exit_head on the same inputs, twice in a row with different inputs,
so that anything left behind in the shared array by the first call would show up in the second; against the
CPU oracle as well; that the call leaves the device's free memory and torch's allocator untouched; and that a
wait which gives up inside the array can be read and recovered from, since the caller has no pointer to it.

Collected last on purpose: a failure here cannot hide another test's result under `pytest -x`.
"""
import numpy as np
import pytest
import torch

import gen
from _util import ENTROPY_TOL, MAXPROB_TOL, assert_head_matches, dev, dev_bf16, head_to_dev, oracle_head

pytestmark = pytest.mark.gpu


def _both(ee, cfg, tau, out_static):
    hd = head_to_dev(cfg["heads"][0])
    h = dev_bf16(cfg["h"])
    tau_arg = dev(tau) if isinstance(tau, np.ndarray) else tau
    ref = ee.ee_exit_head(h, hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], tau_arg)
    ee.ee_exit_head_static(h, hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], tau_arg, out=out_static)
    torch.cuda.synchronize()
    return ref


def _assert_same(got, ref, label):
    assert torch.equal(got["argmax"], ref["argmax"]), label
    assert torch.equal(got["exit_mask"], ref["exit_mask"]), label
    assert (got["entropy"] - ref["entropy"]).abs().max().item() <= ENTROPY_TOL, label
    assert (got["maxprob"] - ref["maxprob"]).abs().max().item() <= MAXPROB_TOL, label
    assert torch.isfinite(got["entropy"]).all(), label


def test_static_scratch_entry_point_matches_the_workspace_one_on_two_calls_in_a_row():
    import paper_2407_21082_b200 as ee
    first = gen.make_config("c1", seed=21, planted=True, M=32, V=50304)
    second = gen.make_config("c0", seed=22, planted=True, M=5, V=7001, d=520)
    out1, out2 = ee.new_outputs(32), ee.new_outputs(5)
    ref1 = _both(ee, first, 1.0, out1)
    _assert_same(out1, ref1, "first call (32 rows, d=1024, V=50304)")
    assert 0 < int(ref1["exit_mask"].sum()) < 32          # both outcomes occur
    tau2 = np.linspace(0.25, 3.0, 5).astype(np.float32)
    ref2 = _both(ee, second, tau2, out2)
    _assert_same(out2, ref2, "second call (5 rows, d=520, V=7001, per-row thresholds)")
    # and the first inputs again: nothing of the second call lingers
    ref3 = _both(ee, first, 1.0, out1)
    _assert_same(out1, ref3, "third call")
    assert torch.equal(ref3["argmax"], ref1["argmax"]) and torch.equal(ref3["entropy"], ref1["entropy"])


def test_static_scratch_entry_point_matches_the_oracle_and_allocates_nothing():
    import paper_2407_21082_b200 as ee
    cfg = gen.make_config("c1", seed=23, planted=True, M=32, V=50304)
    hd = head_to_dev(cfg["heads"][0])
    h = dev_bf16(cfg["h"])
    out = ee.new_outputs(32)
    ee.ee_exit_head_static(h, hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], 1.0, out=out)      # set-up call
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    torch_before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
    for _ in range(3):
        ee.ee_exit_head_static(h, hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], 1.0, out=out)
    assert ee.ee_exit_head_static_query_error() == 0
    free_after, _ = torch.cuda.mem_get_info()
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == torch_before
    assert free_after == free_before                       # nothing was taken from the device either
    ref = oracle_head(cfg["h"], cfg["heads"][0], 1.0)
    assert_head_matches(out, ref, label="static entry point against the oracle (32 rows, d=1024, V=50304)")


def test_a_wait_that_gives_up_in_the_built_in_array_is_reported_and_recovered_from():
    import paper_2407_21082_b200 as ee
    cfg = gen.make_config("c0", seed=24, planted=True, M=8, V=3001, d=512)
    hd = head_to_dev(cfg["heads"][0])
    h = dev_bf16(cfg["h"])
    out = ee.new_outputs(8)
    ee.ee_exit_head_static(h, hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], 1.0, out=out)
    assert ee.ee_exit_head_static_query_error() == 0
    ee.ee_exit_head_static_selftest_timeout()              # a bounded wait that nothing ends: no fault, an error word
    assert ee.ee_exit_head_static_query_error() == 7       # EE_ERR_TIMEOUT, and the control block is zeroed again
    assert ee.ee_exit_head_static_query_error() == 0       # reading cleared it
    ee.ee_exit_head_static(h, hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], 1.0, out=out)
    assert ee.ee_exit_head_static_query_error() == 0
    assert_head_matches(out, oracle_head(cfg["h"], cfg["heads"][0], 1.0), label="static call after the recovery")


def test_static_wrapper_checks_its_arguments_on_the_host():
    import paper_2407_21082_b200 as ee
    cfg = gen.make_config("c0", seed=3, M=4, V=300, d=64)
    hd = head_to_dev(cfg["heads"][0])
    h = dev_bf16(cfg["h"])
    out = ee.new_outputs(4)
    with pytest.raises(ValueError):                        # W of another width would be read out of bounds
        ee.ee_exit_head_static(h, hd["gamma"], hd["beta"], 1e-5, hd["W"][:, :32].contiguous(), 1.0, out=out)
    with pytest.raises(ValueError):                        # strided W
        ee.ee_exit_head_static(h, hd["gamma"], hd["beta"], 1e-5, hd["W"][::2], 1.0, out=out)
    with pytest.raises(ValueError):                        # gamma too short
        ee.ee_exit_head_static(h, hd["gamma"][:32], hd["beta"], 1e-5, hd["W"], 1.0, out=out)
    with pytest.raises(ValueError):                        # outputs too short
        ee.ee_exit_head_static(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, out=ee.new_outputs(2))
    with pytest.raises(ValueError):                        # per-row tau of the wrong length
        ee.ee_exit_head(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], torch.ones(3, device="cuda"))


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    import paper_2407_21082_b200 as ee
    cfg = gen.make_config("c0", seed=3, M=ee.EE_STATIC_MAX_ROWS + 1, V=300, d=64)
    hd = head_to_dev(cfg["heads"][0])
    with pytest.raises(ee.EExitError) as e:
        ee.ee_exit_head_static(dev_bf16(cfg["h"]), hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0,
                               out=ee.new_outputs(ee.EE_STATIC_MAX_ROWS + 1))
    assert e.value.code == 2                               # EE_ERR_SHAPE: more rows than the built-in scratch serves
    wide = gen.make_config("c0", seed=3, M=32, V=300, d=4096)
    hd = head_to_dev(wide["heads"][0])
    with pytest.raises(ee.EExitError) as e:
        ee.ee_exit_head_static(dev_bf16(wide["h"]), hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, out=ee.new_outputs(32))
    assert e.value.code == 2                               # 32 rows of width 4096 do not fit one launch
