"""The error path of the bounded device-side waits, driven without any fault: a wait that is made to run out
records its status, the host reads it, and the context, the workspace and the library stay usable."""
import numpy as np
import pytest
import torch

import gen
from _util import assert_head_matches, dev_bf16, head_to_dev, oracle_head

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_nothing_else_breaks():
    import paper_2407_21082_b200 as ee
    cfg = gen.make_config("c0", seed=4, planted=True, M=12, d=128, V=900)
    hd = head_to_dev(cfg["heads"][0])
    h = dev_bf16(cfg["h"])
    ws = ee.new_workspace(12, 128, 900)
    assert ee.ee_query_async_error(ws) == 0
    ee.ee_selftest_wait_timeout(ws)
    assert ee.ee_query_async_error(ws) == 7                   # EE_ERR_TIMEOUT, read after the kernel returned
    assert ee.ee_query_async_error(ws) == 0                   # reading clears it
    out = ee.ee_exit_head(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, workspace=ws)
    torch.cuda.synchronize()
    assert_head_matches(out, oracle_head(cfg["h"], cfg["heads"][0], 1.0), label="after the self-test")
    assert ee.ee_query_async_error(ws) == 0
    # an error word left unread does not stop later calls from running; it is still there to be read
    ee.ee_selftest_wait_timeout(ws)
    again = ee.ee_exit_head(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, workspace=ws)
    torch.cuda.synchronize()
    for k in out:
        assert torch.equal(out[k], again[k])
    assert ee.ee_query_async_error(ws) == 7
    with pytest.raises(ee.EExitError) as e:
        ee.ee_selftest_wait_timeout(torch.zeros(64, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 4


def test_read_stream_diagnostic_runs_clean_and_checks_its_arguments():
    import paper_2407_21082_b200 as ee
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for nbytes in (16384, 16384 * 148 + 5000, 64 << 20):      # one stage, a ragged split over the SMs, larger than the rings
        buf = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        ee.ee_selftest_read_stream(buf, ws)
        ee.ee_selftest_read_stream(buf, ws)
        assert ee.ee_query_async_error(ws) == 0
    with pytest.raises(ee.EExitError) as e:
        ee.ee_selftest_read_stream(torch.zeros(1000, dtype=torch.uint8, device="cuda"), ws)
    assert e.value.code == 2
    with pytest.raises(ee.EExitError) as e:
        ee.ee_selftest_read_stream(torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")[8:], ws)
    assert e.value.code == 3
