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
