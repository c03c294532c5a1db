"""ee_compact and dssd_accept against the oracle (bit-exact), and the c2 / c3 pipelines end to end."""
import os

import numpy as np
import pytest
import torch

import gen
import oracle
from _util import assert_head_matches, dev, dev_bf16, head_to_dev, oracle_head

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ee():
    import paper_2407_21082_b200 as ee
    return ee


def _check_compact(ee, mask, h_bits):
    M = mask.size
    out = ee.ee_compact(dev(mask), dev_bf16(h_bits) if h_bits is not None else None)
    ref = oracle.compact(mask, h_bits)
    n = int(out["kept_count"].item())
    assert n == ref["kept_count"]
    assert np.array_equal(out["kept_idx"].cpu().numpy()[:n], ref["kept_idx"])
    if h_bits is not None:
        got = out["h_out"].view(torch.int16).cpu().numpy().view(np.uint16)[:n]
        assert np.array_equal(got, ref["h_out"])


@pytest.mark.parametrize("M,d", [(1, 8), (31, 64), (32, 64), (33, 72), (256, 2048), (1000, 40), (5000, 16), (16384, 64), (100000, 8)])
def test_compact_random_masks(ee, M, d):
    rng = np.random.default_rng(M)
    h = rng.integers(0, 65536, size=(M, d)).astype(np.uint16)
    for p in (0.0, 0.3, 0.97, 1.0):
        mask = (rng.random(M) < p).astype(np.uint8) * rng.integers(1, 256, size=M).astype(np.uint8)
        _check_compact(ee, mask, h)
    _check_compact(ee, (np.arange(M) % 2).astype(np.uint8), None)
    if M >= 64:                        # a mask that does not start on a 16-byte boundary (the survivors are counted 16 bytes at a time)
        for off in (1, 7, 15):
            big = dev(np.concatenate([np.zeros(off, np.uint8), (rng.random(M - off) < 0.5).astype(np.uint8)]))
            sub = big[off:]
            out = ee.ee_compact(sub)
            torch.cuda.synchronize()
            ref = oracle.compact(sub.cpu().numpy())
            n = int(out["kept_count"].item())
            assert n == ref["kept_count"] and np.array_equal(out["kept_idx"].cpu().numpy()[:n], ref["kept_idx"])


def test_compact_hand_masks_and_empty(ee):
    for mask in ([0], [1], [0, 0, 0, 0], [1, 1, 1, 1], [1, 0, 1, 0, 1, 0, 1], [0] + [1] * 40, [1] * 40 + [0]):
        mask = np.array(mask, np.uint8)
        h = (np.arange(mask.size * 8).reshape(mask.size, 8) % 65536).astype(np.uint16)
        _check_compact(ee, mask, h)
    out = ee.ee_compact(torch.empty(0, dtype=torch.uint8, device="cuda"))
    assert int(out["kept_count"].item()) == 0


def test_compact_leaves_rows_beyond_count_untouched_and_supports_strides(ee):
    M, d = 40, 16
    rng = np.random.default_rng(3)
    wide = torch.from_numpy(rng.integers(0, 30000, size=(M, 32)).astype(np.int16)).cuda().view(torch.bfloat16)
    mask = (rng.random(M) < 0.5).astype(np.uint8)
    out = dict(kept_idx=torch.full((M,), -7, dtype=torch.int32, device="cuda"),
               kept_count=torch.zeros(1, dtype=torch.int32, device="cuda"),
               h_out=torch.full((M, d), 3.0, dtype=torch.bfloat16, device="cuda"))
    ee.ee_compact(dev(mask), wide[:, :d], out=out)
    n = int(out["kept_count"].item())
    ref = oracle.compact(mask, wide[:, :d].contiguous().view(torch.int16).cpu().numpy().view(np.uint16))
    assert n == ref["kept_count"] and torch.all(out["kept_idx"][n:] == -7) and torch.all(out["h_out"][n:] == 3.0)
    assert np.array_equal(out["h_out"][:n].view(torch.int16).cpu().numpy().view(np.uint16), ref["h_out"])


def _golden_cases():
    path = os.path.join(os.path.dirname(__file__), "golden", "dssd_accept_cases.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, d, c, v, want = [f.strip() for f in line.split(";")]
        yield name, [int(x) for x in d.split()], [int(x) for x in c.split()], [int(x) for x in v.split()], \
            [int(x) for x in want.split()]


def test_accept_hand_worked_cases(ee):
    for name, d, c, v, want in _golden_cases():
        out = ee.dssd_accept(dev(np.array([d], np.int32)), dev(np.array([c], np.uint8)), dev(np.array([v], np.int32)))
        got = [int(out[k].item()) for k in ("draft_len", "accept_len", "next_tok")]
        assert got == want, name


@pytest.mark.parametrize("S,k,kv", [(1, 1, 1), (32, 8, 8), (33, 8, 9), (7, 32, 32), (5, 33, 40), (64, 100, 101), (1000, 5, 5)])
def test_accept_random_against_oracle(ee, S, k, kv):
    c = gen.random_token_case(S + k, S, k, kv)
    ref = oracle.dssd_accept(c["draft_tok"], c["draft_exit_mask"], c["verify_tok"])
    out = ee.dssd_accept(dev(c["draft_tok"]), dev(c["draft_exit_mask"]), dev(c["verify_tok"]))
    for key in ("draft_len", "accept_len", "next_tok"):
        assert np.array_equal(out[key].cpu().numpy(), ref[key]), key
    ref = oracle.dssd_accept(c["draft_tok"], None, c["verify_tok"])
    out = ee.dssd_accept(dev(c["draft_tok"]), None, dev(c["verify_tok"]))
    for key in ("draft_len", "accept_len", "next_tok"):
        assert np.array_equal(out[key].cpu().numpy(), ref[key]), key


def test_c2_pipeline_exit_then_compact(ee):
    cfg = gen.make_config("c2", seed=0, planted=True)
    hd = head_to_dev(cfg["heads"][0])
    h = dev_bf16(cfg["h"])
    out = ee.ee_exit_head(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], dev(cfg["tau_per_row"]))
    comp = ee.ee_compact(out["exit_mask"], h)
    ref = oracle_head(cfg["h"], cfg["heads"][0], cfg["tau_per_row"])
    info = assert_head_matches(out, ref, label="c2")
    assert 20 < ref["exit_mask"].sum() < 236
    # compaction is exact with respect to the mask it was given ...
    mask = out["exit_mask"].cpu().numpy()
    cref = oracle.compact(mask, cfg["h"])
    n = int(comp["kept_count"].item())
    assert n == cref["kept_count"] and np.array_equal(comp["kept_idx"].cpu().numpy()[:n], cref["kept_idx"])
    assert np.array_equal(comp["h_out"][:n].view(torch.int16).cpu().numpy().view(np.uint16), cref["h_out"])
    # ... and equals the oracle's own pipeline when no row sits within 1e-3 of its threshold
    if info["excluded"]["exit_mask"].size == 0:
        assert np.array_equal(cref["kept_idx"], oracle.compact(ref["exit_mask"])["kept_idx"])


@pytest.mark.parametrize("planted", [True, False])
def test_c3_pipeline_draft_verify_accept(ee, planted):
    cfg = gen.make_config("c3", seed=0, planted=planted)
    S, k = cfg["S"], cfg["k"]
    draft_hd, final_hd = head_to_dev(cfg["heads"][0]), head_to_dev(cfg["heads"][1])
    d_out = ee.ee_exit_head(dev_bf16(cfg["h_draft"]), draft_hd["gamma"], draft_hd["beta"], 1e-5, draft_hd["W"], cfg["tau"])
    v_out = ee.ee_exit_head(dev_bf16(cfg["h_verify"]), final_hd["gamma"], final_hd["beta"], 1e-5, final_hd["W"], cfg["tau"])
    acc = ee.dssd_accept(d_out["argmax"].view(S, k), d_out["exit_mask"].view(S, k), v_out["argmax"].view(S, k))
    d_ref = oracle_head(cfg["h_draft"], cfg["heads"][0], cfg["tau"])
    v_ref = oracle_head(cfg["h_verify"], cfg["heads"][1], cfg["tau"])
    di = assert_head_matches(d_out, d_ref, label="c3 draft head")
    vi = assert_head_matches(v_out, v_ref, label="c3 final head")
    a_ref = oracle.dssd_accept(d_ref["argmax"].reshape(S, k), d_ref["exit_mask"].reshape(S, k), v_ref["argmax"].reshape(S, k))
    # sequences containing a listed near-tie row are excluded from the end-to-end comparison
    undecided = np.zeros(S * k, bool)
    for info in (di, vi):
        undecided[info["excluded"]["argmax"]] = True
        undecided[info["excluded"]["exit_mask"]] = True
    ok = ~undecided.reshape(S, k).any(axis=1)
    for key in ("draft_len", "accept_len", "next_tok"):
        assert np.array_equal(acc[key].cpu().numpy()[ok], a_ref[key][ok]), key
    assert ok.sum() >= S - 4
    if planted:
        assert a_ref["draft_len"].max() > 0          # some sequences draft at least one token
    else:
        assert a_ref["draft_len"].max() == 0         # the literal inputs are never confident


@pytest.mark.parametrize("M,d,S,k,kv", [(64, 1024, 8, 8, 8), (1, 8, 1, 1, 1), (33, 72, 70, 5, 9), (1000, 40, 3, 40, 40),
                                        (40, 16, 0, 4, 4), (0, 16, 9, 4, 6)])
def test_compact_accept_one_launch_matches_oracle(ee, M, d, S, k, kv):
    """The fused call gives bit for bit what the oracle gives for the two operations, twice in a row."""
    rng = np.random.default_rng(1000 * M + S)
    h = rng.integers(0, 65536, size=(M, d)).astype(np.uint16)
    mask = (rng.random(M) < 0.4).astype(np.uint8) * rng.integers(1, 256, size=M).astype(np.uint8)
    case = gen.random_token_case(seed=M + S, S=max(S, 1), k=k, kv=kv)
    draft, conf, verify = (case[n][:S] for n in ("draft_tok", "draft_exit_mask", "verify_tok"))
    ref_c = oracle.compact(mask, h)
    ref_a = oracle.dssd_accept(draft, conf, verify) if S else None
    h_dev = dev_bf16(h) if M else torch.empty((0, d), dtype=torch.bfloat16, device="cuda")
    for _ in range(2):
        out = ee.ee_compact_accept(dev(mask), h_dev, dev(draft.reshape(S, k)), dev(conf.reshape(S, k)),
                                   dev(verify.reshape(S, kv)))
        n = int(out["compact"]["kept_count"].item())
        assert n == ref_c["kept_count"]
        assert np.array_equal(out["compact"]["kept_idx"].cpu().numpy()[:n], ref_c["kept_idx"])
        got = out["compact"]["h_out"].view(torch.int16).cpu().numpy().view(np.uint16)[:n]
        assert np.array_equal(got, ref_c["h_out"])
        if S:
            for name in ("draft_len", "accept_len", "next_tok"):
                assert np.array_equal(out["accept"][name].cpu().numpy(), ref_a[name]), name
