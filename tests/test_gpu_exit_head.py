"""Parity of ee_exit_head (both kernels) with the fp64 oracle, through the C ABI."""
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
    assert torch.cuda.is_available()
    return ee


def _run(ee, cfg, head_id, tau, path, h_key="h"):
    hd = head_to_dev(cfg["heads"][head_id])
    tau_arg = dev(tau) if isinstance(tau, np.ndarray) else tau
    out = ee.ee_exit_head(dev_bf16(cfg[h_key]), hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], tau_arg, path=path)
    torch.cuda.synchronize()
    return out


# Reduced shapes: several vocabulary tiles with a ragged last one, K tails (d % 64 != 0, d % 32 != 0),
# partial row tiles, degenerate V = 1, and row counts around the slab (32) and tile (128) sizes.
SMALL = [
    # name, M, d, V
    ("v1", 3, 64, 1), ("tiny", 1, 8, 5), ("ragged", 5, 72, 257), ("k_tail", 8, 520, 1000),
    ("two_ntiles", 16, 128, 300), ("slab_edge", 32, 256, 2049), ("slab_over", 33, 264, 1031),
    ("mtile_edge", 128, 64, 700), ("mtile_over", 129, 320, 515), ("wide_d", 4, 4096, 600),
    # vocabulary sizes around one tile, the smallest d, and row counts at the tensor-core path's switches:
    # 64 / 65 rows (64- vs 128-row MMAs), 512 / 513 (merge inside the GEMM kernel vs merge kernel),
    # 1024 / 1025 (runtime-width vs 256-wide variant)
    ("v2", 2, 8, 2), ("v127", 3, 64, 127), ("v128", 127, 64, 128), ("v129", 1, 64, 129),
    ("m64", 64, 128, 400), ("m65", 65, 128, 400), ("m512", 512, 64, 300), ("m513", 513, 64, 300),
    ("m1024", 1024, 64, 300), ("m1025", 1025, 64, 520),
    # an even number of 128-row tiles: two CTAs share each 256-row tile (runtime-width and 256-wide variants,
    # ragged last vocabulary tiles, row counts that are not multiples of 128)
    ("pair_m256", 256, 136, 700), ("pair_ragged", 200, 256, 3001), ("pair_m768", 768, 192, 2049),
    ("pair_m1280", 1280, 128, 1500), ("pair_m2000", 2000, 72, 260),
]


PATHS = {"stream": 1, "tcgen05": 2, "skinny": 3}


@pytest.mark.parametrize("path_name", ["stream", "tcgen05", "skinny"])
@pytest.mark.parametrize("name,M,d,V", SMALL + [("sk_n32", 17, 192, 3001), ("sk_n64", 64, 512, 2500), ("sk_n64b", 33, 1024, 1500)])
def test_small_shapes_match_oracle(ee, path_name, name, M, d, V):
    path = PATHS[path_name]
    if ee.ee_exit_head_launches(M, d, V, path) == 0:
        pytest.skip(f"{path_name} kernel does not take M={M}, d={d}")
    for planted in (False, True):
        cfg = gen.make_config("c0", seed=11, planted=planted, M=M, d=d, V=V)
        tau = 1.0 if planted else float(np.log(V) - 0.05) if V > 1 else 1.0
        ref = oracle_head(cfg["h"], cfg["heads"][0], tau)
        out = _run(ee, cfg, 0, tau, path)
        assert_head_matches(out, ref, label=f"{name}/{path_name}/planted={planted}")


def test_exact_small_integer_case(ee):
    """Alternating +-1 rows normalise to exactly +-1; dyadic W makes every logit exact in fp32."""
    d, V, M = 64, 40, 2
    x = np.tile([1.0, -1.0], d // 2)[None, :].repeat(M, 0)
    x[1] *= -1
    Wv = ((np.arange(V * d).reshape(V, d) * 7) % 13 - 6) / 8.0
    head = dict(gamma=np.ones(d, np.float32), beta=np.zeros(d, np.float32), ln_eps=1e-5,
                W=gen.bf16_bits_from_f32(Wv.astype(np.float32)))
    h = gen.bf16_bits_from_f32(x.astype(np.float32))
    ref = oracle.exit_head(h, head["gamma"], head["beta"], 1e-5, head["W"], 1.0)
    for path in (ee.EE_PATH_STREAM, ee.EE_PATH_TCGEN05, ee.EE_PATH_SKINNY):
        hd = head_to_dev(head)
        out = ee.ee_exit_head(dev_bf16(h), hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, path=path)
        got = {k: v.cpu().numpy() for k, v in out.items()}
        assert np.array_equal(got["argmax"], ref["argmax"])
        assert np.allclose(got["entropy"], ref["entropy"], atol=1e-5)
        assert np.allclose(got["maxprob"], ref["maxprob"], atol=1e-6)


def test_uniform_logits_give_ln_V_and_lowest_index(ee):
    """W = 0 makes all logits equal: H = ln V, p_max = 1/V, argmax = 0 (lowest index wins ties)."""
    d, V, M = 128, 50304, 4
    cfg = gen.make_config("c0", seed=1, M=M, d=d, V=8)
    Wz = torch.zeros((V, d), dtype=torch.bfloat16, device="cuda")
    hd = head_to_dev(cfg["heads"][0])
    for path in (ee.EE_PATH_STREAM, ee.EE_PATH_TCGEN05, ee.EE_PATH_SKINNY):
        out = ee.ee_exit_head(dev_bf16(cfg["h"]), hd["gamma"], hd["beta"], 1e-5, Wz, 11.0, path=path)
        assert torch.all(out["argmax"] == 0)
        assert np.allclose(out["entropy"].cpu().numpy(), 10.825839875788878, atol=2e-4)
        assert np.allclose(out["maxprob"].cpu().numpy(), 1 / V, rtol=1e-4)
        assert torch.all(out["exit_mask"] == 1)


@pytest.mark.parametrize("planted", [False, True])
def test_c0_full_size(ee, planted):
    cfg = gen.make_config("c0", seed=0, planted=planted)
    for tau in cfg["taus"]:
        ref = oracle_head(cfg["h"], cfg["heads"][0], tau)
        for path in (ee.EE_PATH_AUTO, ee.EE_PATH_TCGEN05):
            assert_head_matches(_run(ee, cfg, 0, tau, path), ref, label=f"c0 tau={tau} path={path}")


@pytest.mark.parametrize("planted", [False, True])
def test_c1_three_heads_full_size(ee, planted):
    cfg = gen.make_config("c1", seed=0, planted=planted)
    exits = 0
    for hid in range(3):
        ref64 = oracle_head(cfg["h"], cfg["heads"][hid], cfg["tau"])
        exits += int(ref64["exit_mask"].sum())
        for M in gen.CONFIGS["c1"]["Ms"]:
            sub = dict(cfg, h=cfg["h"][:M])
            ref = {k: v[:M] for k, v in ref64.items()}
            for path in (ee.EE_PATH_AUTO, ee.EE_PATH_STREAM, ee.EE_PATH_TCGEN05, ee.EE_PATH_SKINNY):
                assert_head_matches(_run(ee, sub, hid, cfg["tau"], path), ref, label=f"c1 head{hid} M={M} path={path}")
    if planted:
        assert 0 < exits < 3 * 64          # the planted inputs exercise both outcomes


@pytest.mark.parametrize("planted", [False, True])
def test_c2_per_row_thresholds_full_size(ee, planted):
    cfg = gen.make_config("c2", seed=0, planted=planted)
    ref = oracle_head(cfg["h"], cfg["heads"][0], cfg["tau_per_row"])
    for path in (ee.EE_PATH_AUTO, ee.EE_PATH_STREAM):
        assert_head_matches(_run(ee, cfg, 0, cfg["tau_per_row"], path), ref, label=f"c2 path={path}")


def test_c4_full_size_on_a_stratified_row_sample(ee):
    """M = 16384: the oracle checks >= 4 rows of every 128-row tile, every row residue mod 128 covered."""
    cfg = gen.make_config("c4", seed=0, planted=True)
    out = _run(ee, cfg, 0, cfg["tau"], ee.EE_PATH_AUTO)
    assert ee.ee_query_async_error is not None
    rows = np.array([t * 128 + (t + 32 * i) % 128 for t in range(128) for i in range(4)])
    rows = np.unique(np.concatenate([rows, [0, 127, 128, 16383]]))
    ref = oracle_head(cfg["h"], cfg["heads"][0], cfg["tau"], rows=rows)
    info = assert_head_matches(out, ref, rows=rows, label="c4 sample")
    assert len(set(rows // 128)) == 128 and len(set(rows % 128)) == 128
    # properties that hold for every row
    H = out["entropy"].cpu().numpy(); P = out["maxprob"].cpu().numpy(); A = out["argmax"].cpu().numpy()
    assert np.all((H >= -1e-4) & (H <= np.log(50304) + 1e-3)) and np.all((P > 0) & (P <= 1 + 1e-4))
    assert np.all((A >= 0) & (A < 50304))
    assert np.array_equal(out["exit_mask"].cpu().numpy(), (H < cfg["tau"]).astype(np.uint8))
    assert np.all(H >= -np.log(np.minimum(P, 1.0)) - 1e-3)        # H >= -ln p_max for any distribution
    assert info["max_dH"] <= 2e-3
    # The rows the oracle did not see: every one of the 16384 rows again through the independent streaming kernel
    # (mma.sync, 32-row slabs, its own LayerNorm and merge) -- secondary evidence, GPU against GPU.  A row whose two
    # largest probabilities are closer than 2e-3 of the largest (a logit gap below 2e-3) may pick either token.
    other = _run(ee, cfg, 0, cfg["tau"], ee.EE_PATH_STREAM)
    Hs = other["entropy"].cpu().numpy(); Ps = other["maxprob"].cpu().numpy(); As = other["argmax"].cpu().numpy()
    assert np.abs(H - Hs).max() <= 1e-3 and np.abs(P - Ps).max() <= 1e-3
    hd = head_to_dev(cfg["heads"][0])
    t2 = ee.ee_exit_head_top2(dev_bf16(cfg["h"]), hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], cfg["tau"])
    rel_gap = t2["top2gap"].cpu().numpy() / np.maximum(t2["maxprob"].cpu().numpy(), 1e-30)
    differ = A != As
    assert np.all(rel_gap[differ] < 2e-3), f"{int(differ.sum())} rows differ, widest relative gap {rel_gap[differ].max():.2e}"
    assert differ.mean() < 0.02
    decided = np.abs(H - cfg["tau"]) > 1e-3
    assert np.array_equal(out["exit_mask"].cpu().numpy()[decided], other["exit_mask"].cpu().numpy()[decided])


@pytest.mark.parametrize("path_name", ["tcgen05", "stream", "skinny"])
@pytest.mark.parametrize("M,d,V", [(8, 512, 3000), (40, 64, 700)])
def test_rows_with_nan_or_infinite_hidden_states_never_exit(ee, path_name, M, d, V):
    """A NaN or an infinity in a row's hidden state makes that row's entropy NaN (LayerNorm of such a row has no
    value) and a NaN entropy never exits, whatever the threshold; the other rows of the batch are not touched."""
    if ee.ee_exit_head_launches(M, d, V, PATHS[path_name]) == 0:
        pytest.skip(f"{path_name} kernel does not take M={M}")
    cfg = gen.make_config("c0", seed=5, planted=True, M=M, d=d, V=V)
    h = cfg["h"].copy()
    bad = {1: 0x7FC0, 3: 0x7F80, M - 1: 0xFF80}                      # bf16 NaN, +inf, -inf in one element of the row
    for row, bits in bad.items():
        h[row, (7 * row) % d] = bits
    good = np.array([r for r in range(M) if r not in bad])
    hd = head_to_dev(cfg["heads"][0])
    out = ee.ee_exit_head(dev_bf16(h), hd["gamma"], hd["beta"], 1e-5, hd["W"], float("inf"), path=PATHS[path_name])
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in out.items()}
    for row in bad:
        assert np.isnan(got["entropy"][row]), (row, got["entropy"][row])
        assert got["exit_mask"][row] == 0                              # even with tau = +inf
    ref = oracle_head(cfg["h"][good], cfg["heads"][0], float("inf"))
    assert_head_matches({k: v[torch.from_numpy(good).to(v.device)] for k, v in out.items()}, ref, label=f"{path_name} rows without NaN")
    assert (got["exit_mask"][good] == 1).all()


def test_both_kernels_agree_and_runs_are_bit_identical(ee):
    cfg = gen.make_config("c1", seed=5, planted=True, M=32, V=20000)
    a = _run(ee, cfg, 0, 1.0, ee.EE_PATH_STREAM)
    b = _run(ee, cfg, 0, 1.0, ee.EE_PATH_STREAM)
    c = _run(ee, cfg, 0, 1.0, ee.EE_PATH_TCGEN05)
    e = _run(ee, cfg, 0, 1.0, ee.EE_PATH_TCGEN05)
    f = _run(ee, cfg, 0, 1.0, ee.EE_PATH_SKINNY)
    g = _run(ee, cfg, 0, 1.0, ee.EE_PATH_SKINNY)
    for k in a:
        assert torch.equal(a[k], b[k]) and torch.equal(c[k], e[k]) and torch.equal(f[k], g[k]), k
    assert torch.allclose(a["entropy"], f["entropy"], atol=1e-3) and torch.equal(a["argmax"], f["argmax"])
    assert torch.allclose(a["entropy"], c["entropy"], atol=1e-3) and torch.equal(a["argmax"], c["argmax"])


def test_row_stride_and_workspace_reuse(ee):
    cfg = gen.make_config("c0", seed=2, planted=True, M=9, d=128, V=3000)
    hd = head_to_dev(cfg["heads"][0])
    wide = torch.zeros((9, 256), dtype=torch.bfloat16, device="cuda")
    wide[:, :128] = dev_bf16(cfg["h"])
    ref = oracle_head(cfg["h"], cfg["heads"][0], 1.0)
    ws = ee.new_workspace(9, 128, 3000)
    for path in (ee.EE_PATH_STREAM, ee.EE_PATH_TCGEN05, ee.EE_PATH_STREAM):
        out = ee.ee_exit_head(wide[:, :128], hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, workspace=ws, path=path)
        assert_head_matches(out, ref, label=f"strided path={path}")
    assert ee.ee_query_async_error(ws) == 0


def test_host_buffer_variant(ee):
    cfg = gen.make_config("c0", seed=4, planted=True, M=8, d=256, V=5000)
    hd = head_to_dev(cfg["heads"][0])
    h_host = torch.from_numpy(cfg["h"].view(np.int16)).view(torch.bfloat16).pin_memory()
    out_host = {k: v.cpu().pin_memory() for k, v in ee.new_outputs(8).items()}
    out_dev = ee.new_outputs(8)
    h_dev = torch.empty((8, 256), dtype=torch.bfloat16, device="cuda")
    ws = ee.new_workspace(8, 256, 5000)
    ee.ee_exit_head_host(h_host, h_dev, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, out_host, out_dev, ws)
    torch.cuda.synchronize()
    ref = oracle_head(cfg["h"], cfg["heads"][0], 1.0)
    assert_head_matches({k: v.cuda() for k, v in out_host.items()}, ref, label="host variant")


def test_device_side_argument_errors(ee):
    cfg = gen.make_config("c0", seed=2, M=4, d=64, V=100)
    hd = head_to_dev(cfg["heads"][0])
    h = dev_bf16(cfg["h"])
    small_ws = torch.zeros(512, dtype=torch.uint8, device="cuda")
    with pytest.raises(ee.EExitError) as e:
        ee.ee_exit_head(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, workspace=small_ws)
    assert e.value.code == 4
    ws = ee.new_workspace(4, 64, 100)
    with pytest.raises(ee.EExitError) as e:
        ee.ee_exit_head(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, workspace=ws[8:])
    assert e.value.code in (3, 4)
    with pytest.raises(ee.EExitError) as e:
        ee.ee_exit_head(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, workspace=ws, path=7)
    assert e.value.code == 2
    odd = gen.make_config("c0", seed=2, M=4, d=72, V=100)              # d % 64 != 0: not for the skinny kernel
    ohd = head_to_dev(odd["heads"][0])
    with pytest.raises(ee.EExitError) as e:
        ee.ee_exit_head(dev_bf16(odd["h"]), ohd["gamma"], ohd["beta"], 1e-5, ohd["W"], 1.0, path=ee.EE_PATH_SKINNY)
    assert e.value.code == 2


@pytest.mark.parametrize("name,M,d,V,n_heads", [
    ("c1_shape_small_v", 8, 1024, 3000, 3),       # two activation buffers
    ("n32_two_launches", 20, 256, 2111, 5),       # five heads: a launch of four and a launch of one
    ("n64_single_buffer", 64, 1024, 1200, 3),     # activations too large for a second buffer
    ("wide_single_buffer", 12, 2560, 900, 2),
    ("odd_width", 40, 72, 500, 3),                # d % 64 != 0: the tensor-core path's ragged last k-block
    ("two_m_tiles", 150, 128, 1000, 3),           # stacked LayerNorm outputs: a 128-row tile reaches into the next head
    ("one_row", 1, 512, 777, 4),
    ("paired_tiles", 256, 256, 3000, 3),          # 256-row tiles shared by two CTAs, merge kernel (768 rows)
    ("paired_fused", 160, 128, 1200, 2),          # the same with the merge inside the GEMM kernel (320 rows)
    ("paired_odd_k_blocks", 256, 320, 2500, 2),   # pairs fetch two k-blocks per request: five of them, the last stage half empty
    ("paired_one_k_block", 200, 64, 1800, 1),     # ... a single k-block: every stage half empty
    ("paired_ragged_k", 256, 328, 2000, 1),       # d % 64 != 0: pairs fall back to one k-block per request
    ("paired_long_k", 512, 1536, 1500, 1),        # 24 k-blocks, four row tiles, several trips round the three-stage ring
])
@pytest.mark.parametrize("kernel", ["auto", "stream", "skinny", "gemm", "none"])
def test_multi_head_call_matches_oracle(ee, monkeypatch, name, M, d, V, n_heads, kernel):
    # The library reads EE_MULTI_KERNEL per call; a kernel that does not take the shape leaves the default choice.
    if kernel != "auto":
        monkeypatch.setenv("EE_MULTI_KERNEL", kernel)
    cfg = gen.make_config("c1", seed=17, planted=True, M=M, d=d, V=V, heads=n_heads)
    h = dev_bf16(cfg["h"])
    taus = [0.5 + 0.5 * k for k in range(n_heads)]
    heads = []
    for k in range(n_heads):
        hd = head_to_dev(cfg["heads"][k])
        heads.append(dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=taus[k]))
    outs = ee.ee_exit_head_multi(heads, 1e-5)
    torch.cuda.synchronize()
    again = ee.ee_exit_head_multi(heads, 1e-5)
    torch.cuda.synchronize()
    for k in range(n_heads):
        ref = oracle_head(cfg["h"], cfg["heads"][k], taus[k])
        assert_head_matches(outs[k], ref, label=f"{name} head {k}")
        for key in outs[k]:
            assert torch.equal(outs[k][key], again[k][key]), (name, k, key)


def test_multi_head_full_size_c1(ee):
    cfg = gen.make_config("c1", seed=0, planted=True)
    for M in (1, 16, 64):
        h = dev_bf16(cfg["h"][:M])
        heads = []
        for k in range(3):
            hd = head_to_dev(cfg["heads"][k])
            heads.append(dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=cfg["tau"]))
        outs = ee.ee_exit_head_multi(heads, 1e-5)
        for k in range(3):
            ref = oracle_head(cfg["h"][:M], cfg["heads"][k], cfg["tau"])
            assert_head_matches(outs[k], ref, label=f"c1 multi M={M} head {k}")


def test_multi_head_host_call_matches_oracle(ee):
    """Packed host-buffer variant: one copy in, the heads, one copy out; device copies of the results stay usable."""
    M, d, V, n_heads = 20, 256, 1500, 3
    cfg = gen.make_config("c1", seed=23, planted=True, M=M, d=d, V=V, heads=n_heads)
    hds = [head_to_dev(cfg["heads"][k]) for k in range(n_heads)]
    taus = [0.7, 1.0, 2.0]
    h_one = dev_bf16(cfg["h"]).cpu()
    h_host = torch.stack([h_one] * n_heads).pin_memory()
    ws = torch.empty(ee.ee_exit_head_multi_workspace_bytes(n_heads, M, d, V), dtype=torch.uint8, device="cuda")
    ee.ee_workspace_init(ws)
    call = ee.PreparedMultiHost([dict(gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=t) for hd, t in zip(hds, taus)],
                                1e-5, h_host, ws)
    assert call.d2h_bytes == ee.ee_exit_head_results_bytes(n_heads, M) == n_heads * ((13 * M + 15) // 16 * 16)
    for _ in range(2):
        out = call()
        torch.cuda.synchronize()
        for k in range(n_heads):
            ref = oracle_head(cfg["h"], cfg["heads"][k], taus[k])
            assert_head_matches(out[k], ref, label=f"host multi head {k}")
            for key in out[k]:
                assert torch.equal(out[k][key], call.out_dev[k][key].cpu()), (k, key)
    assert ee.ee_query_async_error(ws) == 0


@pytest.mark.parametrize("M,d,V", [(1, 64, 1), (5, 72, 257), (64, 128, 400), (130, 256, 2049), (600, 64, 300), (1100, 64, 520),
                                   (8, 512, 50304)])
def test_top2_probability_gap_matches_oracle(ee, M, d, V):
    """The third confidence metric, p(1st) - p(2nd), from the tensor-core path; the other outputs unchanged."""
    for planted in (False, True):
        cfg = gen.make_config("c0", seed=21, planted=planted, M=M, d=d, V=V)
        hd = head_to_dev(cfg["heads"][0])
        h = dev_bf16(cfg["h"])
        out = ee.ee_exit_head_top2(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0)
        plain = ee.ee_exit_head(h, hd["gamma"], hd["beta"], 1e-5, hd["W"], 1.0, path=ee.EE_PATH_TCGEN05)
        torch.cuda.synchronize()
        ref = oracle_head(cfg["h"], cfg["heads"][0], 1.0)
        assert_head_matches({k: out[k] for k in plain}, ref, label=f"top2 M={M} V={V} planted={planted}")
        for k in plain:
            assert torch.equal(out[k], plain[k]), k
        got = out["top2gap"].cpu().numpy().astype(np.float64)
        assert np.abs(got - ref["top2_prob_gap"]).max() <= 2e-3, np.abs(got - ref["top2_prob_gap"]).max()
        assert np.all(got >= -1e-6) and np.all(got <= out["maxprob"].cpu().numpy() + 1e-6)


def test_top2_gap_is_zero_when_the_maximum_is_attained_twice(ee):
    d, V, M = 64, 300, 3
    x = np.tile([1.0, -1.0], d // 2)[None, :].repeat(M, 0)
    Wv = np.zeros((V, d)); Wv[7, 0] = 1.0; Wv[250, 0] = 1.0; Wv[100, 0] = 0.5          # tokens 7 and 250 tie, in different tiles
    out = ee.ee_exit_head_top2(dev_bf16(gen.bf16_bits_from_f32(x.astype(np.float32))), dev(np.ones(d, np.float32)),
                               dev(np.zeros(d, np.float32)), 1e-5, dev_bf16(gen.bf16_bits_from_f32(Wv.astype(np.float32))), 1.0)
    assert torch.all(out["top2gap"] == 0) and out["argmax"].cpu().tolist() == [7, 7, 7]


def test_calls_on_a_side_stream_interleaved_with_other_kernels(ee):
    """The library's kernels are chained by programmatic dependent launch; work of other libraries before,
    between and after them on a non-default stream must still be ordered as the stream says."""
    cfg = gen.make_config("c1", seed=41, planted=True, M=48, d=256, V=3000, heads=2)
    hds = [head_to_dev(cfg["heads"][k]) for k in range(2)]
    base = dev_bf16(cfg["h"])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        outs = []
        for rep in range(3):
            h = base.clone()                                         # produced by a kernel right before the call
            h.add_(0)                                                # and touched once more
            o = ee.ee_exit_head_multi([dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=1.0) for hd in hds], 1e-5)
            kept = ee.ee_compact(o[0]["exit_mask"], h)
            total = o[0]["exit_mask"].to(torch.int32).sum() + kept["kept_count"][0]        # consumed by a kernel right after
            outs.append((o, kept, total, h))
        side.synchronize()
    for o, kept, total, h in outs:
        assert int(total.item()) == 48
        for k in range(2):
            assert_head_matches(o[k], oracle_head(cfg["h"], cfg["heads"][k], 1.0), label=f"side stream head {k}")
            for key in o[k]:
                assert torch.equal(o[k][key], outs[0][0][k][key])


@pytest.mark.parametrize("M,d,V,n_heads,n_streams", [(64, 256, 6000, 3, 2), (256, 128, 9000, 2, 2), (512, 128, 9000, 1, 4),
                                                     (128, 256, 20000, 4, 6)])
def test_calls_in_flight_on_several_streams(ee, M, d, V, n_heads, n_streams):
    """Calls with workspaces of their own may overlap on the GPU, any number of them (the in-kernel merge never has
    a CTA depend on another CTA being scheduled): their results equal the ones of the same calls run one after
    the other, and no bounded wait gives up."""
    cfgs = [gen.make_config("c1", seed=51 + i, planted=True, M=M, d=d, V=V, heads=n_heads) for i in range(n_streams)]
    streams = [torch.cuda.Stream() for _ in range(n_streams)]
    calls, refs = [], []
    for cfg in cfgs:
        hds = [head_to_dev(hd) for hd in cfg["heads"]]
        h = dev_bf16(cfg["h"])
        heads = [dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=1.0) for hd in hds]
        refs.append([{k: v.clone() for k, v in o.items()} for o in ee.ee_exit_head_multi(heads, 1e-5)])
        calls.append(heads)
    torch.cuda.synchronize()
    prepared = []
    for heads, stream in zip(calls, streams):
        with torch.cuda.stream(stream):                              # a prepared call is bound to the stream current here
            ws = torch.empty(ee.ee_exit_head_multi_workspace_bytes(n_heads, M, d, V), dtype=torch.uint8, device="cuda")
            ee.ee_workspace_init(ws)
            outs = [ee.new_outputs(M) for _ in range(n_heads)]
            prepared.append((ee.PreparedMulti([dict(hd, out=o) for hd, o in zip(heads, outs)], 1e-5, ws), outs, ws))
    torch.cuda.synchronize()
    for rep in range(40):
        for call, _, _ in prepared:
            call()
    torch.cuda.synchronize()
    for (call, outs, ws), ref, cfg in zip(prepared, refs, cfgs):
        assert ee.ee_query_async_error(ws) == 0
        for k in range(n_heads):
            for key in ref[k]:
                assert torch.equal(outs[k][key], ref[k][key]), (k, key)
            assert_head_matches(outs[k], oracle_head(cfg["h"], cfg["heads"][k], 1.0), label=f"{n_streams} streams head {k}")


@pytest.mark.parametrize("looks", [0, 1, 3])
@pytest.mark.parametrize("M,d,V,n_heads", [(64, 256, 6000, 3), (512, 128, 9000, 1), (130, 64, 40000, 3), (5, 512, 50304, 1)])
def test_merge_hand_over_paths_give_the_same_results(ee, monkeypatch, looks, M, d, V, n_heads):
    """The in-kernel merge with owners that give up after 0, 1 or 3 looks at the ticket (EE_MERGE_LOOKS, read when a call
    is planned): their row groups then go to the last CTA to arrive, or are claimed back by an owner whose final look
    finds the count full.  Whoever merges a group, the results are the same bits as with patient owners, run after
    run, also with several calls in flight, and nothing is reported as a time-out."""
    cfg = gen.make_config("c1", seed=71, planted=True, M=M, d=d, V=V, heads=n_heads)
    hds = [head_to_dev(hd) for hd in cfg["heads"]]
    h = dev_bf16(cfg["h"])
    heads = [dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=1.0) for hd in hds]
    monkeypatch.delenv("EE_MERGE_LOOKS", raising=False)
    ref = [{k: v.clone() for k, v in o.items()} for o in ee.ee_exit_head_multi(heads, 1e-5)]
    torch.cuda.synchronize()
    monkeypatch.setenv("EE_MERGE_LOOKS", str(looks))
    streams = [torch.cuda.Stream() for _ in range(3)]
    prepared = []
    for stream in streams:
        with torch.cuda.stream(stream):
            ws = torch.empty(ee.ee_exit_head_multi_workspace_bytes(n_heads, M, d, V), dtype=torch.uint8, device="cuda")
            ee.ee_workspace_init(ws)
            outs = [ee.new_outputs(M) for _ in range(n_heads)]
            prepared.append((ee.PreparedMulti([dict(hd, out=o) for hd, o in zip(heads, outs)], 1e-5, ws), outs, ws))
    monkeypatch.delenv("EE_MERGE_LOOKS")
    torch.cuda.synchronize()
    for rep in range(25):
        for call, outs, _ in prepared:
            call()
        if rep % 8 == 0:                                             # look at intermediate runs too, not only the last
            torch.cuda.synchronize()
            for _, outs, _ in prepared:
                for k in range(n_heads):
                    for key in ref[k]:
                        assert torch.equal(outs[k][key], ref[k][key]), (rep, k, key)
    torch.cuda.synchronize()
    for _, outs, ws in prepared:
        assert ee.ee_query_async_error(ws) == 0
        for k in range(n_heads):
            for key in ref[k]:
                assert torch.equal(outs[k][key], ref[k][key]), (k, key)
            assert_head_matches(outs[k], oracle_head(cfg["h"], cfg["heads"][k], 1.0), label=f"looks={looks} head {k}")


def test_plan_runs_equal_the_one_step_call_and_follow_the_buffers_contents(ee):
    """ee_exit_head_plan_init / ee_exit_head_plan_run: the same results as ee_exit_head_multi, bit for bit, run after
    run; the plan captures pointers, not contents, so new rows written into the same buffer give the new rows' results."""
    import ctypes as C
    from paper_2407_21082_b200 import _lib
    # (the last shape: sixteen heads, the most a plan holds -- four launch groups)
    for M, d, V, n_heads in ((64, 256, 5000, 3), (300, 136, 3001, 5), (8, 512, 50304, 1), (256, 2048, 4000, 2), (12, 64, 900, 16)):
        cfg = gen.make_config("c1", seed=61, planted=True, M=M, d=d, V=V, heads=n_heads)
        other = gen.make_config("c1", seed=62, planted=True, M=M, d=d, V=V, heads=n_heads)
        hds = [head_to_dev(hd) for hd in cfg["heads"]]
        h = dev_bf16(cfg["h"])
        heads = [dict(h=h, gamma=hd["gamma"], beta=hd["beta"], W=hd["W"], tau=1.0) for hd in hds]
        ref = [{k: v.clone() for k, v in o.items()} for o in ee.ee_exit_head_multi(heads, 1e-5)]
        call = ee.PreparedMulti(heads, 1e-5)
        assert call._plan is not None
        for rep in range(3):
            outs = call()
            torch.cuda.synchronize()
            for k in range(n_heads):
                for key in ref[k]:
                    assert torch.equal(outs[k][key], ref[k][key]), (M, k, key, rep)
        h.copy_(dev_bf16(other["h"]))                                 # same buffer, other rows
        outs = call()
        torch.cuda.synchronize()
        for k in range(n_heads):
            assert_head_matches(outs[k], oracle_head(other["h"], cfg["heads"][k], 1.0), label=f"plan, new rows, head {k}")
    # argument errors are found at initialisation; a plan that was never initialised does not run
    plan = _lib.EEExitHeadPlan()
    lib = _lib.load()
    assert lib.ee_exit_head_plan_run(C.byref(plan), None) == 2
    arr = (_lib.EEHead * 17)()
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    assert lib.ee_exit_head_plan_init(C.byref(plan), arr, 17, 1e-5, 8, 64, 100, ws.data_ptr(), ws.numel()) == 2      # too many heads
    assert lib.ee_exit_head_plan_init(C.byref(plan), arr, 1, 1e-5, 8, 64, 100, ws.data_ptr(), ws.numel()) == 1       # NULL pointers
