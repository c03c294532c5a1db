"""The seeded generators: determinism, shapes, value ranges.  No early-exit arithmetic lives there."""
import numpy as np

import gen


def test_same_seed_same_tensors_and_streams_are_independent():
    a = gen.make_config("c0", seed=0, V=300, d=64)
    b = gen.make_config("c0", seed=0, V=300, d=64)
    c = gen.make_config("c0", seed=1, V=300, d=64)
    assert np.array_equal(a["h"], b["h"]) and np.array_equal(a["heads"][0]["W"], b["heads"][0]["W"])
    assert not np.array_equal(a["h"], c["h"])
    # growing M keeps nothing fixed by accident but the head (its stream does not depend on M)
    e = gen.make_config("c0", seed=0, V=300, d=64, M=20)
    assert np.array_equal(e["heads"][0]["W"], a["heads"][0]["W"]) and e["h"].shape == (20, 64)


def test_shapes_dtypes_and_statistics():
    c = gen.make_config("c1", seed=0, V=4096, d=128, M=16)
    assert len(c["heads"]) == 3 and c["h"].dtype == np.uint16 and c["h"].shape == (16, 128)
    W = gen.f32_from_bf16_bits(c["heads"][1]["W"])
    assert W.shape == (4096, 128) and abs(W.std() - 0.02) < 5e-4 and abs(W.mean()) < 1e-3
    assert not np.array_equal(c["heads"][0]["W"], c["heads"][1]["W"])
    g = c["heads"][0]["gamma"]
    assert g.dtype == np.float32 and abs(g.mean() - 1) < 0.05 and c["heads"][0]["beta"].dtype == np.float32
    assert (c["a"] >= 0).all() and (c["a"] <= 6).all()


def test_planting_adds_directions_to_distinct_token_rows():
    lit = gen.make_config("c0", seed=0, V=500, d=64)
    pl = gen.make_config("c0", seed=0, planted=True, V=500, d=64)
    W = gen.f32_from_bf16_bits(pl["heads"][0]["W"])
    norms = np.linalg.norm(W, axis=1)
    assert (norms > 2).sum() == 64                    # 64 rows carry a kappa = 4 direction
    assert lit["planted"] is False and pl["planted"] is True


def test_c2_c3_extras():
    c2 = gen.make_config("c2", seed=0, V=300, d=64, M=40)
    assert c2["tau_per_row"].shape == (40,) and c2["tau_per_row"].min() >= 0.25 and c2["tau_per_row"].max() <= 3.0
    c3 = gen.make_config("c3", seed=0, planted=True, V=300, d=64, M=24)
    assert c3["S"] == 3 and c3["k"] == 8 and c3["h_draft"].shape == c3["h_verify"].shape == (24, 64)
    assert len(c3["heads"]) == 2 and c3["sigma"].shape == (3,)


def test_bf16_pack_unpack():
    x = np.float32([1.0, 1.00390625, 1.01171875, -2.5, 0.0])      # 1 + 2^-8 is a tie -> even (1.0); 1 + 3*2^-8 -> 1.015625
    bits = gen.bf16_bits_from_f32(x)
    assert gen.f32_from_bf16_bits(bits).tolist() == [1.0, 1.0, 1.015625, -2.5, 0.0]
