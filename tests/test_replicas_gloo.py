"""N > 1 host logic on CPU: two gloo ranks split a batch, each evaluates its rows, and the pieces are put
together.  The per-rank evaluation here is the oracle (the test checks the sharding and the aggregation, not
a kernel): rows are independent, so rank-ordered concatenation must equal the evaluation of the whole batch,
compaction indices shift by the shard offset, and the timing aggregate is max-time / summed units."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import gen
import oracle
from paper_2407_21082_b200 import replicas


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = gen.make_config("c0", seed=3, planted=True, M=13, V=640, d=64)
        hd = cfg["heads"][0]
        b, e = replicas.shard_rows(cfg["M"], world, rank)
        tau = cfg["tau"]
        local = oracle.exit_head(cfg["h"][b:e], hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], tau)
        comp = oracle.compact(local["exit_mask"], cfg["h"][b:e])
        whole = {k: replicas.gather_rows(local[k], dist) for k in ("argmax", "entropy", "maxprob", "exit_mask")}
        kept = replicas.gather_rows(comp["kept_idx"] + b, dist)
        h_kept = replicas.gather_rows(comp["h_out"], dist)
        agg = replicas.aggregate_timing(10.0 * (rank + 1), float(e - b), dist)
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), kept=kept, h_kept=h_kept, elapsed=agg["elapsed_ms"], units=agg["units"],
                 rate=agg["units_per_s"], shard=np.array([b, e]), **whole)
    finally:
        dist.destroy_process_group()


def test_shard_rows_partitions():
    for total in (0, 1, 7, 64, 65, 1000):
        for world in (1, 2, 3, 8):
            spans = [replicas.shard_rows(total, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        replicas.shard_rows(4, 2, 2)


def test_rank_seeds_distinct():
    assert len({replicas.rank_seed(0, r) for r in range(64)}) == 64
    assert replicas.rank_seed(5, 1) == replicas.rank_seed(5, 1)


def test_single_process_aggregate():
    agg = replicas.aggregate_timing(2.0, 100.0)
    assert agg["world_size"] == 1 and agg["units_per_s"] == pytest.approx(50_000.0)


@pytest.mark.timeout(120)
def test_two_gloo_ranks_match_whole_batch(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    cfg = gen.make_config("c0", seed=3, planted=True, M=13, V=640, d=64)
    hd = cfg["heads"][0]
    ref = oracle.exit_head(cfg["h"], hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], cfg["tau"])
    ref_comp = oracle.compact(ref["exit_mask"], cfg["h"])
    assert 0 < ref_comp["kept_count"] < cfg["M"]             # the case has both exits and survivors
    spans = []
    for rank in range(world):
        got = np.load(os.path.join(str(tmp_path), f"rank{rank}.npz"))
        for k in ("argmax", "exit_mask"):
            np.testing.assert_array_equal(got[k], ref[k])
        for k in ("entropy", "maxprob"):
            np.testing.assert_allclose(got[k], ref[k], rtol=0, atol=1e-12)
        np.testing.assert_array_equal(got["kept"], ref_comp["kept_idx"])
        np.testing.assert_array_equal(got["h_kept"], ref_comp["h_out"])
        assert float(got["elapsed"]) == 20.0                 # the slower rank
        assert float(got["units"]) == 13.0                   # all rows
        assert float(got["rate"]) == pytest.approx(13.0 / 20e-3)
        spans.append(tuple(int(x) for x in got["shard"]))
    assert spans == [(0, 7), (7, 13)]
