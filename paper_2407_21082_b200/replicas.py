"""Host-side plumbing for running the exit-head path on several GPUs.

Rows are independent and every head's weights are replicated, so the path has no exchange step: each rank
(one process per GPU) evaluates its own rows and no collective touches the data.  This module holds the
little that remains: which rows a rank takes when one batch is split, the seed of a rank's own synthetic
batch, and the aggregation of a timed run (time = slowest rank, work = sum over ranks).  It uses
`torch.distributed` only for those scalars and works with any backend (NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations


def shard_rows(total_rows: int, world_size: int, rank: int) -> tuple[int, int]:
    """[begin, end) of the rows rank `rank` takes when `total_rows` rows are split over `world_size` ranks.

    Contiguous, ordered by rank, sizes differ by at most one (the first `total_rows % world_size` ranks take
    the extra row), so concatenating the ranks' outputs in rank order restores the batch order.
    """
    if world_size < 1 or not 0 <= rank < world_size or total_rows < 0:
        raise ValueError("shard_rows: need world_size >= 1, 0 <= rank < world_size, total_rows >= 0")
    base, extra = divmod(total_rows, world_size)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic batch of one replica: distinct per rank, reproducible."""
    return int(base_seed) * 1_000_003 + int(rank)


def aggregate_timing(local_ms: float, local_units: float, dist=None, device=None) -> dict:
    """Whole-job figures of a timed region: elapsed = max over ranks, units = sum over ranks.

    `dist` is `torch.distributed` with an initialised process group, or None for a single process.
    """
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return dict(elapsed_ms=float(local_ms), units=float(local_units), world_size=1,
                    units_per_s=float(local_units) / (float(local_ms) * 1e-3) if local_ms > 0 else 0.0)
    import torch
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    ms, units = float(t.item()), float(u.item())
    return dict(elapsed_ms=ms, units=units, world_size=dist.get_world_size(),
                units_per_s=units / (ms * 1e-3) if ms > 0 else 0.0)


def gather_rows(local, dist=None):
    """Concatenation, in rank order, of the per-rank output arrays of a split batch (numpy, on the host).

    For callers that need the whole batch's decisions on every rank; the hot path itself never calls it.
    """
    import numpy as np
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return np.asarray(local)
    parts = [None] * dist.get_world_size()
    dist.all_gather_object(parts, np.asarray(local))
    return np.concatenate(parts, axis=0)
