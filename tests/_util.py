"""Helpers shared by the GPU parity tests: moving generator output to the device and the comparison rule."""
import numpy as np
import torch

import oracle

ENTROPY_TOL = 2e-3      # absolute, nats
MAXPROB_TOL = 2e-3      # absolute
GAP_MIN = 1e-3          # rows whose two largest oracle logits are closer than this are not compared on argmax
MARGIN_MIN = 1e-3       # rows with |H - tau| below this are not compared on the exit mask


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def head_to_dev(head: dict) -> dict:
    return dict(gamma=dev(head["gamma"]), beta=dev(head["beta"]), W=dev_bf16(head["W"]), ln_eps=head["ln_eps"])


def oracle_head(h_bits, head, tau, rows=None):
    if rows is not None:
        h_bits = h_bits[rows]
        if isinstance(tau, np.ndarray):
            tau = tau[rows]
    return oracle.exit_head(h_bits, head["gamma"], head["beta"], head["ln_eps"], head["W"], tau)


def assert_head_matches(out: dict, ref: dict, rows=None, label=""):
    """out: dict of CUDA tensors from ee_exit_head; ref: oracle dict (for `rows` of the batch if given)."""
    got = {k: v.cpu().numpy() for k, v in out.items()}
    if rows is not None:
        got = {k: v[rows] for k, v in got.items()}
    keep = oracle.decisive_rows(ref, GAP_MIN, MARGIN_MIN)
    dH = np.abs(got["entropy"].astype(np.float64) - ref["entropy"])
    dP = np.abs(got["maxprob"].astype(np.float64) - ref["maxprob"])
    assert np.all(np.isfinite(got["entropy"])), label
    assert dH.max() <= ENTROPY_TOL, f"{label}: entropy off by {dH.max():.3e} at row {dH.argmax()}"
    assert dP.max() <= MAXPROB_TOL, f"{label}: maxprob off by {dP.max():.3e} at row {dP.argmax()}"
    bad = np.flatnonzero((got["argmax"] != ref["argmax"]) & keep["argmax"])
    assert bad.size == 0, f"{label}: argmax differs on decisive rows {bad[:8]} got {got['argmax'][bad[:8]]} want {ref['argmax'][bad[:8]]}"
    bad = np.flatnonzero((got["exit_mask"] != ref["exit_mask"]) & keep["exit_mask"])
    assert bad.size == 0, f"{label}: exit mask differs on decisive rows {bad[:8]}"
    # undecisive rows must still be valid: the chosen token is one of the near-tied maxima
    excluded = dict(argmax=np.flatnonzero(~keep["argmax"]), exit_mask=np.flatnonzero(~keep["exit_mask"]))
    return dict(max_dH=float(dH.max()), max_dP=float(dP.max()), excluded=excluded)
