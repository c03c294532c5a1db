"""Seeded synthetic tensors with the shapes of the Pythia-sized exit-head workloads.

Every tensor comes from its own counter-based Philox stream whose 128-bit key is a hash of
(seed, workload tag, tensor name), so a tensor does not change when another one is added or resized.
bf16 tensors are returned as numpy uint16 bit patterns (round-to-nearest-even from fp32); consumers
decode them however they like.  Nothing here evaluates the exit head.

Two families of inputs:

* literal  -- hidden rows h = a*u + N(0, I) with one random unit vector u and a ~ U(0, 6) per row,
  LayerNorm gamma = 1 + N(0, 0.1^2), beta = N(0, 0.02^2), W = N(0, 0.02^2).  With an iid random W every
  row ends up with an entropy close to ln V - sigma_z^2 / 2, so no row is confident.
* planted  -- J random unit directions u_j are tied to J distinct tokens t_j by adding kappa*u_j to row
  t_j of W before rounding; each hidden row follows one of the directions with strength a ~ U(0, 6).
  Strong rows become confident about their token, weak rows stay near-uniform, which gives a wide spread
  of entropies and non-trivial exit masks.  The same (t_j, u_j) are planted in every head of a workload.
"""
from __future__ import annotations

import hashlib

import numpy as np

V_PYTHIA = 50304

# Shapes of the five workloads (d, rows, heads, thresholds in nats).
CONFIGS = {
    "c0": dict(d=512, V=V_PYTHIA, M=8, heads=1, taus=(0.5, 1.0, 2.0)),
    "c1": dict(d=1024, V=V_PYTHIA, Ms=(1, 4, 16, 64), M=64, heads=3, taus=(1.0,), layers=(6, 12, 18)),
    "c2": dict(d=2048, V=V_PYTHIA, M=256, heads=1, tau_range=(0.25, 3.0)),
    "c3": dict(d=2560, V=V_PYTHIA, S=32, k=8, M=256, heads=2, taus=(1.0,), sigma_range=(0.0, 1.5)),
    "c4": dict(d=2560, V=V_PYTHIA, M=16384, heads=1, taus=(1.0,)),
}


def _rng(seed: int, *names) -> np.random.Generator:
    text = "|".join([str(int(seed))] + [str(n) for n in names]).encode()
    digest = hashlib.blake2b(text, digest_size=16).digest()
    key = np.frombuffer(digest, dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def bf16_bits_from_f32(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest, ties to even.  Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def f32_from_bf16_bits(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> the fp32 values they denote (exact)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _unit_rows(rng: np.random.Generator, n: int, d: int) -> np.ndarray:
    u = rng.standard_normal((n, d), dtype=np.float32)
    u /= np.linalg.norm(u.astype(np.float64), axis=1, keepdims=True).astype(np.float32)
    return u


def make_planting(seed: int, tag: str, d: int, V: int, J: int = 64) -> dict:
    """J unit directions and J distinct token ids they are tied to."""
    J = min(J, V)
    rng = _rng(seed, tag, "planting")
    tokens = rng.choice(V, size=J, replace=False).astype(np.int64)
    return dict(tokens=tokens, U=_unit_rows(rng, J, d))


def make_head(seed: int, tag: str, head_id: int, d: int, V: int,
              planting: dict | None = None, kappa: float = 4.0) -> dict:
    """One exit head: LayerNorm (gamma, beta fp32 [d]) and W (bf16 bits [V, d]), eps = 1e-5."""
    rng = _rng(seed, tag, "head", head_id)
    gamma = (1.0 + 0.1 * rng.standard_normal(d, dtype=np.float32)).astype(np.float32)
    beta = (0.02 * rng.standard_normal(d, dtype=np.float32)).astype(np.float32)
    W = rng.standard_normal((V, d), dtype=np.float32)
    W *= np.float32(0.02)
    if planting is not None:
        W[planting["tokens"]] += np.float32(kappa) * planting["U"]
    return dict(gamma=gamma, beta=beta, W=bf16_bits_from_f32(W), ln_eps=1e-5)


def _hidden_f32(rng: np.random.Generator, M: int, d: int, planting: dict | None):
    a = rng.uniform(0.0, 6.0, size=M).astype(np.float32)
    if planting is None:
        u = _unit_rows(rng, 1, d)
        direction = np.broadcast_to(u, (M, d))
        j = np.zeros(M, dtype=np.int64)
    else:
        j = rng.integers(0, planting["U"].shape[0], size=M)
        direction = planting["U"][j]
    h = rng.standard_normal((M, d), dtype=np.float32)
    h += a[:, None] * direction
    return h, a, j


def make_hidden(seed: int, tag: str, M: int, d: int, planting: dict | None = None) -> dict:
    """Hidden rows h (bf16 bits [M, d]) = a*u + N(0, I)."""
    rng = _rng(seed, tag, "hidden")
    h, a, j = _hidden_f32(rng, M, d, planting)
    return dict(h=bf16_bits_from_f32(h), a=a, j=j)


def make_dssd_hidden(seed: int, tag: str, S: int, k: int, d: int, planting: dict | None = None,
                     sigma_range=(0.0, 1.5)) -> dict:
    """Verify rows [S*k, d] as in make_hidden, and draft rows = verify + sigma_s * N(0, I) per sequence."""
    rng = _rng(seed, tag, "dssd_hidden")
    hv, a, j = _hidden_f32(rng, S * k, d, planting)
    hv_bits = bf16_bits_from_f32(hv)
    sigma = rng.uniform(sigma_range[0], sigma_range[1], size=S).astype(np.float32)
    noise = rng.standard_normal((S * k, d), dtype=np.float32)
    hd = f32_from_bf16_bits(hv_bits) + np.repeat(sigma, k)[:, None] * noise
    return dict(h_verify=hv_bits, h_draft=bf16_bits_from_f32(hd), sigma=sigma, a=a, j=j)


def make_config(name: str, seed: int = 0, planted: bool = False, *, M: int | None = None,
                V: int | None = None, d: int | None = None, heads: int | None = None) -> dict:
    """All tensors of one workload.  M, V, d, heads override the shape (reduced-size test variants)."""
    spec = dict(CONFIGS[name])
    d = int(d if d is not None else spec["d"])
    V = int(V if V is not None else spec["V"])
    n_heads = int(heads if heads is not None else spec["heads"])
    tag = f"{name}/{'planted' if planted else 'literal'}/d{d}/V{V}"
    planting = make_planting(seed, tag, d, V) if planted else None
    out = dict(name=name, d=d, V=V, planted=planted, ln_eps=1e-5,
               heads=[make_head(seed, tag, hid, d, V, planting) for hid in range(n_heads)])
    if name == "c3":
        S, k = spec["S"], spec["k"]
        if M is not None:
            S = max(1, int(M) // k)
        out.update(S=S, k=k, M=S * k, tau=spec["taus"][0])
        out.update(make_dssd_hidden(seed, tag, S, k, d, planting, spec["sigma_range"]))
        return out
    M = int(M if M is not None else spec["M"])
    out.update(M=M, **make_hidden(seed, tag, M, d, planting))
    if name == "c2":
        lo, hi = spec["tau_range"]
        out["tau_per_row"] = _rng(seed, tag, "tau").uniform(lo, hi, size=M).astype(np.float32)
    else:
        out["taus"] = spec["taus"]
        out["tau"] = spec["taus"][min(1, len(spec["taus"]) - 1)]
    return out


def random_token_case(seed: int, S: int, k: int, kv: int, alphabet: int = 3, p_confident: float = 0.85,
                      p_mismatch: float = 0.15) -> dict:
    """Random draft/verify token arrays: the verifier's tokens equal the draft's except for slots replaced
    with probability p_mismatch (small alphabet, so a replacement can still coincide), and extra verifier
    columns beyond k are random.  Every prefix length occurs for moderate S."""
    rng = _rng(seed, "tokens", S, k, kv, alphabet)
    draft = rng.integers(0, alphabet, size=(S, k)).astype(np.int32)
    verify = rng.integers(0, alphabet, size=(S, kv)).astype(np.int32)
    keep = rng.random((S, k)) >= p_mismatch
    verify[:, :k] = np.where(keep, draft, verify[:, :k])
    return dict(draft_tok=draft, verify_tok=verify,
                draft_exit_mask=(rng.random((S, k)) < p_confident).astype(np.uint8))


def make_calibration_set(seed: int, n: int, V: int = 50304, ties: bool = False) -> dict:
    """A stand-in for the scores a calibration epoch stores per head: an entropy per token (nats, spread over
    0 .. ln V like the planted workloads' entropies: a surer half and a diffuse half), the head's token and the
    full model's token, which agree more often where the entropy is low.  `ties` rounds the entropies to two
    decimals so that many tokens share a value."""
    rng = _rng(seed, "calibration", n, V)
    sure = rng.random(n) < 0.45
    H = np.where(sure, rng.gamma(1.2, 0.25, size=n), np.log(V) - rng.gamma(2.0, 1.2, size=n))
    H = np.clip(H, 0.0, np.log(V)).astype(np.float32)
    if ties:
        H = np.round(H, 2).astype(np.float32)
    final = rng.integers(0, V, size=n).astype(np.int32)
    agree = rng.random(n) < np.exp(-H.astype(np.float64) / 2.5)
    head = np.where(agree, final, (final + 1 + rng.integers(0, V - 1, size=n)) % V).astype(np.int32)
    return dict(entropy=H, argmax_head=head, argmax_final=final)


def make_markov_model(seed: int, V: int, d: int, planting: dict | None, sigma: float = 0.5) -> dict:
    """A stand-in for the transformer below the heads in a decoding loop: the hidden state of a position depends
    on the previous token only.  Two tables of bf16 rows [V, d], one read by the draft head and one by the full
    model's head; row t is a*u + N(0, I) as in make_hidden (with a planting the direction is one of the planted
    ones, so the heads answer with that direction's token), the draft table = the other + sigma * N(0, I)."""
    rng = _rng(seed, "markov", V, d)
    hv, a, j = _hidden_f32(rng, V, d, planting)
    hv_bits = bf16_bits_from_f32(hv)
    hd = f32_from_bf16_bits(hv_bits) + np.float32(sigma) * rng.standard_normal((V, d), dtype=np.float32)
    return dict(E_verify=hv_bits, E_draft=bf16_bits_from_f32(hd), a=a, j=j)

