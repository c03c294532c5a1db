"""fp64 CPU oracle for the self-supervised training objective of a head, forward pass (paper section 3.3,
paragraph "Losses": L_KL(y_hat || f_theta) = 1/L sum_t sum_v y_hat_v log(y_hat_v / f_theta(v)), with y_hat the
head's distribution and f_theta the main model's).

TEST INFRASTRUCTURE ONLY (see oracle/exit_head.py).  Shares no code with the CUDA sources.

Per token: both distributions are softmaxes of logits computed as in oracle.exit_head (LayerNorm rounded to bf16,
fp64 projection): the head's from its hidden states and weights, the teacher's from the final hidden states and
the main model's head.  kl = sum_v p_head(v) (log p_head(v) - log p_teacher(v)); the loss is the mean over tokens.

Pins (tests/test_oracle_kl.py): zero when head and teacher coincide, non-negativity, a two-class closed form,
compensated summation of the definition term by term, invariance to a shift of either logit vector.
"""
from __future__ import annotations

import numpy as np

from .exit_head import bf16_decode, layer_norm


def kl_from_logits(z_head: np.ndarray, z_teacher: np.ndarray) -> np.ndarray:
    """Per row: sum_v p(v) (log p(v) - log q(v)) with p = softmax(z_head), q = softmax(z_teacher)."""
    lp = z_head - z_head.max(axis=1, keepdims=True)
    lp = lp - np.log(np.exp(lp).sum(axis=1, keepdims=True))
    lq = z_teacher - z_teacher.max(axis=1, keepdims=True)
    lq = lq - np.log(np.exp(lq).sum(axis=1, keepdims=True))
    return (np.exp(lp) * (lp - lq)).sum(axis=1)


def ce_from_logits(z_head: np.ndarray, labels: np.ndarray) -> np.ndarray:
    """Per row: -log softmax(z_head)[label] (the supervised objective L_CE of the same paragraph)."""
    m = z_head.max(axis=1)
    log_z = m + np.log(np.exp(z_head - m[:, None]).sum(axis=1))
    return log_z - z_head[np.arange(z_head.shape[0]), labels]


def kl_to_teacher(h_head_bits, head, h_teacher_bits, teacher, rows_per_block: int = 64, labels=None) -> dict:
    """kl [M] per token and their mean (the loss); with labels also ce [M] and its mean (the hybrid objective is
    alpha * ce_loss + (1 - alpha) * loss).  head / teacher: dict(gamma, beta, ln_eps, W)."""
    M = h_head_bits.shape[0]
    Wh = bf16_decode(head["W"]).T.copy()
    Wt = bf16_decode(teacher["W"]).T.copy()
    parts, ce_parts = [], []
    for r0 in range(0, M, rows_per_block):
        yh = layer_norm(h_head_bits[r0:r0 + rows_per_block], head["gamma"], head["beta"], head["ln_eps"], True)
        yt = layer_norm(h_teacher_bits[r0:r0 + rows_per_block], teacher["gamma"], teacher["beta"], teacher["ln_eps"], True)
        zh = yh @ Wh
        parts.append(kl_from_logits(zh, yt @ Wt))
        if labels is not None:
            ce_parts.append(ce_from_logits(zh, np.asarray(labels)[r0:r0 + rows_per_block]))
    kl = np.concatenate(parts) if parts else np.zeros(0)
    out = dict(kl=kl, loss=float(kl.mean()) if M else 0.0)
    if labels is not None:
        ce = np.concatenate(ce_parts) if ce_parts else np.zeros(0)
        out.update(ce=ce, ce_loss=float(ce.mean()) if M else 0.0)
    return out
