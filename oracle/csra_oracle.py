"""CPU oracle of the Cross-Step Representation Alignment objective.  TEST INFRASTRUCTURE: only the tests and the
bench's CPU-baseline leg may call it; it shares no code with the CUDA library and is never a fallback for it.

What it computes (CORAL Section 3.1, Eq. 2; Appendix A: temperature 0.07; the appendix on discrepancies between
training steps uses the same quantity between the features of two steps):

    q_i  : n query features (the B x S output features of the current step), k_j : m = views * n key features
           (the features of `views` other steps and/or the targets, block s holding positions 0 .. n-1),
    sim  : cosine similarity, sim(q, k) = q . k / (|q| |k|),
    loss_i = - mean over the views s of  log [ exp(sim(q_i, k_{i + s n}) / tau) / sum_j exp(sim(q_i, k_j) / tau) ]
           = LSE_j(sim(q_i, k_j) / tau) - mean_s sim(q_i, k_{i + s n}) / tau,
    loss   = mean_i loss_i.

`infonce` is that definition and nothing else: the bf16 inputs widened exactly to float64, float64 norms, a float64
quotient, a plain matmul, a plain log-sum-exp.  No intermediate is rounded to a narrower type.

Readings (the paper leaves them open): which features make up the key set F is the caller's choice (whatever
is passed as K); the positives of query i are the keys at the same position i in every block; several positives
are averaged; a zero feature is left at zero (its similarities are 0).

`infonce_bf16_operands` is a SECONDARY, diagnostic variant, not the definition: the same steps with the unit vectors
rounded once to bf16 (nearest-even) before the matmul, i.e. what a contraction with bf16 operands sees.  It exists
so that a test can separate "the kernel's arithmetic is wrong" from "the kernel's operand precision costs this
much"; parity is judged against `infonce`.

The paper prints InfoNCE values only for trained models on its own data, so value parity with the paper is
unpinned; the functions are pinned by closed forms, a library log-softmax, invariances and brute force
(tests/test_csra_oracle_pins.py).
"""
from __future__ import annotations

import numpy as np


def _widen(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def normalise(bits: np.ndarray) -> np.ndarray:
    """Rows of bf16 bit patterns -> float64 unit vectors x / |x| (a zero row stays zero)."""
    x = _widen(bits)
    nrm = np.sqrt((x * x).sum(axis=1, keepdims=True))
    with np.errstate(invalid="ignore", divide="ignore"):
        return np.where(nrm > 0, x / nrm, 0.0)


def _objective(qn: np.ndarray, kn: np.ndarray, views: int, tau: float):
    n = qn.shape[0]
    logits = (qn @ kn.T) / tau
    mx = logits.max(axis=1)
    lse = mx + np.log(np.exp(logits - mx[:, None]).sum(axis=1))
    idx = np.arange(n)
    pos = np.stack([logits[idx, idx + s * n] for s in range(views)], axis=1)
    row_loss = lse - pos.mean(axis=1)
    return {"logits": logits, "lse": lse, "pos": pos, "row_loss": row_loss, "loss": float(row_loss.mean())}


def _check(Q_bits, K_bits, views):
    if K_bits.shape[0] != views * Q_bits.shape[0] or views < 1:
        raise ValueError("K must hold views * n rows")


def infonce(Q_bits: np.ndarray, K_bits: np.ndarray, views: int, tau: float = 0.07):
    """Eq. 2 in float64.  Q_bits [n, D], K_bits [views * n, D] (bf16 bit patterns).  Returns dict(logits [n, m],
    lse [n], pos [n, views], row_loss [n], loss)."""
    _check(Q_bits, K_bits, views)
    return _objective(normalise(Q_bits), normalise(K_bits), views, tau)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bf16 (ties to even) in one rounding, returned as float64 values.  bf16 keeps 7 of the
    52 fraction bits of a double; values here lie in (2^-100, 1], far inside bf16's exponent range."""
    u = np.ascontiguousarray(x, dtype=np.float64).view(np.uint64)
    keep_lsb = (u >> np.uint64(45)) & np.uint64(1)
    r = ((u + np.uint64((1 << 44) - 1) + keep_lsb) >> np.uint64(45)) << np.uint64(45)
    return r.view(np.float64)


def infonce_bf16_operands(Q_bits: np.ndarray, K_bits: np.ndarray, views: int, tau: float = 0.07):
    """Diagnostic variant (see the module docstring): unit vectors rounded to bf16 before the matmul."""
    _check(Q_bits, K_bits, views)
    return _objective(round_to_bf16(normalise(Q_bits)), round_to_bf16(normalise(K_bits)), views, tau)
