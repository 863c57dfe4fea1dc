"""GPU parity of the CSRA objective (Eq. 2) through the C ABI against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import csra_oracle as co
from paper_2502_16880_b200 import lmhead, synth
from tests import parity_harness as ph

pytestmark = pytest.mark.gpu
TAU = 0.07


def _features(n, D, seed, rho=0.6):
    """Queries and `views` key blocks that share a per-position component (so that positives score high)."""
    rng = np.random.default_rng(seed)
    base = rng.standard_normal((n, D)).astype(np.float32)
    def view():
        return synth.fp32_to_bf16_bits(rho * base + math.sqrt(1 - rho * rho) * rng.standard_normal((n, D)).astype(np.float32))
    return view


def _run(Q, K, views, tau=TAU, logits=True):
    n, D = Q.shape
    ws = torch.empty(lmhead.coral_csra_workspace_bytes(n, views, D), dtype=torch.uint8, device="cuda")
    loss = torch.empty(1, dtype=torch.float32, device="cuda")
    rows = torch.empty(n, dtype=torch.float32, device="cuda")
    lg = torch.empty((n, views * n), dtype=torch.float32, device="cuda") if logits else None
    lmhead.coral_csra_infonce(ph.to_dev_bf16(Q), ph.to_dev_bf16(K), views, tau, ws, loss, rows, lg)
    assert lmhead.coral_csra_status(ws) == 0
    return float(loss.item()), rows.cpu().numpy(), None if lg is None else lg.cpu().numpy()


# Tolerance against the definition (Eq. 2 in float64).  The contraction's operands are the unit vectors held in
# bf16 (8 significant bits, spacing 2^-7 relative, round to nearest): each element moves by at most 2^-8 relative, a
# product of two by at most 2^-7 + 2^-16, so a scaled similarity by at most QUANT * sum_d |q_d k_d| / tau - a bound
# per element, at most QUANT / tau = 0.11 when |q| and |k| are parallel.  On top of it the fp32 accumulation over D products and the
# fp32 log-sum-exp: ACC_ATOL + ACC_RTOL |x| (measured on the LM head, same accumulator: 1e-6 on values of size 1).
# Rounding errors are independent and symmetric, so the error over many elements must also look like noise: its
# RMS at most that of uniform rounding (relative std at most 2^-7 / sqrt(12) per operand element), its mean close to zero -
# a truncating or doubly rounding conversion fails these two although it passes the bound.
QUANT = 2.0 ** -7 + 2.0 ** -16
SIGMA_REL = 2.0 ** -7 / math.sqrt(12.0)
ACC_ATOL, ACC_RTOL = 1e-4, 1e-4


def _bounds(Q, K, tau=TAU):
    qn, kn = co.normalise(Q), co.normalise(K)
    hard = QUANT * (np.abs(qn) @ np.abs(kn).T) / tau
    sigma = SIGMA_REL * np.sqrt(2.0 * ((qn * qn) @ (kn * kn).T)) / tau
    return hard, sigma


@pytest.mark.parametrize("n,D,views", [
    (1, 8, 1),            # the smallest problem: one query, one key
    (5, 40, 1),           # less than a tile; D not a multiple of 64
    (128, 64, 2),         # exactly one row block, two key tiles (one batch)
    (200, 328, 3),        # ragged rows, ragged last key tile, last 64-column block partly outside D
    (700, 256, 4),        # several row blocks and runs; positives in four different tiles
    (300, 512, 8),        # the maximum number of views
])
def test_csra_matches_oracle(n, D, views):
    v = _features(n, D, seed=n + views)
    Q = v()
    K = np.concatenate([v() for _ in range(views)])
    loss, rows, lg = _run(Q, K, views)
    ref = co.infonce(Q, K, views, TAU)                       # the definition: no rounded intermediate
    hard, sigma = _bounds(Q, K)
    err = lg.astype(np.float64) - ref["logits"]
    assert np.all(np.abs(err) <= hard + ACC_ATOL + ACC_RTOL * np.abs(ref["logits"])), np.abs(err).max()
    row_tol = 2 * hard.max(axis=1) + ACC_ATOL + ACC_RTOL * np.abs(ref["row_loss"])
    assert np.all(np.abs(rows - ref["row_loss"]) <= row_tol), np.abs(rows - ref["row_loss"]).max()
    assert abs(loss - ref["loss"]) <= row_tol.max()
    if err.size >= 1000:                                      # enough elements for the noise model to mean something
        rms_model = math.sqrt(float((sigma ** 2).mean()))
        assert math.sqrt(float((err ** 2).mean())) <= rms_model + ACC_ATOL
        assert abs(float(err.mean())) <= 5 * rms_model / math.sqrt(err.size) + ACC_ATOL
    # diagnostic, second: against the same steps with bf16 unit vectors the kernel's own arithmetic error is what is left
    quant = co.infonce_bf16_operands(Q, K, views, TAU)
    assert np.all(ph.close(lg, quant["logits"])), np.abs(lg - quant["logits"]).max()
    assert np.all(ph.close(rows, quant["row_loss"]))
    again = _run(Q, K, views)
    assert again[0] == loss and np.array_equal(again[1], rows)          # bitwise reproducible


def test_csra_closed_forms_on_the_gpu():
    n, D = 130, 256
    E = np.zeros((n, D), np.float32)
    E[np.arange(n), np.arange(n)] = 1.0 + (np.arange(n) % 7)
    Qb = synth.fp32_to_bf16_bits(E)
    loss, rows, _ = _run(Qb, Qb, 1, logits=False)
    want = math.log(math.exp(1 / TAU) + n - 1) - 1 / TAU
    assert np.allclose(rows, want, atol=1e-4) and abs(loss - want) < 1e-4
    d = synth.fp32_to_bf16_bits(np.tile(np.arange(1, D + 1, dtype=np.float32) % 5 - 2.0, (n, 1)))
    loss, rows, _ = _run(d, np.concatenate([d, d]), 2, logits=False)
    assert np.allclose(rows, math.log(2 * n), atol=2e-3)               # all similarities equal


def test_csra_full_size_sampled_rows():
    """The size the bench times (n = 4096 positions, three other steps + targets, D = 4096): sampled rows against
    the definition."""
    n, D, views = 4096, 4096, 4
    v = _features(n, D, seed=99)
    Q = v()
    K = np.concatenate([v() for _ in range(views)])
    loss, rows, _ = _run(Q, K, views, logits=False)
    pick = np.unique(np.linspace(0, n - 1, 16).astype(int))
    kn = co.normalise(K)
    qn = co.normalise(Q[pick])
    lg = qn @ kn.T / TAU
    mx = lg.max(axis=1)
    lse = mx + np.log(np.exp(lg - mx[:, None]).sum(axis=1))
    pos = np.stack([lg[np.arange(len(pick)), pick + s * n] for s in range(views)], 1).mean(axis=1)
    hard = QUANT * (np.abs(qn) @ np.abs(kn).T) / TAU
    sigma = SIGMA_REL * np.sqrt(2.0 * ((qn * qn) @ (kn * kn).T)) / TAU
    want = lse - pos
    assert np.all(np.abs(rows[pick] - want) <= 2 * hard.max(axis=1) + ACC_ATOL + ACC_RTOL * np.abs(want))
    # a row loss is a difference of two weighted means of similarities: its noise is at most that of two of them
    assert np.abs(rows[pick] - want).max() <= 8 * 2 * float(sigma.max()) + ACC_ATOL + ACC_RTOL * np.abs(want).max()
    assert abs(loss - rows.astype(np.float64).mean()) < 1e-4


def test_csra_argument_errors():
    lib = lmhead.load_library()
    import ctypes
    b = ctypes.c_size_t(0)
    assert lib.coral_csra_workspace_bytes(0, 1, 64, ctypes.byref(b)) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_csra_workspace_bytes(8, 9, 64, ctypes.byref(b)) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_csra_workspace_bytes(8, 1, 60, ctypes.byref(b)) == lmhead.CORAL_ERR_INVALID
    Q = ph.to_dev_bf16(_features(4, 64, 1)())
    ws = torch.empty(lmhead.coral_csra_workspace_bytes(4, 1, 64), dtype=torch.uint8, device="cuda")
    loss = torch.empty(1, dtype=torch.float32, device="cuda")
    with pytest.raises(lmhead.CoralError):
        lmhead.coral_csra_infonce(Q, Q, 1, 0.0, ws, loss)
