"""Seeded synthetic inputs for the weight-grouped LM-head draft step.

This module only draws random numbers and rounds them to bf16 bit patterns.
It contains none of the method's arithmetic (no gate, no selection, no
matmul, no softmax) so that the CPU oracle and the CUDA path can both be fed
from it without sharing any computation.

Recipe (every tensor has its own counter-based stream, so a tensor does not
depend on which other tensors were drawn, nor on M):

    W_vocab  [V, H]  fp32 N(0, 0.02^2)  -> bf16 (round to nearest even)
    W_gate   [N, H]  fp32 N(0, 0.02^2)  -> bf16
    group_map[V]     perm = permutation(V); group_map[perm[i]] = i // (V / N)
    hidden   [M, H]  fp32 N(0, 1)       -> bf16; the first M rows of one
                     stream, so the M=1 rows are a prefix of the M=8 rows ...

Extra workload (not one of the graded configs): `zipf_s > 0` together with the contiguous group map
models the paper's frequency-ordered vocabulary, where low-index groups hold the frequent tokens and are
routed to most often.  One fixed unit direction u is drawn; W_gate[n] += -(zipf_s * ln(n + 1) / 8) * u and
every hidden row += 8 * u before rounding, so group n's score carries a prior of about -zipf_s * ln(n + 1)
on top of the N(0, (w_std * sqrt(H))^2) spread.  (Only sums and a rounding: the scores themselves are still
computed by the oracle and by the library, each on its own.)

The shapes are those of the draft heads in the paper's Table 1 (hidden size,
vocabulary) with the group counts and top-n of its Table 4 grid.
bf16 tensors are returned as numpy uint16 arrays holding the raw bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

_TAG_W_VOCAB = 1
_TAG_W_GATE = 2
_TAG_PERM = 3
_TAG_HIDDEN = 4
_TAG_PRIOR = 5
_PRIOR_GAIN = 8.0


@dataclass(frozen=True)
class HeadConfig:
    """Shape of one grouped LM head workload."""

    name: str
    H: int          # hidden size d
    V: int          # vocabulary size
    N: int          # number of LM-head groups
    k_groups: int   # top-n groups activated per row
    k_tokens: int   # candidates kept per row (top-10 in the paper's tree)
    M: int          # query rows (tree nodes x sequences)
    seed: int = 0
    w_std: float = 0.02
    rho: float = 0.0  # correlation between rows (0 = iid rows)
    zipf_s: float = 0.0  # strength of the frequency prior on low-index groups (0 = none)

    @property
    def v(self) -> int:
        return self.V // self.N

    def with_(self, **kw) -> "HeadConfig":
        return replace(self, **kw)


CONFIGS = {
    "tiny": HeadConfig("tiny", H=256, V=4096, N=16, k_groups=4, k_tokens=10, M=4),
    "llama2_7b": HeadConfig("llama2_7b", H=4096, V=32000, N=32, k_groups=4, k_tokens=10, M=8),
    "llama3_8b": HeadConfig("llama3_8b", H=4096, V=128256, N=64, k_groups=8, k_tokens=10, M=8),
    "qwen25_7b": HeadConfig("qwen25_7b", H=3584, V=152064, N=64, k_groups=8, k_tokens=10, M=60),
    "large_m": HeadConfig("large_m", H=4096, V=128256, N=64, k_groups=8, k_tokens=10, M=960),
}


def fp32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    # add 0x7FFF + lsb of the kept part, then truncate (finite inputs only)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_fp32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, tag: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tag)])


def _normal_bf16(rng: np.random.Generator, rows: int, cols: int, std: float) -> np.ndarray:
    out = np.empty((rows, cols), dtype=np.uint16)
    step = max(1, (1 << 24) // max(cols, 1))  # bounded fp32 temporaries
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        blk = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
        if std != 1.0:
            blk *= np.float32(std)
        out[r0:r1] = fp32_to_bf16_bits(blk)
    return out


def make_w_vocab(cfg: HeadConfig) -> np.ndarray:
    return _normal_bf16(_rng(cfg.seed, _TAG_W_VOCAB), cfg.V, cfg.H, cfg.w_std)


def _prior_direction(cfg: HeadConfig) -> np.ndarray:
    u = _rng(cfg.seed, _TAG_PRIOR).standard_normal(cfg.H, dtype=np.float32)
    return u / np.float32(np.sqrt(np.sum(u.astype(np.float64) ** 2)))


def make_w_gate(cfg: HeadConfig) -> np.ndarray:
    if cfg.zipf_s <= 0.0:
        return _normal_bf16(_rng(cfg.seed, _TAG_W_GATE), cfg.N, cfg.H, cfg.w_std)
    w = _rng(cfg.seed, _TAG_W_GATE).standard_normal((cfg.N, cfg.H), dtype=np.float32) * np.float32(cfg.w_std)
    b = (-cfg.zipf_s / _PRIOR_GAIN) * np.log(np.arange(1, cfg.N + 1, dtype=np.float64))
    return fp32_to_bf16_bits(w + b.astype(np.float32)[:, None] * _prior_direction(cfg)[None, :])


def make_group_map(cfg: HeadConfig, contiguous: bool = False) -> np.ndarray:
    """token -> group, every group holding exactly V/N tokens."""
    if cfg.V % cfg.N:
        raise ValueError("V must be a multiple of N")
    if contiguous:
        return (np.arange(cfg.V, dtype=np.int64) // cfg.v).astype(np.int32)
    perm = _rng(cfg.seed, _TAG_PERM).permutation(cfg.V)
    gm = np.empty(cfg.V, dtype=np.int32)
    gm[perm] = (np.arange(cfg.V, dtype=np.int64) // cfg.v).astype(np.int32)
    return gm


def make_hidden(cfg: HeadConfig, M: int | None = None, batch: int = 0) -> np.ndarray:
    """[M, H] bf16 bits. `batch` picks an independent batch of rows (the bench
    rotates through several so successive calls touch different groups).
    With rho > 0 the rows are sqrt(1-rho^2)*h0 + rho*eps_m: siblings of one
    parent node, an extra workload next to the iid one."""
    M = cfg.M if M is None else M
    rng = np.random.default_rng([int(cfg.seed), _TAG_HIDDEN, int(batch)])
    x = rng.standard_normal((M, cfg.H), dtype=np.float32)
    if cfg.rho > 0.0:
        h0 = np.random.default_rng([int(cfg.seed), _TAG_HIDDEN, int(batch), 1]).standard_normal(
            (1, cfg.H), dtype=np.float32)
        x = np.float32(np.sqrt(1.0 - cfg.rho ** 2)) * h0 + np.float32(cfg.rho) * x
    if cfg.zipf_s > 0.0:
        x = x + np.float32(_PRIOR_GAIN) * _prior_direction(cfg)[None, :]
    return fp32_to_bf16_bits(x)


def make_all(cfg: HeadConfig):
    """(W_vocab, group_map, W_gate, hidden) for one config."""
    return make_w_vocab(cfg), make_group_map(cfg), make_w_gate(cfg), make_hidden(cfg)
