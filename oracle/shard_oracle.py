"""CPU oracle for the vocab-sharded draft step.  TEST INFRASTRUCTURE: only the tests may call it; it shares no
code with the CUDA library and is never a fallback for it.

With `world` GPUs the N groups of the LM head (paper Section 3.3: V split equally into N groups) are dealt
round-robin, group n to rank n % world.  Appendix B's cost statement - the groups involved by the rows are
what must be read - then splits by rank: a rank computes, for every row, the logits of those of the row's
selected groups that it owns, and summarises them in one record per row:

    max of its logits, sum of exp(logit - max), its k_tokens largest logits (descending, equal -> lower
    token id) and their token ids;  (-inf, 0, -inf..., NO_TOKEN...) when it owns none of the row's groups.

The joint softmax over a row's active logits (the reading the workload definitions fix) is recovered exactly
from the records: LSE = M + log sum_r s_r exp(m_r - M) with M = max_r m_r, and the row's k_tokens best tokens
are the best of the ranks' lists.  Arithmetic in float64, from the logits of lmhead_oracle.draft.

Pins (tests/test_shard_oracle_pins.py): merging the records of any world size reproduces the unsharded
oracle's ids and log-probs; world = 1 is the identity; the ranks' active sets partition the row's.
"""
from __future__ import annotations

import numpy as np

NO_TOKEN = 0x7FFFFFFF


def records(result, rank: int, world: int, k_tokens: int):
    """result: OracleResult of lmhead_oracle.draft (with logits).  Returns (mx [M], sm [M], z [M, k_tokens],
    ids [M, k_tokens]) for the groups n of each row with n % world == rank."""
    M = result.groups.shape[0]
    mx = np.full(M, -np.inf)
    sm = np.zeros(M)
    z = np.full((M, k_tokens), -np.inf)
    ids = np.full((M, k_tokens), NO_TOKEN, dtype=np.int64)
    for m in range(M):
        slots = [s for s, n in enumerate(result.groups[m]) if n % world == rank]
        if not slots:
            continue
        lg = np.concatenate([result.logits[m, s] for s in slots])
        tk = np.concatenate([result.logit_tokens[m, s] for s in slots])
        mx[m] = lg.max()
        sm[m] = np.exp(lg - mx[m]).sum()
        order = np.lexsort((tk, -lg))[:k_tokens]          # logit descending, token id ascending among equals
        z[m, :len(order)] = lg[order]
        ids[m, :len(order)] = tk[order]
    return mx, sm, z, ids


def pack(mx, sm, z, ids) -> np.ndarray:
    """The exchange format: [M, 2 + 2 k_tokens] 32-bit words (max, sum, logits as float32; ids as int32)."""
    M, k = z.shape
    out = np.empty((M, 2 + 2 * k), dtype=np.int32)
    out[:, 0] = mx.astype(np.float32).view(np.int32)
    out[:, 1] = sm.astype(np.float32).view(np.int32)
    out[:, 2:2 + k] = z.astype(np.float32).view(np.int32)
    out[:, 2 + k:] = ids.astype(np.int32)
    return out


def merge(gathered: np.ndarray, k_tokens: int):
    """gathered: [world, M, 2 + 2 k_tokens] int32 words, rank-major.  Returns (ids [M, k], logprobs [M, k])."""
    world, M, _ = gathered.shape
    k = k_tokens
    mx = gathered[:, :, 0].copy().view(np.float32).astype(np.float64)
    sm = gathered[:, :, 1].copy().view(np.float32).astype(np.float64)
    z = gathered[:, :, 2:2 + k].copy().view(np.float32).astype(np.float64)
    ids = gathered[:, :, 2 + k:].astype(np.int64)
    out_ids = np.empty((M, k), dtype=np.int64)
    out_lp = np.empty((M, k))
    for m in range(M):
        top = mx[:, m].max()
        with np.errstate(invalid="ignore"):
            w = np.where(np.isneginf(mx[:, m]), 0.0, sm[:, m] * np.exp(mx[:, m] - top))
        lse = top + np.log(w.sum())
        cz, ci = z[:, m].ravel(), ids[:, m].ravel()
        order = np.lexsort((ci, -cz))[:k]
        out_ids[m] = ci[order]
        out_lp[m] = cz[order] - lse
    return out_ids, out_lp
