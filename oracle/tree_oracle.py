"""CPU oracle of the tree-expansion score step.  TEST INFRASTRUCTURE only (tests, smoke, bench baseline).

What it computes (CORAL Section 2.2: several candidates per timestep form a draft tree; Section 4.1: depth 6,
60 candidate tokens; Appendix B: top 10 candidates per node): for each sequence, every node's candidates get
  child score = parent's cumulative log-score + candidate log-probability,
and the K children with the highest score are kept, sorted descending, equal scores ordered by the flat
(node, candidate) index.  The paper does not spell the rule out (it refers to EAGLE-2's dynamic tree), so the
cumulative-log-probability ranking is a reading of the paper, not a quotation.  The addition is taken in fp32,
the precision the kernel decides in, so that the selected indices can be compared bit for bit.
Plain numpy, a full stable sort, no shortcuts.
"""
from __future__ import annotations

import numpy as np


def expand(parent_scores, cand_ids, cand_logprobs, K):
    """parent_scores [n_seq, nodes] f32; cand_ids, cand_logprobs [n_seq, nodes, k_tokens] (logprobs may be None
    with k_tokens = 1; ids may be None).  Returns (parent [n_seq, K] i32, token [n_seq, K] i32, score [n_seq, K] f32)."""
    ps = np.asarray(parent_scores, np.float32)
    n_seq, nodes = ps.shape
    if cand_logprobs is None:
        k_tokens = 1
        child = ps.reshape(n_seq, nodes, 1).copy()
    else:
        lp = np.asarray(cand_logprobs, np.float32)
        k_tokens = lp.shape[2]
        child = (ps[:, :, None] + lp).astype(np.float32)          # one fp32 addition per child
    C = nodes * k_tokens
    if not 1 <= K <= C:
        raise ValueError("K out of range")
    parent = np.zeros((n_seq, K), np.int32)
    token = np.zeros((n_seq, K), np.int32)
    score = np.zeros((n_seq, K), np.float32)
    for s in range(n_seq):
        flat = child[s].reshape(C)
        order = sorted(range(C), key=lambda i: (-float(flat[i]), i))[:K]
        for r, i in enumerate(order):
            parent[s, r] = i // k_tokens
            token[s, r] = i if cand_ids is None else int(np.asarray(cand_ids)[s].reshape(C)[i])
            score[s, r] = flat[i]
    return parent, token, score
