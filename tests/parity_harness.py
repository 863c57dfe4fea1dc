"""Element-by-element comparison of the CUDA draft step with the CPU oracle.

Tolerance (stated by the target for this path): tol(a, b) = 1e-3 + 1e-3 * max(|a|, |b|)
for logits, log-sum-exp and log-probs; group ids and token ids bit-exact except
where the oracle's own scores of the two candidates tie within that tolerance
(fp32 accumulation on the GPU against fp64 in the oracle can order such a pair
either way).  A row whose group choice differs only by such a tie is re-run in
the oracle with the GPU's groups forced, and counted.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from oracle import lmhead_oracle as orc

ATOL = 1e-3
RTOL = 1e-3


def tol(a, b):
    return ATOL + RTOL * np.maximum(np.abs(a), np.abs(b))


def close(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return np.abs(a - b) <= tol(a, b)


def to_dev_bf16(bits: np.ndarray, device="cuda"):
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


@dataclass
class ParityReport:
    rows: int = 0
    tie_resolved_rows: int = 0
    tie_resolved_ids: int = 0
    max_logit_err: float = 0.0
    max_logprob_err: float = 0.0
    max_gate_err: float = 0.0
    errors: list = field(default_factory=list)

    @property
    def ok(self):
        return not self.errors


def compare(W, gm, Wg, hidden_bits, k_groups, k_tokens, gpu, forced_groups=None, max_errors=10, W1=None,
            factorised=False) -> ParityReport:
    """gpu: dict of numpy arrays from LMHead.draft(taps=True) ('groups','gate','logits','lse','ids','logprobs'),
    or just 'ids'/'logprobs' (taps missing are skipped).  forced_groups: the groups the caller forced, if any."""
    rep = ParityReport()
    M = hidden_bits.shape[0]
    rep.rows = M
    g_groups = gpu.get("groups")
    ref = orc.draft(W, gm, Wg, hidden_bits, k_groups, k_tokens, forced_groups=forced_groups, W1=W1,
                    factorised=factorised)
    forced = None
    if g_groups is not None:
        for m in range(M):
            if np.array_equal(g_groups[m], ref.groups[m]):
                continue
            gg = g_groups[m]
            ok = len(set(gg.tolist())) == k_groups and gg.min() >= 0 and gg.max() < Wg.shape[0]
            if ok:
                for s in range(k_groups):
                    if gg[s] != ref.groups[m, s] and not close(ref.gate[m, gg[s]], ref.gate[m, ref.groups[m, s]]):
                        ok = False
            if not ok:
                rep.errors.append(f"row {m}: groups {gg.tolist()} != oracle {ref.groups[m].tolist()}")
            else:
                rep.tie_resolved_rows += 1
                forced = g_groups
        if forced is not None and not rep.errors:
            ref = orc.draft(W, gm, Wg, hidden_bits, k_groups, k_tokens, forced_groups=np.ascontiguousarray(forced),
                            W1=W1, factorised=factorised)
    if rep.errors:
        return rep

    if gpu.get("gate") is not None:
        bad = ~close(gpu["gate"], ref.gate)
        rep.max_gate_err = float(np.abs(gpu["gate"] - ref.gate).max())
        if bad.any():
            rep.errors.append(f"gate mismatch at {np.argwhere(bad)[:3].tolist()}")
    if gpu.get("logits") is not None:
        bad = ~close(gpu["logits"], ref.logits)
        rep.max_logit_err = float(np.abs(gpu["logits"] - ref.logits).max())
        if bad.any():
            idx = np.argwhere(bad)[:3]
            rep.errors.append(f"logits mismatch at {idx.tolist()}: gpu {gpu['logits'][tuple(idx[0])]} "
                              f"oracle {ref.logits[tuple(idx[0])]}")
    if gpu.get("lse") is not None:
        bad = ~close(gpu["lse"], ref.lse)
        if bad.any():
            rep.errors.append(f"lse mismatch rows {np.flatnonzero(bad)[:5].tolist()}")

    ids, lps = gpu["ids"], gpu["logprobs"]
    for m in range(M):
        # the emitted log-probability of every active token: joint = z - LSE(row); factorised (Eq. 8) =
        # log p_router(group) + z - LSE(group)
        if factorised:
            score = ref.log_router[m, ref.groups[m]][:, None] + ref.logits[m] - ref.group_lse[m][:, None]
            if int(factorised) == 2:      # p_router renormalised over the row's selected groups
                sel_lr = ref.log_router[m, ref.groups[m]]
                score = score - (sel_lr.max() + np.log(np.exp(sel_lr - sel_lr.max()).sum()))
        else:
            score = ref.logits[m] - ref.lse[m]
        # score of a token id by binary search in the row's sorted active token list (all rows at full size
        # would cost a Python dictionary of 16 000 entries per row otherwise)
        tokens = ref.logit_tokens[m].ravel()
        order = np.argsort(tokens, kind="stable")
        tok_sorted, score_sorted = tokens[order], score.ravel()[order]

        def lookup(t):
            at = np.minimum(np.searchsorted(tok_sorted, t), tok_sorted.size - 1)
            return tok_sorted[at] == t, score_sorted[at]

        if len(set(ids[m].tolist())) != k_tokens:
            rep.errors.append(f"row {m}: duplicate ids {ids[m].tolist()}")
            continue
        active, got = lookup(ids[m].astype(np.int64))
        _, want_ref = lookup(ref.ids[m].astype(np.int64))
        if not active.all():
            i = int(np.flatnonzero(~active)[0])
            rep.errors.append(f"row {m} pos {i}: id {int(ids[m, i])} is not in an active group")
        else:
            differs = ids[m] != ref.ids[m]
            tie = differs & close(got, want_ref)
            wrong = differs & ~tie
            lp_bad = ~close(lps[m], got)
            rep.tie_resolved_ids += int(tie.sum())
            rep.max_logprob_err = max(rep.max_logprob_err, float(np.abs(lps[m] - got).max()))
            if wrong.any():
                i = int(np.flatnonzero(wrong)[0])
                rep.errors.append(f"row {m} pos {i}: id {int(ids[m, i])} (score={got[i]}) != oracle {int(ref.ids[m, i])} "
                                  f"(score={want_ref[i]})")
            elif lp_bad.any():
                i = int(np.flatnonzero(lp_bad)[0])
                rep.errors.append(f"row {m} pos {i}: logprob {float(lps[m, i])} != oracle {got[i]}")
        if np.any(np.diff(lps[m]) > 0):
            rep.errors.append(f"row {m}: log-probs not sorted descending")
        if len(rep.errors) >= max_errors:
            break
    return rep


def gpu_draft_numpy(head, hidden_bits, k_groups, k_tokens, taps=True, forced_groups=None):
    """Run the CUDA path through the binding and bring everything back as numpy."""
    h = to_dev_bf16(hidden_bits)
    fg = None if forced_groups is None else torch.from_numpy(np.ascontiguousarray(forced_groups, np.int32)).cuda()
    out = head.draft(h, k_groups, k_tokens, taps=True, forced_groups=fg) if taps else None
    if out is None:
        ids, lps = head.draft(h, k_groups, k_tokens)
        out = {"ids": ids, "logprobs": lps}
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}
