"""The pins must be able to fail: plant one plausible mistake at a time in a
copy of the oracle's C source (on the CPU, in a temp directory), build it, and
check that a compact battery of the pins rejects every mutant while the
untouched source passes."""
import math
import os

import numpy as np
import pytest
from scipy.special import log_softmax, logsumexp

from oracle import lmhead_oracle as orc
from paper_2502_16880_b200 import synth

SRC = os.path.join(os.path.dirname(orc.__file__), "lmhead_oracle.c")

MUTANTS = {
    "dot_drops_last_term": ("for (int j = 0; j < H; ++j) a += bf16_value(w[j]) * h[j];",
                            "for (int j = 0; j < H - 1; ++j) a += bf16_value(w[j]) * h[j];"),
    "lse_sign": ("s += exp(z[i] - mx);", "s += exp(z[i] + mx);"),
    "tie_break_reversed": ("return (a->index > b->index) - (a->index < b->index);",
                           "return (a->index < b->index) - (a->index > b->index);"),
    "ascending_sort": ("if (a->score > b->score) return -1;\n    if (a->score < b->score) return 1;",
                       "if (a->score > b->score) return 1;\n    if (a->score < b->score) return -1;"),
    "gate_transposed": ("bf16_value(W_gate[(size_t)n * H + j]) * u[j]", "bf16_value(W_gate[(size_t)j * N + n]) * u[j]"),
    "joint_uses_group_lse": (": z[i] - lse;", ": z[i] - group_lse[s];"),
    "bf16_shift": ("(uint32_t)bits << 16", "(uint32_t)bits << 15"),
    "factorised_drops_router": ("factorised ? log_router[sel[s]] - log_selected_mass + (z[i] - group_lse[s])",
                                "factorised ? (z[i] - group_lse[s])"),
    "renormalised_mass_sign": ("factorised ? log_router[sel[s]] - log_selected_mass +",
                               "factorised ? log_router[sel[s]] + log_selected_mass +"),
    "renormalised_over_all_groups": ("z_sel[s] = log_router[sel[s]];", "z_sel[s] = log_router[s];"),
    "selects_lowest_groups": ("sel[s] = order[s].index;", "sel[s] = order[N - 1 - s].index;"),
    "always_row_zero": ("h[j] = bf16_value(hidden[(size_t)m * H + j]);", "h[j] = bf16_value(hidden[j]);"),
    "router_softmax_not_normalised": ("log_router[n] = g[n] - l;", "log_router[n] = g[n];"),
    "silu_without_residual": ("u[i] = a / (1.0 + exp(-a)) + h[i];", "u[i] = a / (1.0 + exp(-a));"),
    "slot_tokens_unsorted": ("tok[(long)s * v + fill[s]++] = x;", "tok[(long)s * v + (v - 1 - fill[s]++)] = x;"),
}


def _f64(bits):
    return synth.bf16_bits_to_fp32(bits).astype(np.float64)


def _battery(lib_path):
    """Names of the pins that fail for the oracle build at lib_path."""
    failed = []

    def check(name, fn):
        try:
            fn()
        except (AssertionError, ValueError):
            failed.append(name)

    cfg = synth.HeadConfig("toy", H=24, V=96, N=6, k_groups=2, k_tokens=9, M=3, seed=4, w_std=0.5)
    W, gm, Wg, h = synth.make_all(cfg)
    dense = _f64(h) @ _f64(W).T
    gate = _f64(h) @ _f64(Wg).T

    def p1():
        r = orc.draft(W, gm, Wg, h, cfg.N, 9, lib_path=lib_path)
        lp = log_softmax(dense, axis=1)
        for m in range(cfg.M):
            order = np.lexsort((np.arange(cfg.V), -dense[m]))[:9]
            assert np.array_equal(r.ids[m], order)
            np.testing.assert_allclose(r.logprobs[m], lp[m, order], atol=1e-11)

    def p3():
        r = orc.draft(W, gm, Wg, h, 2, 9, lib_path=lib_path)
        for m in range(cfg.M):
            groups = sorted(range(cfg.N), key=lambda n: (-gate[m, n], n))[:2]
            assert r.groups[m].tolist() == groups
            act = [x for x in range(cfg.V) if gm[x] in groups]
            lse = logsumexp(dense[m, act])
            top = sorted(act, key=lambda x: (-dense[m, x], x))[:9]
            assert r.ids[m].tolist() == top
            np.testing.assert_allclose(r.logprobs[m], dense[m, top] - lse, atol=1e-11)
            for s in range(2):
                assert np.all(np.diff(r.logit_tokens[m, s]) > 0)

    def p4():
        Z = np.zeros_like(W)
        r = orc.draft(Z, gm, np.zeros_like(Wg), h, 2, 5, lib_path=lib_path)
        assert r.groups.tolist() == [[0, 1]] * cfg.M
        assert r.ids.tolist() == [np.flatnonzero(gm < 2)[:5].tolist()] * cfg.M
        np.testing.assert_allclose(r.logprobs, -math.log(2 * cfg.v), atol=1e-14)

    def p6():
        ideal = np.stack([[logsumexp(dense[m, gm == n]) for n in range(cfg.N)] for m in range(cfg.M)])
        r = orc.draft(W, gm, Wg, h, cfg.N, 9, gate_override=ideal, factorised=True, lib_path=lib_path)
        lp = log_softmax(dense, axis=1)
        for m in range(cfg.M):
            order = np.lexsort((np.arange(cfg.V), -dense[m]))[:9]
            assert np.array_equal(r.ids[m], order)
            np.testing.assert_allclose(r.logprobs[m], lp[m, order], atol=1e-11)

    def p6r():
        # renormalised variant: the probabilities of the active vocabulary sum to 1 and keep Eq. 8's order
        r1 = orc.draft(W, gm, Wg, h, 2, 9, factorised=1, lib_path=lib_path)
        r2 = orc.draft(W, gm, Wg, h, 2, 9, factorised=2, lib_path=lib_path)
        assert np.array_equal(r1.ids, r2.ids)
        mass = np.exp(r2.log_router[np.arange(cfg.M)[:, None], r2.groups]).sum(axis=1)
        np.testing.assert_allclose(r2.logprobs, r1.logprobs - np.log(mass)[:, None], atol=1e-12)

    def p10():
        W1 = synth._normal_bf16(np.random.default_rng(5), cfg.H, cfg.H, 0.2)
        r = orc.draft(W, gm, Wg, h, 2, 5, W1=W1, want_logits=False, lib_path=lib_path)
        a = _f64(h) @ _f64(W1).T
        g = (a / (1.0 + np.exp(-a)) + _f64(h)) @ _f64(Wg).T
        np.testing.assert_allclose(r.gate, g, atol=1e-12)

    for name, fn in [("p1", p1), ("p3", p3), ("p4", p4), ("p6", p6), ("p6r", p6r), ("p10", p10)]:
        check(name, fn)
    return failed


def test_unmodified_oracle_passes_battery(tmp_path):
    out = str(tmp_path / "liboracle_ref.so")
    orc.build(force=True, src=SRC, out=out)
    assert _battery(out) == []


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, tmp_path):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation site for {name} not found"
    src = tmp_path / f"mut_{name}.c"
    src.write_text(text.replace(old, new))
    out = str(tmp_path / f"libmut_{name}.so")
    orc.build(force=True, src=str(src), out=out)
    assert _battery(out), f"mutant {name} passed every pin"
