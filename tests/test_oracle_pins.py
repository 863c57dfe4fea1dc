"""Pins for the CPU oracle: checks against things the paper and the mathematics
fix, none of which re-use the oracle's own code.

P1  all groups active == dense LM head (numpy matmul + scipy log_softmax)
P2  probabilities over the active vocabulary sum to 1 (Section 3.3)
P3  brute force in pure Python on toy sizes (different language, dense-then-mask)
P4  closed forms: zero weights, one-hot hidden states with integer weights
P5  monotonicity in the number of active groups
P6  ideal-router identity: Eq. 8 with q_router(n) = sum of the group's target
    probabilities reproduces the dense softmax (Section 3.3)
P7  relabelling groups / permuting token ids
P8  contiguous grouping vs an arbitrary map with permuted weights
P9  the paper's "1002M memory access" for the Llama3-8B head (Appendix B) and
    the 2 x 10 = 20 worst-case union (Appendix B, tree decoding)
P10 Eq. 7's router argument W2(act(W1 h) + h) against numpy
"""
import math

import numpy as np
import pytest
from scipy.special import log_softmax, logsumexp

from oracle import lmhead_oracle as orc
from paper_2502_16880_b200 import synth

TINY = synth.CONFIGS["tiny"]


def _f64(bits):
    return synth.bf16_bits_to_fp32(bits).astype(np.float64)


def _toy(H, V, N, M, seed, std=0.5):
    cfg = synth.HeadConfig("toy", H=H, V=V, N=N, k_groups=1, k_tokens=1, M=M, seed=seed, w_std=std)
    return cfg, synth.make_all(cfg)


def _stable_desc(scores):
    # descending score, ascending index among equals
    return np.lexsort((np.arange(scores.size), -scores))


# ---------------------------------------------------------------- P1
@pytest.mark.parametrize("cfg", [TINY, TINY.with_(seed=3, M=7, k_tokens=25)])
def test_p1_all_groups_equals_dense_head(cfg):
    W, gm, Wg, h = synth.make_all(cfg)
    r = orc.draft(W, gm, Wg, h, cfg.N, cfg.k_tokens)
    dense = _f64(h) @ _f64(W).T                      # [M, V] library matmul
    lp = log_softmax(dense, axis=1)
    for m in range(cfg.M):
        order = _stable_desc(dense[m])[: cfg.k_tokens]
        assert np.array_equal(r.ids[m], order)
        np.testing.assert_allclose(r.logprobs[m], lp[m, order], rtol=0, atol=1e-11)
        np.testing.assert_allclose(r.lse[m], logsumexp(dense[m]), rtol=0, atol=1e-11)
        # every token appears exactly once in the slot layout
        assert np.array_equal(np.sort(r.logit_tokens[m].ravel()), np.arange(cfg.V))
        np.testing.assert_allclose(r.logits[m].ravel(), dense[m, r.logit_tokens[m].ravel()], atol=1e-12)


def test_p1_dense_equivalence_non_power_of_two_shape():
    # group size 1000-like raggedness at small scale: v = 75, H = 72
    cfg, (W, gm, Wg, h) = _toy(H=72, V=600, N=8, M=5, seed=11, std=0.2)
    r = orc.draft(W, gm, Wg, h, 8, 12)
    dense = _f64(h) @ _f64(W).T
    lp = log_softmax(dense, axis=1)
    for m in range(5):
        order = _stable_desc(dense[m])[:12]
        assert np.array_equal(r.ids[m], order)
        np.testing.assert_allclose(r.logprobs[m], lp[m, order], atol=1e-12)


# ---------------------------------------------------------------- P2
@pytest.mark.parametrize("k", [1, 4, 16])
def test_p2_active_probabilities_sum_to_one(k):
    W, gm, Wg, h = synth.make_all(TINY)
    r = orc.draft(W, gm, Wg, h, k, 10)
    p = np.exp(r.logits - r.lse[:, None, None])
    np.testing.assert_allclose(p.sum(axis=(1, 2)), 1.0, rtol=0, atol=1e-12)
    # and the emitted log-probs are those of the emitted ids
    for m in range(TINY.M):
        flat_tok = r.logit_tokens[m].ravel()
        pos = {int(t): i for i, t in enumerate(flat_tok)}
        z = np.array([r.logits[m].ravel()[pos[int(t)]] for t in r.ids[m]])
        np.testing.assert_allclose(r.logprobs[m], z - r.lse[m], atol=1e-13)


# ---------------------------------------------------------------- P3
def _brute_row(Wf, gm, Wgf, hf, N, k_groups, k_tokens):
    """Pure-Python definition: dense scores for everything, then mask."""
    H = len(hf)
    gate = [math.fsum(Wgf[n][j] * hf[j] for j in range(H)) for n in range(N)]
    groups = sorted(range(N), key=lambda n: (-gate[n], n))[:k_groups]
    dense = [math.fsum(Wf[x][j] * hf[j] for j in range(H)) for x in range(len(Wf))]
    active = [x for x in range(len(Wf)) if gm[x] in groups]
    mx = max(dense[x] for x in active)
    lse = mx + math.log(math.fsum(math.exp(dense[x] - mx) for x in active))
    top = sorted(active, key=lambda x: (-dense[x], x))[:k_tokens]
    return gate, groups, lse, top, [dense[x] - lse for x in top]


@pytest.mark.parametrize("H,V,N,kg,kt,seed", [
    (4, 8, 2, 1, 3, 0), (4, 8, 4, 2, 4, 1), (8, 24, 3, 2, 16, 2), (16, 60, 6, 5, 7, 3), (5, 12, 4, 4, 12, 4)])
def test_p3_brute_force_on_toys(H, V, N, kg, kt, seed):
    cfg, (W, gm, Wg, h) = _toy(H, V, N, M=3, seed=seed)
    r = orc.draft(W, gm, Wg, h, kg, kt)
    Wf, Wgf, hf = _f64(W).tolist(), _f64(Wg).tolist(), _f64(h).tolist()
    for m in range(3):
        gate, groups, lse, top, lps = _brute_row(Wf, gm.tolist(), Wgf, hf[m], N, kg, kt)
        np.testing.assert_allclose(r.gate[m], gate, atol=1e-13)
        assert r.groups[m].tolist() == groups
        assert r.ids[m].tolist() == top
        np.testing.assert_allclose(r.lse[m], lse, atol=1e-13)
        np.testing.assert_allclose(r.logprobs[m], lps, atol=1e-13)


def test_p3_brute_force_on_tiny_config_row0():
    W, gm, Wg, h = synth.make_all(TINY)
    r = orc.draft(W, gm, Wg, h, TINY.k_groups, TINY.k_tokens)
    gate, groups, lse, top, lps = _brute_row(_f64(W).tolist(), gm.tolist(), _f64(Wg).tolist(),
                                             _f64(h)[0].tolist(), TINY.N, TINY.k_groups, TINY.k_tokens)
    assert r.groups[0].tolist() == groups and r.ids[0].tolist() == top
    np.testing.assert_allclose(r.logprobs[0], lps, atol=1e-12)


# ---------------------------------------------------------------- P4
def test_p4_zero_weights_closed_form():
    H, V, N, M, kg, kt = 8, 40, 5, 2, 2, 6
    W = np.zeros((V, H), np.uint16)
    Wg = np.zeros((N, H), np.uint16)
    gm = synth.make_group_map(synth.HeadConfig("z", H, V, N, kg, kt, M, seed=5))
    h = synth.make_hidden(synth.HeadConfig("z", H, V, N, kg, kt, M, seed=5))
    r = orc.draft(W, gm, Wg, h, kg, kt)
    # all gate scores tie -> groups 0..kg-1; all logits tie -> smallest ids
    assert r.groups.tolist() == [[0, 1]] * M
    active = np.flatnonzero(gm < kg)
    assert r.ids.tolist() == [active[:kt].tolist()] * M
    np.testing.assert_allclose(r.logprobs, -math.log(kg * (V // N)), atol=1e-15)
    np.testing.assert_allclose(r.lse, math.log(kg * (V // N)), atol=1e-15)


def test_p4_one_hot_hidden_integer_weights():
    # h = e_c (bf16 1.0 = 0x3F80): z[x] = W[x, c], gate[n] = Wg[n, c]: known integers
    H, V, N = 4, 12, 3
    one = np.uint16(0x3F80)
    ints = lambda a: synth.fp32_to_bf16_bits(np.asarray(a, np.float32))
    Wv = np.arange(V * H, dtype=np.float32).reshape(V, H) % 7 - 3       # small integers
    Wgv = np.array([[1, 5, 2, 0], [3, 4, 9, 0], [2, 6, 1, 0]], np.float32)
    gm = np.array([0, 1, 2] * 4, np.int32)
    for c in range(3):
        h = np.zeros((1, H), np.uint16)
        h[0, c] = one
        r = orc.draft(ints(Wv), gm, ints(Wgv), h, 2, 3)
        np.testing.assert_array_equal(r.gate[0], Wgv[:, c])
        exp_groups = sorted(range(N), key=lambda n: (-Wgv[n, c], n))[:2]
        assert r.groups[0].tolist() == exp_groups
        act = [x for x in range(V) if gm[x] in exp_groups]
        zs = {x: float(Wv[x, c]) for x in act}
        lse = math.log(sum(math.exp(z) for z in zs.values()))
        top = sorted(act, key=lambda x: (-zs[x], x))[:3]
        assert r.ids[0].tolist() == top
        np.testing.assert_allclose(r.logprobs[0], [zs[x] - lse for x in top], atol=1e-14)


def test_p4_transposed_or_shifted_operands_would_fail():
    # W[x, j] = 1 only at (x=3, j=1): with h = e_1 exactly token 3 scores 1
    H, V, N = 4, 8, 2
    W = np.zeros((V, H), np.uint16)
    W[3, 1] = 0x3F80
    h = np.zeros((1, H), np.uint16)
    h[0, 1] = 0x3F80
    Wg = np.zeros((N, H), np.uint16)
    Wg[1, 1] = 0x3F80                        # group 1 wins for e_1
    gm = np.array([0, 0, 0, 1, 1, 1, 1, 0], np.int32)
    r = orc.draft(W, gm, Wg, h, 1, 2)
    assert r.groups[0].tolist() == [1]
    assert r.ids[0].tolist() == [3, 4]
    lse = math.log(math.e + 3.0)
    np.testing.assert_allclose(r.logprobs[0], [1 - lse, -lse], atol=1e-15)


# ---------------------------------------------------------------- P5
def test_p5_monotone_in_number_of_groups():
    W, gm, Wg, h = synth.make_all(TINY)
    prev = None
    for k in range(1, TINY.N + 1):
        r = orc.draft(W, gm, Wg, h, k, 5, want_logits=False)
        if prev is not None:
            assert np.array_equal(prev.groups, r.groups[:, : k - 1])      # nested selections
            assert np.all(r.lse >= prev.lse)
            for m in range(TINY.M):                                        # a kept token can only lose mass
                common = set(prev.ids[m]) & set(r.ids[m])
                for t in common:
                    a = prev.logprobs[m][list(prev.ids[m]).index(t)]
                    b = r.logprobs[m][list(r.ids[m]).index(t)]
                    assert b <= a + 1e-15
        prev = r


# ---------------------------------------------------------------- P6
def test_p6_ideal_router_reproduces_dense_softmax():
    cfg = TINY.with_(M=3)
    W, gm, Wg, h = synth.make_all(cfg)
    dense = _f64(h) @ _f64(W).T
    lp_dense = log_softmax(dense, axis=1)
    # q_router(n) = sum of dense probabilities in group n  <=>  score = per-group LSE
    ideal = np.stack([[logsumexp(dense[m, gm == n]) for n in range(cfg.N)] for m in range(cfg.M)])
    r = orc.draft(W, gm, Wg, h, cfg.N, 20, gate_override=ideal, factorised=True)
    for m in range(cfg.M):
        order = _stable_desc(dense[m])[:20]
        assert np.array_equal(r.ids[m], order)
        np.testing.assert_allclose(r.logprobs[m], lp_dense[m, order], atol=1e-11)
    # Section 3.3: p_router and each p_group are normalised, so p(x) is too
    fact = r.log_router[np.arange(cfg.M)[:, None], r.groups][:, :, None] + r.logits - r.group_lse[:, :, None]
    np.testing.assert_allclose(np.exp(fact).sum(axis=(1, 2)), 1.0, atol=1e-12)
    np.testing.assert_allclose(np.exp(r.log_router).sum(axis=1), 1.0, atol=1e-12)


def test_p6_factorised_partial_selection_mass_is_router_mass():
    W, gm, Wg, h = synth.make_all(TINY)
    r = orc.draft(W, gm, Wg, h, 4, 10, factorised=True)
    fact = r.log_router[np.arange(TINY.M)[:, None], r.groups][:, :, None] + r.logits - r.group_lse[:, :, None]
    sel_mass = np.exp(r.log_router[np.arange(TINY.M)[:, None], r.groups]).sum(axis=1)
    np.testing.assert_allclose(np.exp(fact).sum(axis=(1, 2)), sel_mass, atol=1e-12)
    # ranking is by the factorised log-probability
    for m in range(TINY.M):
        flat = fact[m].ravel()
        order = np.lexsort((r.logit_tokens[m].ravel(), -flat))[:10]
        assert np.array_equal(r.ids[m], r.logit_tokens[m].ravel()[order])
        np.testing.assert_allclose(r.logprobs[m], flat[order], atol=1e-13)


def test_p6_renormalised_router_mass_is_one_over_the_active_vocabulary():
    """Eq. 8 with p_router renormalised over the selected groups (the paper is silent on this): the active
    vocabulary then carries probability 1, every log-probability moves by the same per-row constant
    -log(selected router mass), so ids are those of Eq. 8; with every group selected it is Eq. 8 itself."""
    W, gm, Wg, h = synth.make_all(TINY)
    r1 = orc.draft(W, gm, Wg, h, 4, 10, factorised=1)
    r2 = orc.draft(W, gm, Wg, h, 4, 10, factorised=2)
    rows = np.arange(TINY.M)[:, None]
    sel_lr = r2.log_router[rows, r2.groups]
    renorm = sel_lr - logsumexp(sel_lr, axis=1)[:, None]                 # log of p_router / selected mass
    full = renorm[:, :, None] + r2.logits - r2.group_lse[:, :, None]
    np.testing.assert_allclose(np.exp(full).sum(axis=(1, 2)), 1.0, atol=1e-12)
    assert np.array_equal(r1.ids, r2.ids)
    np.testing.assert_allclose(r2.logprobs, r1.logprobs - logsumexp(sel_lr, axis=1)[:, None], atol=1e-12)
    for m in range(TINY.M):
        flat = full[m].ravel()
        order = np.lexsort((r2.logit_tokens[m].ravel(), -flat))[:10]
        np.testing.assert_allclose(r2.logprobs[m], flat[order], atol=1e-13)
    ra = orc.draft(W, gm, Wg, h, TINY.N, 10, factorised=1)
    rb = orc.draft(W, gm, Wg, h, TINY.N, 10, factorised=2)
    assert np.array_equal(ra.ids, rb.ids)
    np.testing.assert_allclose(ra.logprobs, rb.logprobs, atol=1e-12)


# ---------------------------------------------------------------- P7
def test_p7_group_relabelling_invariance():
    W, gm, Wg, h = synth.make_all(TINY)
    base = orc.draft(W, gm, Wg, h, 4, 10)
    sigma = np.random.default_rng(7).permutation(TINY.N)     # new label of old group n
    gm2 = sigma[gm].astype(np.int32)
    Wg2 = np.empty_like(Wg)
    Wg2[sigma] = Wg
    r = orc.draft(W, gm2, Wg2, h, 4, 10)
    assert np.array_equal(r.groups, sigma[base.groups])
    assert np.array_equal(r.ids, base.ids)
    np.testing.assert_allclose(r.logprobs, base.logprobs, atol=1e-13)


def test_p7_token_permutation_maps_ids():
    W, gm, Wg, h = synth.make_all(TINY)
    base = orc.draft(W, gm, Wg, h, 4, 10)
    pi = np.random.default_rng(8).permutation(TINY.V)        # old token x becomes pi[x]
    W2 = np.empty_like(W)
    W2[pi] = W
    gm2 = np.empty_like(gm)
    gm2[pi] = gm
    r = orc.draft(W2, gm2, Wg, h, 4, 10)
    assert np.array_equal(r.groups, base.groups)
    assert np.array_equal(r.ids, pi[base.ids])               # no exact ties in this seed
    np.testing.assert_allclose(r.logprobs, base.logprobs, atol=1e-12)


# ---------------------------------------------------------------- P8
def test_p8_contiguous_grouping_equals_permuted_random_map():
    W, gm, Wg, h = synth.make_all(TINY)
    base = orc.draft(W, gm, Wg, h, 4, 10)
    order = np.argsort(gm, kind="stable")                    # tokens of group 0, then 1, ...
    Wc = W[order]                                            # new id i holds old token order[i]
    gmc = synth.make_group_map(TINY, contiguous=True)
    r = orc.draft(Wc, gmc, Wg, h, 4, 10)
    assert np.array_equal(r.groups, base.groups)
    assert np.array_equal(order[r.ids], base.ids)
    np.testing.assert_allclose(r.logprobs, base.logprobs, atol=1e-12)
    assert np.array_equal(order[r.logit_tokens], base.logit_tokens)


# ---------------------------------------------------------------- P9
def test_p9_paper_byte_count_and_union_bound():
    llama3 = synth.CONFIGS["llama3_8b"]
    head_bytes = llama3.V * llama3.H * 2
    assert head_bytes == 1_050_673_152
    assert head_bytes / 2 ** 20 == pytest.approx(1002, abs=0.5)         # "1002M memory access"
    assert round(head_bytes / (768 * 2 ** 30) * 1e3, 1) == 1.3       # its "theoretical time of 1.3ms" at 768 GB/s
    # union of selected groups over rows: |U| <= min(N, M * k)
    cfg = TINY.with_(M=10)
    W, gm, Wg, h = synth.make_all(cfg)
    r = orc.draft(W, gm, Wg, h, 2, 10, want_logits=False)
    assert len(set(r.groups.ravel().tolist())) <= min(cfg.N, 2 * 10) == 16
    assert 2 * 10 == 20 and 20 < 32                                     # 32 groups are never all active


# ---------------------------------------------------------------- P10
def test_p10_two_layer_router_argument():
    cfg = TINY.with_(M=3, seed=2)
    W, gm, Wg, h = synth.make_all(cfg)
    W1 = synth._normal_bf16(np.random.default_rng(99), cfg.H, cfg.H, 0.05)
    r = orc.draft(W, gm, Wg, h, 4, 10, W1=W1, want_logits=False)
    hf = _f64(h)
    a = hf @ _f64(W1).T
    u = a / (1.0 + np.exp(-a)) + hf
    g = u @ _f64(Wg).T
    np.testing.assert_allclose(r.gate, g, atol=1e-12)
    np.testing.assert_allclose(r.log_router, log_softmax(g, axis=1), atol=1e-12)
    for m in range(cfg.M):
        assert r.groups[m].tolist() == _stable_desc(g[m])[:4].tolist()


# ---------------------------------------------------------------- argument checks, forced groups
def test_forced_groups_and_errors():
    W, gm, Wg, h = synth.make_all(TINY)
    forced = np.tile(np.array([5, 1, 9], np.int32), (TINY.M, 1))
    r = orc.draft(W, gm, Wg, h, 3, 10, forced_groups=forced)
    assert np.array_equal(r.groups, forced)
    for m in range(TINY.M):
        assert set(gm[r.logit_tokens[m, 1]]) == {1}
        assert np.all(np.diff(r.logit_tokens[m, 1]) > 0)
    with pytest.raises(ValueError):
        orc.draft(W, gm, Wg, h, TINY.N + 1, 10)
    with pytest.raises(ValueError):
        orc.draft(W, gm, Wg, h, 1, TINY.v + 1)
    bad = gm.copy()
    bad[0] = (bad[0] + 1) % TINY.N                    # unequal groups
    with pytest.raises(ValueError):
        orc.draft(W, bad, Wg, h, 2, 10)
