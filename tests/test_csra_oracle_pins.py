"""Pins of the CSRA (InfoNCE, Eq. 2) oracle: closed forms, a library log-softmax, invariances, brute force."""
import math

import numpy as np
import pytest
from scipy.special import log_softmax

from oracle import csra_oracle as co
from paper_2502_16880_b200 import synth

TAU = 0.07


def _bits(x):
    return synth.fp32_to_bf16_bits(np.asarray(x, np.float32))


def _rand(n, D, seed):
    return _bits(np.random.default_rng(seed).standard_normal((n, D)))


def test_closed_form_orthonormal_features():
    """Keys = queries = distinct unit vectors: sim = 1 on the diagonal, 0 elsewhere, so every row's loss is
    log(e^{1/tau} + n - 1) - 1/tau, whatever positive scale the rows carry."""
    n, D = 6, 16
    E = np.zeros((n, D), np.float32)
    E[np.arange(n), np.arange(n) * 2] = [1.0, 2.0, 0.5, 4.0, 8.0, 0.25]
    r = co.infonce(_bits(E), _bits(3.0 * E), views=1, tau=TAU)
    want = math.log(math.exp(1 / TAU) + n - 1) - 1 / TAU
    assert np.allclose(r["row_loss"], want, rtol=0, atol=1e-12)
    assert abs(r["loss"] - want) < 1e-12


def test_closed_form_all_keys_parallel_to_the_query():
    """Every key is a positive multiple of every query: all similarities are equal, the loss is log(m)."""
    n, D, views = 5, 8, 3
    d = np.array([1, -2, 0.5, 4, -1, 2, 0.25, -8], np.float32)      # exactly representable, norm^2 = 90.3125
    Q = np.outer([1, 2, 4, 0.5, 8], d)
    K = np.outer(np.r_[[2, 1, 0.5, 4, 1] * views], d)
    r = co.infonce(_bits(Q), _bits(K), views=views, tau=TAU)
    assert np.allclose(r["row_loss"], math.log(n * views), atol=1e-9)
    assert np.allclose(r["logits"], r["logits"][0, 0])


def _positive_mask(n, views):
    mask = np.zeros((n, views * n), bool)
    for s in range(views):
        mask[np.arange(n), np.arange(n) + s * n] = True
    return mask


def test_against_library_norms_and_a_library_log_softmax():
    """The definition spelled with library routines only: numpy's vector norm, scipy's log-softmax, the positives
    picked with a boolean mask.  Nothing of the oracle is called on the expected side."""
    n, D, views = 24, 40, 2
    Q, K = _rand(n, D, 1), _rand(views * n, D, 2)
    r = co.infonce(Q, K, views, TAU)
    qf = synth.bf16_bits_to_fp32(Q).astype(np.float64)
    kf = synth.bf16_bits_to_fp32(K).astype(np.float64)
    qn = qf / np.linalg.norm(qf, axis=1, keepdims=True)
    kn = kf / np.linalg.norm(kf, axis=1, keepdims=True)
    assert np.allclose(co.normalise(Q), qn, rtol=0, atol=1e-15)
    assert np.allclose(np.linalg.norm(co.normalise(K), axis=1), 1.0, rtol=0, atol=1e-15)
    lp = log_softmax(qn @ kn.T / TAU, axis=1)
    want_rows = -(lp * _positive_mask(n, views)).sum(axis=1) / views
    assert np.allclose(r["row_loss"], want_rows, rtol=1e-12, atol=1e-12)
    assert abs(r["loss"] - want_rows.mean()) < 1e-12
    assert np.allclose(r["logits"], qn @ kn.T / TAU, rtol=0, atol=1e-12)


def test_brute_force_on_a_toy():
    """Pure-Python arithmetic from the widened inputs on: norms by math.sqrt of an exactly rounded sum of squares,
    dot products and sums by math.fsum.  Neither numpy nor the oracle's normalise is on the expected side."""
    n, D, views = 3, 5, 2
    Q, K = _rand(n, D, 3), _rand(views * n, D, 4)
    r = co.infonce(Q, K, views, TAU)

    def unit(bits_row):
        x = [float(v) for v in synth.bf16_bits_to_fp32(bits_row)]
        nrm = math.sqrt(math.fsum(v * v for v in x))
        return [v / nrm for v in x]

    qv = [unit(row) for row in Q]
    kv = [unit(row) for row in K]
    tot = 0.0
    for i in range(n):
        sims = [math.fsum(a * b for a, b in zip(qv[i], kv[j])) / TAU for j in range(views * n)]
        den = math.fsum(math.exp(s) for s in sims)
        li = -math.fsum(math.log(math.exp(sims[i + s * n]) / den) for s in range(views)) / views
        assert abs(li - r["row_loss"][i]) < 1e-10
        tot += li
    assert abs(tot / n - r["loss"]) < 1e-10


def test_bf16_rounding_helper_is_round_to_nearest_even():
    """round_to_bf16 (used only by the diagnostic variant) against a search over the two neighbouring bf16 values
    built from bit patterns, and on exact half-way points."""
    x = np.abs(np.random.default_rng(11).standard_normal(4000)) * 0.3 + 1e-3
    got = co.round_to_bf16(x)
    down_bits = (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)      # a bf16 at or just below/above x
    cands = np.stack([synth.bf16_bits_to_fp32((down_bits.astype(np.int64) + d).astype(np.uint16)).astype(np.float64) for d in (-1, 0, 1)])
    best = cands[np.abs(cands - x).argmin(axis=0), np.arange(x.size)]
    assert np.array_equal(got, best)
    # half-way between 1 and 1 + 2^-7 goes to the even neighbour 1; between 1 + 2^-7 and 1 + 2^-6 to 1 + 2^-6
    assert co.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert co.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_operand_rounding_moves_a_similarity_by_at_most_the_derived_bound():
    """bf16 keeps 8 significant bits (spacing 2^-7 relative): each unit-vector element moves by at most 2^-8
    relative, a product of two by at most 2^-7 + 2^-16, so a scaled similarity by at most
    (2^-7 + 2^-16) sum_d |q_d k_d| / tau.  The diagnostic
    variant must stay inside that bound of the definition (and does move: the rounding is really applied)."""
    n, D, views = 40, 96, 2
    Q, K = _rand(n, D, 21), _rand(views * n, D, 22)
    exact = co.infonce(Q, K, views, TAU)
    quant = co.infonce_bf16_operands(Q, K, views, TAU)
    bound = (2.0 ** -7 + 2.0 ** -16) * (np.abs(co.normalise(Q)) @ np.abs(co.normalise(K)).T) / TAU
    gap = np.abs(exact["logits"] - quant["logits"])
    assert np.all(gap <= bound + 1e-12)
    assert gap.max() > 1e-4
    assert np.abs(exact["row_loss"] - quant["row_loss"]).max() <= 2 * bound.max()


def test_invariances_scale_and_order_of_negatives():
    n, D, views = 10, 32, 2
    Qf = np.random.default_rng(5).standard_normal((n, D)).astype(np.float32)
    Kf = np.random.default_rng(6).standard_normal((views * n, D)).astype(np.float32)
    base = co.infonce(_bits(Qf), _bits(Kf), views, TAU)
    # powers of two commute with the bf16 rounding of the inputs: the cosine similarities are unchanged
    scaled = co.infonce(_bits(Qf * 4.0), _bits(Kf * 0.125), views, TAU)
    assert np.allclose(base["row_loss"], scaled["row_loss"], rtol=0, atol=1e-12)
    # a larger temperature flattens the distribution: the loss moves towards log(m)
    warm = co.infonce(_bits(Qf), _bits(Kf), views, 10.0)
    assert abs(warm["loss"] - math.log(views * n)) < abs(base["loss"] - math.log(views * n))
    assert abs(warm["loss"] - math.log(views * n)) < 0.05
    # swapping two positions everywhere (queries and every block of keys) permutes the row losses
    p = np.arange(n)
    p[[1, 7]] = p[[7, 1]]
    Kp = np.concatenate([Kf[s * n:(s + 1) * n][p] for s in range(views)])
    perm = co.infonce(_bits(Qf[p]), _bits(Kp), views, TAU)
    assert np.allclose(perm["row_loss"], base["row_loss"][p], rtol=0, atol=1e-12)
    # a planted mistake is caught: positives taken from the wrong block offset change the loss
    wrong = base["lse"] - np.stack([base["logits"][np.arange(n), (np.arange(n) + 1) % n + s * n]
                                    for s in range(views)], 1).mean(axis=1)
    assert np.abs(wrong - base["row_loss"]).max() > 1.0


def test_zero_feature_and_argument_check():
    Q = _bits(np.zeros((2, 8), np.float32))
    K = _rand(2, 8, 7)
    r = co.infonce(Q, K, 1, TAU)
    assert np.allclose(r["logits"], 0.0) and np.allclose(r["row_loss"], math.log(2))
    with pytest.raises(ValueError):
        co.infonce(Q, _rand(3, 8, 8), 1, TAU)
