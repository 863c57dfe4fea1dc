"""Pins for the tree-expansion oracle: closed forms, brute force with a different algorithm, invariants."""
import itertools

import numpy as np
import pytest

from oracle import tree_oracle as tor


def test_closed_form_small_example():
    # two nodes with cumulative scores 0 and -1; candidates -0.1/-2 and -0.5/-0.6
    ps = np.array([[0.0, -1.0]], np.float32)
    lp = np.array([[[-0.1, -2.0], [-0.5, -0.6]]], np.float32)
    ids = np.array([[[11, 12], [21, 22]]], np.int32)
    parent, token, score = tor.expand(ps, ids, lp, 3)
    # children: (0,11) -0.1, (0,12) -2.0, (1,21) -1.5, (1,22) -1.6
    assert parent.tolist() == [[0, 1, 1]] and token.tolist() == [[11, 21, 22]]
    np.testing.assert_array_equal(score, np.array([[-0.1, -1.5, -1.6]], np.float32))


def test_ties_take_the_lower_flat_index():
    ps = np.zeros((1, 3), np.float32)
    lp = np.zeros((1, 3, 2), np.float32)
    parent, token, _ = tor.expand(ps, None, lp, 4)
    assert parent.tolist() == [[0, 0, 1, 1]] and token.tolist() == [[0, 1, 2, 3]]


def test_brute_force_by_exhaustive_subsets():
    # the K kept children maximise the sum of scores over all K-subsets (no ties in this draw)
    rng = np.random.default_rng(3)
    ps = rng.normal(size=(2, 3)).astype(np.float32)
    lp = -np.abs(rng.normal(size=(2, 3, 3))).astype(np.float32)
    parent, token, score = tor.expand(ps, None, lp, 4)
    for s in range(2):
        child = (ps[s][:, None] + lp[s]).astype(np.float32).ravel()
        best = max(itertools.combinations(range(9), 4), key=lambda c: sum(float(child[i]) for i in c))
        assert sorted(token[s].tolist()) == sorted(best)
        assert np.all(np.diff(score[s]) <= 0)
        assert np.array_equal(parent[s], token[s] // 3)


def test_invariants():
    rng = np.random.default_rng(5)
    ps = -np.abs(rng.normal(size=(3, 10))).astype(np.float32)
    lp = -np.abs(rng.normal(size=(3, 10, 10))).astype(np.float32)
    p_all, t_all, s_all = tor.expand(ps, None, lp, 100)
    assert all(sorted(t_all[s].tolist()) == list(range(100)) for s in range(3))      # K = all: a permutation
    p10, t10, s10 = tor.expand(ps, None, lp, 10)
    assert np.array_equal(t10, t_all[:, :10]) and np.array_equal(s10, s_all[:, :10])  # prefix property
    assert np.all(s10 <= ps[np.arange(3)[:, None], p10])                              # log-probs <= 0 only lower the score
    # re-ranking mode: no candidates, the nodes themselves
    p, t, s = tor.expand(ps, None, None, 4)
    for q in range(3):
        assert p[q].tolist() == np.lexsort((np.arange(10), -ps[q]))[:4].tolist()
    with pytest.raises(ValueError):
        tor.expand(ps, None, lp, 101)
