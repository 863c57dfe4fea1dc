"""GPU parity of the tree-expansion score step against its oracle (bit-exact: fp32 addition on both sides)."""
import numpy as np
import pytest
import torch

from oracle import tree_oracle as tor
from paper_2502_16880_b200 import lmhead

pytestmark = pytest.mark.gpu


def _run(ps, ids, lp, K):
    n_seq = ps.shape[0]
    d = lambda a, t: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to("cuda", t)
    parent = torch.empty((n_seq, K), dtype=torch.int32, device="cuda")
    token = torch.empty((n_seq, K), dtype=torch.int32, device="cuda")
    score = torch.empty((n_seq, K), dtype=torch.float32, device="cuda")
    lmhead.coral_tree_expand(d(ps, torch.float32), d(ids, torch.int32), d(lp, torch.float32), K, parent, token, score)
    torch.cuda.synchronize()
    return parent.cpu().numpy(), token.cpu().numpy(), score.cpu().numpy()


@pytest.mark.parametrize("n_seq,nodes,kt,K", [(1, 1, 10, 10), (16, 10, 10, 10), (3, 60, 10, 60), (2, 204, 10, 256), (5, 7, 3, 21)])
def test_expand_matches_oracle(n_seq, nodes, kt, K):
    rng = np.random.default_rng(nodes * 100 + kt)
    ps = -np.abs(rng.normal(size=(n_seq, nodes))).astype(np.float32)
    lp = -np.abs(rng.normal(size=(n_seq, nodes, kt))).astype(np.float32)
    lp[0, 0, :2] = lp[0, 0, 0]                                    # an exact tie
    ids = rng.integers(0, 128256, size=(n_seq, nodes, kt)).astype(np.int32)
    got = _run(ps, ids, lp, K)
    want = tor.expand(ps, ids, lp, K)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)


def test_rerank_mode_and_errors():
    rng = np.random.default_rng(1)
    ps = rng.normal(size=(4, 300)).astype(np.float32)
    got = _run(ps, None, None, 60)
    want = tor.expand(ps, None, None, 60)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    lib = lmhead.load_library()
    import ctypes
    t = torch.zeros((1, 4096), dtype=torch.float32, device="cuda")
    o = torch.zeros((1, 8), dtype=torch.int32, device="cuda")
    f = torch.zeros((1, 8), dtype=torch.float32, device="cuda")
    p = lambda x: ctypes.c_void_p(x.data_ptr())
    assert lib.coral_tree_expand(p(t), None, None, 1, 4096, 1, 8, p(o), p(o), p(f), None) == lmhead.CORAL_ERR_TOO_LARGE
    assert lib.coral_tree_expand(p(t), None, None, 1, 16, 1, 17, p(o), p(o), p(f), None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_tree_expand(None, None, None, 1, 16, 1, 8, p(o), p(o), p(f), None) == lmhead.CORAL_ERR_INVALID


def test_draft_then_expand_chain():
    """The consumer of the draft head: candidates of a level feed the expansion that picks the next parents."""
    from paper_2502_16880_b200 import synth
    from tests import parity_harness as ph
    cfg = synth.CONFIGS["tiny"]
    W, gm, Wg = synth.make_w_vocab(cfg), synth.make_group_map(cfg), synth.make_w_gate(cfg)
    head = lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg), 20, 4, 10)
    hb = synth.make_hidden(cfg, 20)                                  # 2 sequences x 10 nodes
    ids, lps = head.draft(ph.to_dev_bf16(hb), 4, 10)
    parent_scores = torch.zeros((2, 10), dtype=torch.float32, device="cuda")
    parent = torch.empty((2, 10), dtype=torch.int32, device="cuda")
    token = torch.empty((2, 10), dtype=torch.int32, device="cuda")
    score = torch.empty((2, 10), dtype=torch.float32, device="cuda")
    lmhead.coral_tree_expand(parent_scores, ids.view(2, 10, 10), lps.view(2, 10, 10), 10, parent, token, score)
    torch.cuda.synchronize()
    want = tor.expand(np.zeros((2, 10), np.float32), ids.cpu().numpy().reshape(2, 10, 10),
                      lps.cpu().numpy().reshape(2, 10, 10), 10)
    assert np.array_equal(parent.cpu().numpy(), want[0]) and np.array_equal(token.cpu().numpy(), want[1])
    assert np.array_equal(score.cpu().numpy(), want[2])
    head.close()
