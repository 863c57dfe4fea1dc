"""GPU parity: the CUDA path through the C ABI against the CPU oracle."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2502_16880_b200 import lmhead, synth
from tests import parity_harness as ph

pytestmark = pytest.mark.gpu

PATHS = [lmhead.CORAL_PATH_STREAM, lmhead.CORAL_PATH_SIMT_PLAIN]


def _supported(path, M, H=256):
    return path != lmhead.CORAL_PATH_STREAM or (M <= 128 and H % 256 == 0 and H <= 4096)



def _head(cfg, W, gm, Wg, max_M=None, max_kg=None, max_kt=None):
    return lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg),
                         max_M or cfg.M, max_kg or cfg.N, max_kt or 32)


_cache = {}


def _weights(name):
    """Weights are expensive to draw at the Llama3/Qwen shapes: one set per config per session."""
    if name not in _cache:
        _cache.clear()
        cfg = synth.CONFIGS[name]
        W, gm, Wg = synth.make_w_vocab(cfg), synth.make_group_map(cfg), synth.make_w_gate(cfg)
        _cache[name] = (cfg, W, gm, Wg, _head(cfg, W, gm, Wg, max_M=max(cfg.M, 128)))
    return _cache[name]


def _check(head, W, gm, Wg, hb, kg, kt, path, forced=None):
    if not _supported(path, hb.shape[0], hb.shape[1]):
        pytest.skip("streaming path takes M <= 128 and H a multiple of 256")
    head.set_path(path)
    out = ph.gpu_draft_numpy(head, hb, kg, kt, forced_groups=forced)
    assert head.status() == 0
    rep = ph.compare(W, gm, Wg, hb, kg, kt, out, forced_groups=forced)
    assert rep.ok, rep.errors
    return rep, out


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("M,kg,kt", [(4, 4, 10), (1, 1, 1), (1, 4, 10), (3, 16, 32), (16, 2, 10), (40, 16, 7),
                                     (128, 3, 10), (9, 16, 10), (17, 16, 5)])
def test_tiny(path, M, kg, kt):
    cfg, W, gm, Wg, head = _weights("tiny")
    hb = synth.make_hidden(cfg, M)
    rep, out = _check(head, W, gm, Wg, hb, kg, kt, path)
    st = head.stats()
    assert st.groups_touched == len(set(out["groups"].ravel().tolist()))
    assert st.weight_bytes == st.groups_touched * cfg.v * cfg.H * 2


@pytest.mark.parametrize("path", PATHS)
def test_ragged_shape(path):
    # v = 300 (two full tiles + a tail of 44), H = 328 (not a multiple of 256)
    # v = 300 is 18 items of 16 rows + a tail of 12; H = 328 only runs on the plain path, H = 768 on both
    H = 328 if path == lmhead.CORAL_PATH_SIMT_PLAIN else 768
    cfg = synth.HeadConfig("ragged", H=H, V=1800, N=6, k_groups=3, k_tokens=10, M=13, seed=5, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg)
    for kg, kt in [(3, 10), (6, 32), (1, 5)]:
        _check(head, W, gm, Wg, hb, kg, kt, path)
    head.close()


@pytest.mark.parametrize("path", PATHS)
def test_small_group_fewer_rows_than_k_tokens(path):
    # v = 6 < k_tokens: per-tile candidate lists are padded
    cfg = synth.HeadConfig("small_v", H=256, V=48, N=8, k_groups=4, k_tokens=20, M=5, seed=9, w_std=0.3)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg)
    _check(head, W, gm, Wg, hb, 4, 20, path)
    _check(head, W, gm, Wg, hb, 8, 32, path)
    head.close()


@pytest.mark.parametrize("path", PATHS)
def test_forced_groups(path):
    cfg, W, gm, Wg, head = _weights("tiny")
    hb = synth.make_hidden(cfg, 5)
    forced = np.tile(np.array([7, 0, 15], np.int32), (5, 1))
    rep, out = _check(head, W, gm, Wg, hb, 3, 10, path, forced=forced)
    assert np.array_equal(out["groups"], forced)


@pytest.mark.parametrize("path", PATHS)
def test_exact_ties_zero_weights(path):
    cfg = synth.HeadConfig("zeros", H=256, V=640, N=5, k_groups=2, k_tokens=10, M=3, seed=1)
    gm, hb = synth.make_group_map(cfg), synth.make_hidden(cfg)
    W = np.zeros((cfg.V, cfg.H), np.uint16)
    Wg = np.zeros((cfg.N, cfg.H), np.uint16)
    head = _head(cfg, W, gm, Wg)
    head.set_path(path)
    out = ph.gpu_draft_numpy(head, hb, 2, 10)
    assert out["groups"].tolist() == [[0, 1]] * cfg.M                 # equal scores -> lower index
    assert out["ids"].tolist() == [np.flatnonzero(gm < 2)[:10].tolist()] * cfg.M   # equal logits -> lower id
    np.testing.assert_allclose(out["logprobs"], -np.log(2 * cfg.v), atol=1e-5)
    head.close()


@pytest.mark.parametrize("path", PATHS)
def test_deterministic_bitwise(path):
    cfg, W, gm, Wg, head = _weights("tiny")
    hb = synth.make_hidden(cfg, 33)
    head.set_path(path)
    a = ph.gpu_draft_numpy(head, hb, 4, 10)
    b = ph.gpu_draft_numpy(head, hb, 4, 10)
    for k in a:
        assert np.array_equal(a[k], b[k]), k


def test_argument_errors_return_codes():
    cfg, W, gm, Wg, head = _weights("tiny")
    h = ph.to_dev_bf16(synth.make_hidden(cfg, 4))
    ids = torch.empty((4, 10), dtype=torch.int32, device="cuda")
    lps = torch.empty((4, 10), dtype=torch.float32, device="cuda")
    lib = lmhead.load_library()
    import ctypes
    hp, ip, lp = (ctypes.c_void_p(t.data_ptr()) for t in (h, ids, lps))
    assert lib.coral_lmhead_draft(head.handle, hp, 0, 4, 10, ip, lp, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_draft(head.handle, hp, 10 ** 6, 4, 10, ip, lp, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_draft(head.handle, hp, 4, 0, 10, ip, lp, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_draft(head.handle, hp, 4, cfg.N + 1, 10, ip, lp, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_draft(head.handle, hp, 4, 4, 33, ip, lp, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_draft(head.handle, None, 4, 4, 10, ip, lp, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_draft(head.handle, hp, 4, 4, 10, None, lp, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_draft(None, hp, 4, 4, 10, ip, lp, None) == lmhead.CORAL_ERR_INVALID
    # a forced path that cannot take the call is refused, not silently replaced
    big = lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg), 200, 4, 10)
    h200 = ph.to_dev_bf16(synth.make_hidden(cfg, 200))
    i200 = torch.empty((200, 10), dtype=torch.int32, device="cuda")
    l200 = torch.empty((200, 10), dtype=torch.float32, device="cuda")
    big.set_path(lmhead.CORAL_PATH_STREAM)
    assert lib.coral_lmhead_draft(big.handle, ctypes.c_void_p(h200.data_ptr()), 200, 4, 10,
                                  ctypes.c_void_p(i200.data_ptr()), ctypes.c_void_p(l200.data_ptr()), None) == \
        lmhead.CORAL_ERR_INVALID
    big.close()
    # unequal groups are rejected at create, before anything touches the device
    bad = gm.copy()
    bad[0] = (bad[0] + 1) % cfg.N
    with pytest.raises(lmhead.CoralError) as e:
        lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(bad), ph.to_dev_bf16(Wg), 4, 4, 10)
    assert e.value.code == lmhead.CORAL_ERR_GROUPING
    assert head.status() == 0


def test_library_owned_buffers_and_host_entry():
    cfg = synth.CONFIGS["tiny"]
    W, gm, Wg, hb = synth.make_all(cfg)
    c = lmhead.make_config(cfg.H, cfg.V, cfg.N, 8, cfg.N, 10)
    handle = lmhead.coral_lmhead_create(c, ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg))
    hh = torch.from_numpy(hb.view(np.int16)).pin_memory()
    ids = torch.empty((cfg.M, 10), dtype=torch.int32).pin_memory()
    lps = torch.empty((cfg.M, 10), dtype=torch.float32).pin_memory()
    lmhead.coral_lmhead_draft_host(handle, hh, cfg.k_groups, 10, ids, lps)
    rep = ph.compare(W, gm, Wg, hb, cfg.k_groups, 10, {"ids": ids.numpy(), "logprobs": lps.numpy()})
    assert rep.ok, rep.errors
    # pageable buffers take the staged way (pinned ones are written by the last kernel directly): same results
    ids2 = torch.full((cfg.M, 10), -7, dtype=torch.int32)
    lps2 = torch.zeros((cfg.M, 10), dtype=torch.float32)
    lmhead.coral_lmhead_draft_host(handle, torch.from_numpy(hb.view(np.int16)).clone(), cfg.k_groups, 10, ids2, lps2)
    assert np.array_equal(ids2.numpy(), ids.numpy()) and np.array_equal(lps2.numpy(), lps.numpy())
    # and back to the pinned pair on the same handle
    ids.fill_(-7)
    lmhead.coral_lmhead_draft_host(handle, hh, cfg.k_groups, 10, ids, lps)
    assert np.array_equal(ids2.numpy(), ids.numpy()) and np.array_equal(lps2.numpy(), lps.numpy())
    assert lmhead.coral_lmhead_status(handle) == 0
    lmhead.coral_lmhead_destroy(handle)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,Ms", [("llama2_7b", (1, 8, 60)), ("llama3_8b", (1, 8, 60))])
def test_paper_shapes(path, name, Ms):
    cfg, W, gm, Wg, head = _weights(name)
    for M in Ms:
        hb = synth.make_hidden(cfg, M)
        head.set_path(path)
        out = ph.gpu_draft_numpy(head, hb, cfg.k_groups, cfg.k_tokens)
        assert head.status() == 0
        rep = ph.compare(W, gm, Wg, hb, cfg.k_groups, cfg.k_tokens, out)       # every row, every tap
        assert rep.ok, rep.errors
        st = head.stats()
        assert st.groups_touched == len(set(out["groups"].ravel().tolist()))


@pytest.mark.parametrize("path", PATHS + [lmhead.CORAL_PATH_TCGEN05, lmhead.CORAL_PATH_AUTO])
def test_qwen_shape_group_sweep_and_dense_equivalence(path):
    """Top-k sweep of the Qwen2.5-shaped head on every path.  On the tensor-core path k_groups = 64 has 64 x 19
    pieces per row, more candidates than the merge keeps in shared memory: its global candidate scratch is used.
    AUTO must pick the tensor-core path from 10 rows per group on."""
    cfg, W, gm, Wg, head = _weights("qwen25_7b")
    M = 60
    hb = synth.make_hidden(cfg, M)
    for kg in (2, 4, 8, 16, 64):
        head.set_path(path)
        out = ph.gpu_draft_numpy(head, hb, kg, cfg.k_tokens)
        assert head.status() == 0
        if path == lmhead.CORAL_PATH_AUTO:
            want = lmhead.CORAL_PATH_TCGEN05 if M * kg >= 10 * cfg.N else lmhead.CORAL_PATH_STREAM
            assert head.stats().path == want
        # every row up to the workload's top-8; a spread of 12 rows where a row costs 2x / 8x the oracle time
        rows = np.arange(M) if kg <= 8 else np.unique(np.linspace(0, M - 1, 12).astype(int))
        rep = ph.compare(W, gm, Wg, hb[rows], kg, cfg.k_tokens, {k: v[rows] for k, v in out.items()})
        assert rep.ok, (kg, rep.errors)
    # k_groups = N is the dense head: every row's ids/log-probs equal a dense log-softmax (library, fp32 on GPU)
    Wd, hd = ph.to_dev_bf16(W), ph.to_dev_bf16(hb)
    dense = torch.log_softmax((hd.float() @ Wd.float().T), dim=1)
    top = torch.topk(dense, cfg.k_tokens, dim=1)
    same = (top.indices.cpu().numpy() == out["ids"]).mean()
    assert same > 0.99
    np.testing.assert_allclose(out["logprobs"], top.values.cpu().numpy(), atol=2e-3)


@pytest.mark.parametrize("H,v,N,M,kg,kt", [
    (256, 256, 16, 200, 4, 10),      # one accumulator block per pass, two sub-tiles per batch
    (256, 256, 16, 300, 8, 10),      # groups with more than 128 rows: two accumulator blocks
    (256, 256, 16, 600, 8, 32),      # more than 256 rows per group: second pass; long candidate lists
    (320, 300, 6, 150, 2, 10),       # ragged group size (128 + 128 + 44) and H not a multiple of 256
    (328, 300, 6, 150, 3, 5),        # last 64-column step only partly inside H
    (256, 256, 16, 400, 8, 10),      # 200 rows per group: two passes for every group
    (320, 300, 6, 400, 3, 5),        # two passes, odd number of sub-tiles, ragged group size
    (256, 256, 16, 1200, 8, 10),     # 600 rows per group: five passes, the last one partly filled
])
def test_tensor_core_path(H, v, N, M, kg, kt):
    cfg = synth.HeadConfig("tc", H=H, V=v * N, N=N, k_groups=kg, k_tokens=kt, M=M, seed=7, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=kg, max_kt=32)
    head.set_path(lmhead.CORAL_PATH_TCGEN05)
    out = ph.gpu_draft_numpy(head, hb, kg, kt)
    assert head.status() == 0
    assert head.stats().path == lmhead.CORAL_PATH_TCGEN05
    rep = ph.compare(W, gm, Wg, hb, kg, kt, out)                # every row
    assert rep.ok, rep.errors
    again = ph.gpu_draft_numpy(head, hb, kg, kt)
    for k in out:
        assert np.array_equal(out[k], again[k]), k
    head.close()


def test_large_m_routed_grouped_gemm():
    """16 sequences x 60 tree nodes on the Llama3-8B shape: the tensor-core path, every row and every tap (groups,
    gate, all 960 x 8 x 2004 logits, log-sum-exp, ids, log-probs) against the oracle."""
    cfg, W, gm, Wg, _ = _weights("llama3_8b")
    M = 960
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=cfg.k_groups, max_kt=cfg.k_tokens)
    hb = synth.make_hidden(cfg, M)
    out = ph.gpu_draft_numpy(head, hb, cfg.k_groups, cfg.k_tokens)
    assert head.status() == 0
    st = head.stats()
    assert st.path == lmhead.CORAL_PATH_TCGEN05 and st.groups_touched == cfg.N
    rep = ph.compare(W, gm, Wg, hb, cfg.k_groups, cfg.k_tokens, out, max_errors=20)
    assert rep.ok, rep.errors
    assert rep.rows == M
    first = (out["ids"].copy(), out["logprobs"].copy())
    for _ in range(5):                                   # the same call without taps: the same bits
        ids2, lps2 = head.draft(ph.to_dev_bf16(hb), cfg.k_groups, cfg.k_tokens)
        torch.cuda.synchronize()
        assert np.array_equal(ids2.cpu().numpy(), first[0]) and np.array_equal(lps2.cpu().numpy(), first[1])
    head.close()


def test_draft_is_capturable_in_a_cuda_graph():
    """The draft call enqueues kernels only (no allocation, no host synchronisation): it can be captured once
    and replayed, and the replay gives the same bits as the direct call."""
    cfg, W, gm, Wg, head = _weights("tiny")
    head.set_path(lmhead.CORAL_PATH_AUTO)
    h = ph.to_dev_bf16(synth.make_hidden(cfg, 6))
    ids = torch.empty((6, 10), dtype=torch.int32, device="cuda")
    lps = torch.empty((6, 10), dtype=torch.float32, device="cuda")
    lmhead.coral_lmhead_draft(head.handle, h, 4, 10, ids, lps)
    torch.cuda.synchronize()
    want_ids, want_lps = ids.clone(), lps.clone()
    ids.zero_()
    lps.zero_()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        lmhead.coral_lmhead_draft(head.handle, h, 4, 10, ids, lps)
    for _ in range(2):
        ids.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(ids, want_ids) and torch.equal(lps, want_lps)
    assert head.status() == 0


@pytest.mark.parametrize("path,M,kg", [(lmhead.CORAL_PATH_STREAM, 5, 4), (lmhead.CORAL_PATH_STREAM, 40, 16),
                                       (lmhead.CORAL_PATH_TCGEN05, 200, 4)])
def test_factorised_distribution_eq8(path, M, kg):
    """p(x) = p_router(n) * p_group(x): per-group softmax times the softmax of the router scores (Eq. 7, Eq. 8)."""
    cfg = synth.CONFIGS["tiny"]
    W, gm, Wg = synth.make_w_vocab(cfg), synth.make_group_map(cfg), synth.make_w_gate(cfg)
    hb = synth.make_hidden(cfg, M)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=kg, max_kt=32)
    head.set_path(path)
    lmhead.coral_lmhead_set_output_mode(head.handle, lmhead.CORAL_OUTPUT_FACTORISED)
    out = ph.gpu_draft_numpy(head, hb, kg, 10)
    assert head.status() == 0
    rows = np.unique(np.linspace(0, M - 1, 16).astype(int))
    rep = ph.compare(W, gm, Wg, hb[rows], kg, 10, {k: a[rows] for k, a in out.items()}, factorised=True)
    assert rep.ok, rep.errors
    # the variant with p_router renormalised over the selected groups: same ids, mass 1 over the active vocabulary
    lmhead.coral_lmhead_set_output_mode(head.handle, lmhead.CORAL_OUTPUT_FACTORISED_RENORM)
    out2 = ph.gpu_draft_numpy(head, hb, kg, 10)
    assert head.status() == 0
    rep = ph.compare(W, gm, Wg, hb[rows], kg, 10, {k: a[rows] for k, a in out2.items()}, factorised=2)
    assert rep.ok, rep.errors
    # back to the joint mode on the same handle
    lmhead.coral_lmhead_set_output_mode(head.handle, lmhead.CORAL_OUTPUT_JOINT)
    out = ph.gpu_draft_numpy(head, hb, kg, 10)
    rep = ph.compare(W, gm, Wg, hb[rows], kg, 10, {k: a[rows] for k, a in out.items()})
    assert rep.ok, rep.errors
    head.close()


@pytest.mark.parametrize("M", [3, 50])
def test_two_layer_router_eq7(M):
    """scores = W2 (SiLU(W1 h) + h): groups, gate scores and the final Eq. 8 distribution against the oracle."""
    cfg = synth.CONFIGS["tiny"]
    W, gm, Wg = synth.make_w_vocab(cfg), synth.make_group_map(cfg), synth.make_w_gate(cfg)
    W1 = synth._normal_bf16(np.random.default_rng(21), cfg.H, cfg.H, 0.05)
    hb = synth.make_hidden(cfg, M)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=4, max_kt=10)
    lmhead.coral_lmhead_set_router_mlp(head.handle, ph.to_dev_bf16(W1))
    for factorised in (False, True):
        lmhead.coral_lmhead_set_output_mode(head.handle, int(factorised))
        out = ph.gpu_draft_numpy(head, hb, 4, 10)
        assert head.status() == 0
        rep = ph.compare(W, gm, Wg, hb, 4, 10, out, W1=W1, factorised=factorised)
        assert rep.ok, rep.errors
    lmhead.coral_lmhead_set_router_mlp(head.handle, None)
    lmhead.coral_lmhead_set_output_mode(head.handle, lmhead.CORAL_OUTPUT_JOINT)
    out = ph.gpu_draft_numpy(head, hb, 4, 10)
    rep = ph.compare(W, gm, Wg, hb, 4, 10, out)
    assert rep.ok, rep.errors
    head.close()


@pytest.mark.parametrize("M", [1, 8, 60])
def test_two_layer_router_eq7_on_the_llama3_shape(M):
    """Eq. 7's router at H = 4096 (W1 is 4096 x 4096, 33.5 MB more to read per call): gate scores, groups and the
    Eq. 8 distribution of every row against the oracle."""
    cfg, W, gm, Wg, head = _weights("llama3_8b")
    W1 = synth._normal_bf16(np.random.default_rng(23), cfg.H, cfg.H, 0.01)
    hb = synth.make_hidden(cfg, M)
    head.set_path(lmhead.CORAL_PATH_AUTO)
    lmhead.coral_lmhead_set_router_mlp(head.handle, ph.to_dev_bf16(W1))
    try:
        for mode in (lmhead.CORAL_OUTPUT_JOINT, lmhead.CORAL_OUTPUT_FACTORISED):
            lmhead.coral_lmhead_set_output_mode(head.handle, mode)
            out = ph.gpu_draft_numpy(head, hb, cfg.k_groups, cfg.k_tokens)
            assert head.status() == 0
            rows = np.arange(M) if M <= 8 else np.unique(np.linspace(0, M - 1, 12).astype(int))
            rep = ph.compare(W, gm, Wg, hb[rows], cfg.k_groups, cfg.k_tokens, {k: a[rows] for k, a in out.items()},
                             W1=W1, factorised=mode)
            assert rep.ok, rep.errors
    finally:
        lmhead.coral_lmhead_set_router_mlp(head.handle, None)
        lmhead.coral_lmhead_set_output_mode(head.handle, lmhead.CORAL_OUTPUT_JOINT)


@pytest.mark.parametrize("M,path", [(8, lmhead.CORAL_PATH_STREAM), (60, lmhead.CORAL_PATH_STREAM),
                                    (60, lmhead.CORAL_PATH_SIMT_PLAIN), (200, lmhead.CORAL_PATH_TCGEN05)])
def test_frequency_ordered_contiguous_groups(M, path):
    """Contiguous token-id groups with a Zipf-like prior on low-index groups (the paper's frequency-ordered
    vocabulary): a few hot groups are selected by almost every row, so they need several passes."""
    cfg = synth.HeadConfig("zipf", H=256, V=256 * 16, N=16, k_groups=4, k_tokens=10, M=M, seed=13, w_std=0.05,
                           zipf_s=1.5)
    W, Wg, hb = synth.make_w_vocab(cfg), synth.make_w_gate(cfg), synth.make_hidden(cfg)
    gm = synth.make_group_map(cfg, contiguous=True)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=4)
    head.set_path(path)
    out = ph.gpu_draft_numpy(head, hb, 4, 10)
    assert head.status() == 0 and head.stats().path == path
    counts = np.bincount(out["groups"].ravel(), minlength=16)
    assert counts[:4].sum() > counts[8:].sum()            # the prior is there: low-index groups dominate
    rows = np.unique(np.linspace(0, M - 1, 24).astype(int))
    rep = ph.compare(W, gm, Wg, hb[rows], 4, 10, {k: a[rows] for k, a in out.items()})
    assert rep.ok, rep.errors
    head.close()


@pytest.mark.parametrize("N,M,kg,path", [
    (256, 3, 256, lmhead.CORAL_PATH_STREAM),       # the maximum group count, every group active
    (256, 30, 200, lmhead.CORAL_PATH_STREAM),      # one-launch router with 8 groups per lane
    (256, 40, 7, lmhead.CORAL_PATH_STREAM),        # 40 x 256 slots: too many for the band-ticket router -> four kernels
    (128, 60, 9, lmhead.CORAL_PATH_STREAM),        # band-ticket router with 4 groups per lane
    (128, 60, 9, lmhead.CORAL_PATH_SIMT_PLAIN),
    (256, 150, 20, lmhead.CORAL_PATH_TCGEN05),     # many groups with a handful of rows each on the tensor-core path
])
def test_many_groups(N, M, kg, path):
    v = 48
    cfg = synth.HeadConfig("manyN", H=256, V=v * N, N=N, k_groups=kg, k_tokens=10, M=M, seed=17, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=kg, max_kt=10)
    head.set_path(path)
    out = ph.gpu_draft_numpy(head, hb, kg, 10)
    assert head.status() == 0 and head.stats().path == path
    rows = np.unique(np.linspace(0, M - 1, 12).astype(int))
    rep = ph.compare(W, gm, Wg, hb[rows], kg, 10, {k: a[rows] for k, a in out.items()})
    assert rep.ok, rep.errors
    head.close()


def test_tensor_core_path_mixed_entry_kinds_with_an_odd_number_of_column_steps():
    """Skewed routing over many small groups: every pair's run holds narrow entries, wide ones (129..256 rows) and
    entries of groups that need several passes, so the operand ring is re-cut inside the runs; H = 320 gives five
    64-column steps per unit, so the two producers' turns shift from unit to unit."""
    N, v, M, kg = 200, 300, 1400, 8
    cfg = synth.HeadConfig("mixedkinds", H=320, V=v * N, N=N, k_groups=kg, k_tokens=10, M=M, seed=29, w_std=0.05,
                           zipf_s=1.2)
    W, Wg, hb = synth.make_w_vocab(cfg), synth.make_w_gate(cfg), synth.make_hidden(cfg)
    gm = synth.make_group_map(cfg, contiguous=True)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=kg, max_kt=10)
    head.set_path(lmhead.CORAL_PATH_TCGEN05)
    out = ph.gpu_draft_numpy(head, hb, kg, 10)
    assert head.status() == 0 and head.stats().path == lmhead.CORAL_PATH_TCGEN05
    counts = np.bincount(out["groups"].ravel(), minlength=N)
    assert (counts > 256).any() and ((counts > 128) & (counts <= 256)).any() and ((counts > 0) & (counts <= 128)).any()
    rows = np.unique(np.linspace(0, M - 1, 40).astype(int))
    rep = ph.compare(W, gm, Wg, hb[rows], kg, 10, {k: a[rows] for k, a in out.items()})
    assert rep.ok, rep.errors
    again = ph.gpu_draft_numpy(head, hb, kg, 10)
    for k in ("ids", "logprobs", "groups"):
        assert np.array_equal(out[k], again[k]), k
    head.close()


@pytest.mark.parametrize("zipf", [0.0, 1.5])
def test_tensor_core_path_many_rows_take_the_batches_in_turn(zipf):
    """More than 96 MB of gathered hidden rows (1600 rows x 8 groups x 8 KiB): the pairs take the call's batches
    in turn instead of consecutive runs.  Every group needs several passes of 256 rows (its weights are read
    again), the last tile of a group is ragged, and with the skewed routing narrow entries sit between the wide
    ones, so the operand ring is re-cut between a pair's batches."""
    N, v, M, kg = 16, 300, 1600, 8
    cfg = synth.HeadConfig("turns", H=4096, V=v * N, N=N, k_groups=kg, k_tokens=10, M=M, seed=31, w_std=0.02,
                           zipf_s=zipf)
    W, Wg, hb = synth.make_w_vocab(cfg), synth.make_w_gate(cfg), synth.make_hidden(cfg)
    gm = synth.make_group_map(cfg, contiguous=zipf > 0)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=kg, max_kt=10)
    head.set_path(lmhead.CORAL_PATH_TCGEN05)
    out = ph.gpu_draft_numpy(head, hb, kg, 10)
    assert head.status() == 0 and head.stats().path == lmhead.CORAL_PATH_TCGEN05
    counts = np.bincount(out["groups"].ravel(), minlength=N)
    assert (counts > 256).any()
    if zipf > 0:
        assert ((counts % 256 > 0) & (counts % 256 <= 128)).any()      # some entry is narrow
    rows = np.unique(np.linspace(0, M - 1, 64).astype(int))
    rep = ph.compare(W, gm, Wg, hb[rows], kg, 10, {k: a[rows] for k, a in out.items()})
    assert rep.ok, rep.errors
    again = ph.gpu_draft_numpy(head, hb, kg, 10)
    for k in ("ids", "logprobs", "groups"):
        assert np.array_equal(out[k], again[k]), k
    head.close()


@pytest.mark.parametrize("M,kg,zipf,expect", [
    (40, 2, 0.0, lmhead.CORAL_PATH_STREAM),      # ~5 rows per group: one read per group either way -> streaming kernel
    (60, 4, 1.5, lmhead.CORAL_PATH_TCGEN05),     # hot groups selected by most rows -> tensor-core kernel
    (128, 8, 0.0, lmhead.CORAL_PATH_TCGEN05),    # 64 rows per group: four streaming passes against one
    (100, 3, 0.0, None),                         # near the break-even: either choice, same results
    (8, 4, 0.0, lmhead.CORAL_PATH_STREAM),       # outside 33..128 rows the call is an ordinary one
])
def test_adaptive_path_choice_on_device(M, kg, zipf, expect):
    cfg = synth.HeadConfig("adaptive", H=256, V=256 * 16, N=16, k_groups=kg, k_tokens=10, M=M, seed=23, w_std=0.05,
                           zipf_s=zipf)
    W, Wg, hb = synth.make_w_vocab(cfg), synth.make_w_gate(cfg), synth.make_hidden(cfg)
    gm = synth.make_group_map(cfg, contiguous=zipf > 0)
    head = _head(cfg, W, gm, Wg, max_M=128, max_kg=8)
    head.set_path(lmhead.CORAL_PATH_ADAPTIVE)
    out = ph.gpu_draft_numpy(head, hb, kg, 10)
    assert head.status() == 0
    took = head.stats().path
    assert took in (lmhead.CORAL_PATH_STREAM, lmhead.CORAL_PATH_TCGEN05)
    if expect is not None:
        assert took == expect
    rows = np.unique(np.linspace(0, M - 1, 24).astype(int))
    rep = ph.compare(W, gm, Wg, hb[rows], kg, 10, {k: a[rows] for k, a in out.items()})
    assert rep.ok, rep.errors
    # the same call on the path it took, forced from the host: identical bits
    head.set_path(took)
    again = ph.gpu_draft_numpy(head, hb, kg, 10)
    for k in ("ids", "logprobs", "groups"):
        assert np.array_equal(out[k], again[k]), k
    head.close()


def test_copy_floor_probe_runs_and_checks_arguments():
    cfg, W, gm, Wg, hb = (synth.CONFIGS["tiny"],) + synth.make_all(synth.CONFIGS["tiny"])
    head = _head(cfg, W, gm, Wg)
    lib = lmhead.load_library()
    packed_bytes, _ = lmhead.coral_lmhead_query_sizes(head.cfg)
    lmhead.coral_lmhead_copy_floor(head.handle, packed_bytes)
    lmhead.coral_lmhead_copy_floor(head.handle, 16384 * 3 + 5)
    lmhead.coral_lmhead_copy_floor(head.handle, packed_bytes, in_flight=13, repeats=3)
    lmhead.coral_lmhead_copy_floor(head.handle, packed_bytes, in_flight=1, repeats=2)
    torch.cuda.synchronize()
    assert head.status() == 0
    assert lib.coral_lmhead_copy_floor(head.handle, 100, 0, 1, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_copy_floor(head.handle, packed_bytes + 16384, 0, 1, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_copy_floor(head.handle, packed_bytes, 14, 1, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_copy_floor(head.handle, packed_bytes, 8, 0, None) == lmhead.CORAL_ERR_INVALID
    head.close()


def test_tensor_core_issue_probe_runs_and_checks_arguments():
    cfg = synth.HeadConfig("probe", H=256, V=256 * 16, N=16, k_groups=4, k_tokens=10, M=64, seed=3)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg, max_M=64, max_kg=4, max_kt=10)
    lib = lmhead.load_library()
    out = torch.zeros(2, dtype=torch.int64, device="cuda")
    for n, iss in ((16, 1), (128, 2), (256, 1)):
        lmhead.coral_lmhead_tc_issue_probe(head.handle, n, 4, iss, 200, out)
        torch.cuda.synchronize()
        t_issue, t_done = out.cpu().tolist()
        assert 0 < t_issue <= t_done < 10_000_000
    assert head.status() == 0
    p = ctypes.c_void_p(out.data_ptr())
    assert lib.coral_lmhead_tc_issue_probe(head.handle, 24, 4, 1, 10, p, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_tc_issue_probe(head.handle, 128, 0, 1, 10, p, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_tc_issue_probe(head.handle, 128, 4, 3, 10, p, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_tc_issue_probe(head.handle, 128, 4, 1, 10, None, None) == lmhead.CORAL_ERR_INVALID
    out2 = ph.gpu_draft_numpy(head, hb, 4, 10)                   # the handle still drafts correctly afterwards
    rep = ph.compare(W, gm, Wg, hb[:8], 4, 10, {k: a[:8] for k, a in out2.items()})
    assert rep.ok, rep.errors
    head.close()


def test_expired_wait_is_reported_and_the_handle_stays_usable():
    """Failure detection without a fault: the kernels' bounded wait runs out on a barrier nothing completes,
    the status word says so, and the next draft call on the same handle is correct."""
    cfg = synth.CONFIGS["tiny"]
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg)
    lmhead.coral_lmhead_selftest_wait_expiry(head.handle)
    assert head.status() == lmhead.CORAL_ERR_TIMEOUT
    assert head.status() == 0                          # reading the status clears it
    out = ph.gpu_draft_numpy(head, hb, cfg.k_groups, cfg.k_tokens)
    assert head.status() == 0
    rep = ph.compare(W, gm, Wg, hb, cfg.k_groups, cfg.k_tokens, out)
    assert rep.ok, rep.errors
    head.close()


def test_hot_groups_window_changes_no_result():
    """The persisting-L2 window over the leading groups is a cache hint: same bits with and without it."""
    cfg = synth.HeadConfig("hot", H=256, V=256 * 16, N=16, k_groups=4, k_tokens=10, M=8, seed=29, w_std=0.05, zipf_s=1.5)
    W, Wg, hb = synth.make_w_vocab(cfg), synth.make_w_gate(cfg), synth.make_hidden(cfg)
    gm = synth.make_group_map(cfg, contiguous=True)
    head = _head(cfg, W, gm, Wg, max_M=8, max_kg=4)
    base = ph.gpu_draft_numpy(head, hb, 4, 10)
    lmhead.coral_lmhead_set_hot_groups(head.handle, 3)
    hot = ph.gpu_draft_numpy(head, hb, 4, 10)
    hot2 = ph.gpu_draft_numpy(head, hb, 4, 10)
    assert head.status() == 0
    lmhead.coral_lmhead_set_hot_groups(head.handle, 0)
    off = ph.gpu_draft_numpy(head, hb, 4, 10)
    for k in base:
        assert np.array_equal(base[k], hot[k]) and np.array_equal(base[k], hot2[k]) and np.array_equal(base[k], off[k]), k
    lib = lmhead.load_library()
    assert lib.coral_lmhead_set_hot_groups(head.handle, 17) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_set_hot_groups(head.handle, -1) == lmhead.CORAL_ERR_INVALID
    rep = ph.compare(W, gm, Wg, hb, 4, 10, hot)
    assert rep.ok, rep.errors
    head.close()


def test_streaming_path_repeats_bit_for_bit_with_many_passes():
    """Every row selects every group, so each group is streamed in four passes and every CTA changes segment
    several times, the moment at which a ring slot is refilled the instant it is released: 30 calls must agree
    to the bit (a missing ordering between the warps' reads of a slot and its refill showed up only here)."""
    cfg, W, gm, Wg, head = _weights("llama3_8b")
    head.set_path(lmhead.CORAL_PATH_STREAM)
    M = 60
    hidden = ph.to_dev_bf16(synth.make_hidden(cfg, M))
    ref = None
    for i in range(30):
        ids, lps = head.draft(hidden, cfg.N, cfg.k_tokens)
        torch.cuda.synchronize()
        cur = (ids.cpu().numpy(), lps.cpu().numpy())
        if ref is None:
            ref = cur
        else:
            assert np.array_equal(cur[0], ref[0]) and np.array_equal(cur[1], ref[1]), i
    assert head.status() == 0
    rows = np.array([0, 29, 59])
    hb = synth.make_hidden(cfg, M)
    rep = ph.compare(W, gm, Wg, hb[rows], cfg.N, cfg.k_tokens, {"ids": ref[0][rows], "logprobs": ref[1][rows]})
    assert rep.ok, rep.errors


@pytest.mark.parametrize("seed", [1, 2])
def test_other_seeds_on_the_llama2_shape(seed):
    """The recipe's other seeds (weights, group map and hidden rows all change) on the Llama2-7B-shaped head."""
    cfg = synth.CONFIGS["llama2_7b"].with_(seed=seed)
    W, gm, Wg = synth.make_w_vocab(cfg), synth.make_group_map(cfg), synth.make_w_gate(cfg)
    head = _head(cfg, W, gm, Wg, max_M=60, max_kg=cfg.k_groups, max_kt=cfg.k_tokens)
    for M in (1, 8, 60):
        hb = synth.make_hidden(cfg, M)
        out = ph.gpu_draft_numpy(head, hb, cfg.k_groups, cfg.k_tokens)
        assert head.status() == 0
        rows = np.unique(np.linspace(0, M - 1, 6).astype(int))
        rep = ph.compare(W, gm, Wg, hb[rows], cfg.k_groups, cfg.k_tokens, {k: v[rows] for k, v in out.items()})
        assert rep.ok, (M, rep.errors)
    head.close()


@pytest.mark.parametrize("H,M", [(256, 4), (256, 40), (256, 200), (328, 13)])
def test_bad_router_input_is_reported_and_indexes_nothing(H, M):
    """A NaN hidden row (so NaN router scores) and a forced group named twice, on every router variant (one-launch
    router, band router, band router + bucketing launch, plain kernels for H not a multiple of 32): the status word
    says what happened, every selected group is a valid, distinct index, the kernels after the router stage do
    nothing (the outputs keep what they held), and the handle works again once the status has been read."""
    cfg = synth.HeadConfig("badin", H=H, V=1536, N=6, k_groups=3, k_tokens=10, M=M, seed=11, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=cfg.N, max_kt=10)
    good = ph.gpu_draft_numpy(head, hb, 3, 10)
    assert head.status() == 0

    def run(hidden_bits, forced=None):
        dev = "cuda"
        ids = torch.full((M, 10), -7, dtype=torch.int32, device=dev)
        lps = torch.full((M, 10), 123.0, dtype=torch.float32, device=dev)
        groups = torch.full((M, 3), -1, dtype=torch.int32, device=dev)
        fg = None if forced is None else torch.from_numpy(forced).to(dev)
        lmhead.coral_lmhead_draft_ex(head.handle, ph.to_dev_bf16(hidden_bits), 3, 10, ids, lps, forced_groups=fg,
                                     out_groups=groups)
        torch.cuda.synchronize()
        return ids.cpu().numpy(), lps.cpu().numpy(), groups.cpu().numpy()

    nan_row = hb.copy()
    nan_row[M // 2, 5] = 0x7FC0                                   # a bf16 NaN
    ids, lps, groups = run(nan_row)
    assert head.status() == lmhead.CORAL_ERR_NONFINITE
    assert groups.min() >= 0 and groups.max() < cfg.N
    assert all(len(set(r.tolist())) == 3 for r in groups)
    assert groups[M // 2].tolist() == [0, 1, 2]                   # all scores of that row rank last: lowest indices
    assert np.all(ids == -7) and np.all(lps == 123.0)             # nothing after the router stage ran

    forced = np.tile(np.array([4, 1, 4], np.int32), (M, 1))       # group 4 twice
    ids, lps, groups = run(hb, forced)
    assert head.status() == lmhead.CORAL_ERR_BOUNDS
    assert np.all(ids == -7) and np.all(lps == 123.0)
    forced = np.tile(np.array([4, 99, 0], np.int32), (M, 1))      # a group outside [0, N)
    ids, lps, groups = run(hb, forced)
    assert head.status() == lmhead.CORAL_ERR_BOUNDS
    assert np.all(ids == -7)

    again = ph.gpu_draft_numpy(head, hb, 3, 10)                   # status read: the handle is usable again
    assert head.status() == 0
    for k in good:
        assert np.array_equal(good[k], again[k]), k
    head.close()
