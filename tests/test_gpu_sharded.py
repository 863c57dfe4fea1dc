"""GPU parity of the vocab-sharded draft step (one exchange step, Appendix B's union of groups dealt over
several GPUs): every rank's per-row record is produced on ONE GPU, one rank after the other (nothing waits
on anything), stacked the way an all-gather leaves them, merged, and compared with the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2502_16880_b200 import lmhead, synth
from oracle import lmhead_oracle as orc
from oracle import shard_oracle as sho
from tests import parity_harness as ph

pytestmark = pytest.mark.gpu


def _head(cfg, W, gm, Wg, max_M, max_kg, max_kt=32):
    return lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg), max_M, max_kg, max_kt)


def _sharded(head, hidden, kg, kt, world):
    M = hidden.shape[0]
    W = 2 + 2 * kt
    gathered = torch.full((world, M, W), -1, dtype=torch.int32, device="cuda")
    touched = []
    for r in range(world):
        lmhead.coral_lmhead_set_group_shard(head.handle, r, world)
        lmhead.coral_lmhead_draft_partial(head.handle, hidden, kg, kt, gathered[r])
        torch.cuda.synchronize()
        assert head.status() == 0
        touched.append(head.stats().groups_touched)
    lmhead.coral_lmhead_set_group_shard(head.handle, 0, 1)
    ids = torch.empty((M, kt), dtype=torch.int32, device="cuda")
    lps = torch.empty((M, kt), dtype=torch.float32, device="cuda")
    lmhead.coral_lmhead_merge_partials(gathered, kt, ids, lps)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), lps.cpu().numpy(), touched, gathered.cpu().numpy()


@pytest.mark.parametrize("H,v,N,M,kg,kt,path", [
    (256, 256, 16, 4, 4, 10, lmhead.CORAL_PATH_STREAM),       # few rows: one-launch router
    (256, 256, 16, 1, 2, 10, lmhead.CORAL_PATH_STREAM),       # one row: most ranks own none of its groups
    (256, 300, 12, 60, 5, 10, lmhead.CORAL_PATH_STREAM),      # 33..128 rows: band-ticket router, ragged groups
    (256, 256, 16, 128, 8, 32, lmhead.CORAL_PATH_STREAM),     # groups streamed in several passes
    (256, 256, 16, 200, 4, 10, lmhead.CORAL_PATH_TCGEN05),    # many rows: tensor-core path, four-kernel router
    (320, 300, 6, 150, 3, 5, lmhead.CORAL_PATH_TCGEN05),
])
@pytest.mark.parametrize("world", [2, 3, 8])
def test_vocab_sharded_draft_matches_oracle(H, v, N, M, kg, kt, path, world):
    if world > N:
        pytest.skip("more ranks than groups")
    cfg = synth.HeadConfig("shard", H=H, V=v * N, N=N, k_groups=kg, k_tokens=kt, M=M, seed=11, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg, max_M=M, max_kg=kg)
    head.set_path(path)
    hidden = ph.to_dev_bf16(hb)
    ids1, lps1 = head.draft(hidden, kg, kt)
    torch.cuda.synchronize()
    whole = head.stats().groups_touched
    ids, lps, touched, rec = _sharded(head, hidden, kg, kt, world)
    assert sum(touched) == whole                       # every touched group is read by exactly one rank
    rows = np.unique(np.linspace(0, M - 1, 24).astype(int))
    # every rank's records, element by element, against the shard oracle
    ref = orc.draft(W, gm, Wg, hb[rows], kg, kt)
    for r in range(world):
        mx, sm, z, tid = sho.records(ref, r, world, kt)
        g_mx = rec[r, rows, 0].copy().view(np.float32)
        g_sm = rec[r, rows, 1].copy().view(np.float32)
        g_z = rec[r, rows, 2:2 + kt].copy().view(np.float32)
        g_id = rec[r, rows, 2 + kt:]
        assert np.array_equal(np.isneginf(g_mx), np.isneginf(mx))
        live = ~np.isneginf(mx)
        assert np.all(ph.close(g_mx[live], mx[live]))
        assert np.all(ph.close(np.log(g_sm[live]) + g_mx[live], np.log(sm[live]) + mx[live]))   # the rank's log-sum-exp
        assert np.array_equal(np.isneginf(g_z), np.isneginf(z))
        assert np.all(ph.close(g_z[live], z[live]))
        differ = g_id != tid
        if differ.any():                               # only where the oracle's own logits tie within tolerance
            zmap = [dict(zip(ref.logit_tokens[i].ravel().tolist(), ref.logits[i].ravel().tolist())) for i in range(len(rows))]
            for i, j in np.argwhere(differ):
                assert ph.close(zmap[i][int(g_id[i, j])], z[i, j])
    rep = ph.compare(W, gm, Wg, hb[rows], kg, kt, {"ids": ids[rows], "logprobs": lps[rows]})
    assert rep.ok, rep.errors
    # against the same library on one GPU: same tokens, log-probs equal up to the order of the fp32 sums
    ids1, lps1 = ids1.cpu().numpy(), lps1.cpu().numpy()
    same = ids == ids1
    assert same.mean() > 0.99
    assert np.all(ph.close(lps[same], lps1[same]))
    head.close()


def test_record_of_a_rank_without_local_groups_is_empty():
    cfg = synth.HeadConfig("shard", H=256, V=256 * 16, N=16, k_groups=1, k_tokens=10, M=3, seed=5, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg, max_M=3, max_kg=1)
    _, _, touched, rec = _sharded(head, ph.to_dev_bf16(hb), 1, 10, 4)
    assert sum(touched) <= 3
    empty = 0
    for r in range(4):
        for m in range(3):
            mx = rec[r, m, 0:1].view(np.float32)[0]
            if np.isneginf(mx):
                empty += 1
                assert rec[r, m, 1:2].view(np.float32)[0] == 0.0
                assert np.all(np.isneginf(rec[r, m, 2:12].view(np.float32)))
                assert np.all(rec[r, m, 12:22] == 0x7FFFFFFF)
    assert empty == 3 * 3                              # k_groups = 1: each row lives on exactly one of the 4 ranks
    head.close()


def test_sharded_handle_rejects_unsharded_calls_and_bad_arguments():
    cfg = synth.HeadConfig("shard", H=256, V=256 * 16, N=16, k_groups=4, k_tokens=10, M=4, seed=5, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    head = _head(cfg, W, gm, Wg, max_M=4, max_kg=4)
    lib = lmhead.load_library()
    assert lib.coral_lmhead_set_group_shard(head.handle, 2, 2) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_set_group_shard(head.handle, 0, 17) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_set_group_shard(head.handle, -1, 2) == lmhead.CORAL_ERR_INVALID
    lmhead.coral_lmhead_set_group_shard(head.handle, 1, 2)
    with pytest.raises(lmhead.CoralError):
        head.draft(ph.to_dev_bf16(hb), 4, 10)
    lmhead.coral_lmhead_set_group_shard(head.handle, 0, 1)
    head.draft(ph.to_dev_bf16(hb), 4, 10)
    torch.cuda.synchronize()
    assert head.status() == 0
    ids = torch.empty((4, 32), dtype=torch.int32, device="cuda")
    lps = torch.empty((4, 32), dtype=torch.float32, device="cuda")
    rec = torch.zeros((9, 4, 66), dtype=torch.int32, device="cuda")
    assert lib.coral_lmhead_merge_partials(lmhead._dev_ptr(rec), 9, 4, 32, lmhead._dev_ptr(ids), lmhead._dev_ptr(lps),
                                           None) == lmhead.CORAL_ERR_TOO_LARGE
    head.close()


@pytest.mark.parametrize("M,kg,path", [(8, 4, lmhead.CORAL_PATH_STREAM), (60, 5, lmhead.CORAL_PATH_STREAM),
                                       (200, 4, lmhead.CORAL_PATH_TCGEN05), (5, 3, lmhead.CORAL_PATH_SIMT_PLAIN)])
@pytest.mark.parametrize("world", [2, 3])
def test_handles_that_store_only_their_own_groups(M, kg, path, world):
    """One handle per rank, created with CORAL_CFG_SHARD(rank, world): it packs only the groups n % world == rank
    (about 1/world of the bytes) and produces the same records as a full handle given that shard."""
    H, v, N, kt = 256, 300, 12, 10
    cfg = synth.HeadConfig("shardmem", H=H, V=v * N, N=N, k_groups=kg, k_tokens=kt, M=M, seed=31, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    hidden = ph.to_dev_bf16(hb)
    full = _head(cfg, W, gm, Wg, max_M=M, max_kg=kg)
    full_bytes, _ = lmhead.coral_lmhead_query_sizes(full.cfg)
    if path == lmhead.CORAL_PATH_SIMT_PLAIN:
        # the plain path has no record output; a sharded handle must still refuse cleanly
        sh = lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg), M, kg, 32, shard=(0, world))
        sh.set_path(path)
        rec = torch.empty((M, 2 + 2 * kt), dtype=torch.int32, device="cuda")
        with pytest.raises(lmhead.CoralError):
            lmhead.coral_lmhead_draft_partial(sh.handle, hidden, kg, kt, rec)
        sh.close()
        full.close()
        return
    full.set_path(path)
    want_ids, want_lps, _, want_rec = _sharded(full, hidden, kg, kt, world)
    gathered = torch.empty((world, M, 2 + 2 * kt), dtype=torch.int32, device="cuda")
    total = 0
    for r in range(world):
        sh = lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg), M, kg, 32, shard=(r, world))
        b, _ = lmhead.coral_lmhead_query_sizes(sh.cfg)
        total += b
        assert b == full_bytes // N * len(range(r, N, world))
        sh.set_path(path)
        lib = lmhead.load_library()
        assert lib.coral_lmhead_set_group_shard(sh.handle, (r + 1) % world, world) == lmhead.CORAL_ERR_INVALID
        assert lib.coral_lmhead_set_group_shard(sh.handle, 0, 1) == lmhead.CORAL_ERR_INVALID
        lmhead.coral_lmhead_draft_partial(sh.handle, hidden, kg, kt, gathered[r])
        torch.cuda.synchronize()
        assert sh.status() == 0
        sh.close()
    assert total == full_bytes                              # the ranks' packed copies partition the head
    assert np.array_equal(gathered.cpu().numpy(), want_rec)  # bit-identical to the full handle's records
    ids = torch.empty((M, kt), dtype=torch.int32, device="cuda")
    lps = torch.empty((M, kt), dtype=torch.float32, device="cuda")
    lmhead.coral_lmhead_merge_partials(gathered, kt, ids, lps)
    torch.cuda.synchronize()
    assert np.array_equal(ids.cpu().numpy(), want_ids) and np.array_equal(lps.cpu().numpy(), want_lps)
    rows = np.unique(np.linspace(0, M - 1, 12).astype(int))
    rep = ph.compare(W, gm, Wg, hb[rows], kg, kt, {"ids": want_ids[rows], "logprobs": want_lps[rows]})
    assert rep.ok, rep.errors
    full.close()


@pytest.mark.parametrize("zipf", [0.0, 1.5])
def test_sharded_step_with_the_kernel_chosen_on_the_device(zipf):
    """Vocab sharding together with CORAL_PATH_ADAPTIVE: each rank's router decides from its own groups' row
    counts (so ranks may take different kernels); the merged result still matches the oracle."""
    M, kg, kt, world = 60, 4, 10, 2
    cfg = synth.HeadConfig("shard_adaptive", H=256, V=256 * 16, N=16, k_groups=kg, k_tokens=kt, M=M, seed=37,
                           w_std=0.05, zipf_s=zipf)
    W, Wg, hb = synth.make_w_vocab(cfg), synth.make_w_gate(cfg), synth.make_hidden(cfg)
    gm = synth.make_group_map(cfg, contiguous=zipf > 0)
    head = _head(cfg, W, gm, Wg, max_M=128, max_kg=kg)
    head.set_path(lmhead.CORAL_PATH_ADAPTIVE)
    ids, lps, touched, _ = _sharded(head, ph.to_dev_bf16(hb), kg, kt, world)
    rows = np.unique(np.linspace(0, M - 1, 24).astype(int))
    rep = ph.compare(W, gm, Wg, hb[rows], kg, kt, {"ids": ids[rows], "logprobs": lps[rows]})
    assert rep.ok, rep.errors
    head.close()
