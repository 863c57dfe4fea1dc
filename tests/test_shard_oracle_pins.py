"""Pins of the vocab-shard oracle against the unsharded oracle (itself pinned in test_oracle_pins.py) and
against what the arithmetic fixes; plus the exchange step on two gloo ranks."""
import os
import sys

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import lmhead_oracle as orc
from oracle import shard_oracle as sho
from paper_2502_16880_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _case(M=6, kg=5, kt=10, N=12, v=40, H=64, seed=3):
    cfg = synth.HeadConfig("shard", H=H, V=v * N, N=N, k_groups=kg, k_tokens=kt, M=M, seed=seed, w_std=0.05)
    W, gm, Wg, hb = synth.make_all(cfg)
    return cfg, orc.draft(W, gm, Wg, hb, kg, kt), (W, gm, Wg, hb)


@pytest.mark.parametrize("world", [1, 2, 3, 5, 12])
def test_merged_records_reproduce_the_unsharded_result(world):
    cfg, ref, _ = _case()
    kt = cfg.k_tokens
    gathered = np.stack([sho.pack(*sho.records(ref, r, world, kt)) for r in range(world)])
    ids, lps = sho.merge(gathered, kt)
    assert np.array_equal(ids, ref.ids)
    # records travel as float32: the log-probs agree to float32 rounding of logits of size ~1
    assert np.abs(lps - ref.logprobs).max() < 1e-5


def test_ranks_partition_the_active_set_and_probabilities_sum_to_one():
    cfg, ref, _ = _case(M=4, kg=7, kt=3)
    world = 4
    for m in range(4):
        total = 0.0
        owners = [n % world for n in ref.groups[m]]
        for r in range(world):
            mx, sm, z, ids = sho.records(ref, r, world, 3)
            if r not in owners:
                assert np.isneginf(mx[m]) and sm[m] == 0 and np.all(ids[m] == sho.NO_TOKEN)
            else:
                total += sm[m] * np.exp(mx[m] - ref.lse[m])     # this rank's share of the row's probability mass
                assert set(ids[m].tolist()) <= {int(t) for s, n in enumerate(ref.groups[m]) if n % world == r
                                                for t in ref.logit_tokens[m, s]}
        assert abs(total - 1.0) < 1e-12


def test_closed_form_zero_weights():
    """All-zero head: every logit is 0, so a rank owning g of a row's groups reports max 0, sum g * v and the g * v
    lowest token ids first; the merged log-prob is -log(k_groups * v)."""
    N, v, H, kg, kt, world = 6, 8, 16, 4, 5, 3
    W = np.zeros((N * v, H), dtype=np.uint16)
    gm = (np.arange(N * v) // v).astype(np.int32)
    Wg = synth.fp32_to_bf16_bits(np.random.default_rng(0).normal(size=(N, H)).astype(np.float32))
    hb = synth.fp32_to_bf16_bits(np.random.default_rng(1).normal(size=(2, H)).astype(np.float32))
    ref = orc.draft(W, gm, Wg, hb, kg, kt)
    gathered = []
    for r in range(world):
        mx, sm, z, ids = sho.records(ref, r, world, kt)
        for m in range(2):
            g = sum(1 for n in ref.groups[m] if n % world == r)
            if g:
                assert mx[m] == 0 and sm[m] == g * v
                mine = sorted(t for n in ref.groups[m] if n % world == r for t in range(n * v, n * v + v))
                assert ids[m].tolist() == mine[:kt]
        gathered.append(sho.pack(mx, sm, z, ids))
    ids, lps = sho.merge(np.stack(gathered), kt)
    assert np.allclose(lps, -np.log(kg * v), atol=1e-6)
    assert np.array_equal(ids, ref.ids)


def _rank_main(rank, world, port, q):
    import torch
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    cfg, ref, _ = _case()
    mine = torch.from_numpy(sho.pack(*sho.records(ref, rank, world, cfg.k_tokens)))
    gathered = torch.empty((world,) + tuple(mine.shape), dtype=torch.int32)
    dist.all_gather_into_tensor(gathered.view(-1, mine.shape[1]), mine)   # the one exchange step of the sharded path
    ids, lps = sho.merge(gathered.numpy(), cfg.k_tokens)
    q.put((rank, bool(np.array_equal(ids, ref.ids)), float(np.abs(lps - ref.logprobs).max())))
    dist.destroy_process_group()


def test_exchange_step_on_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, same, err in res:
        assert same and err < 1e-5
