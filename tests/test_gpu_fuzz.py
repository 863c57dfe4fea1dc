"""Seeded random shapes on every path and option against the CPU oracle (ragged sizes, odd group counts,
row counts around every switch of router and head kernel)."""
import numpy as np
import pytest
import torch

from paper_2502_16880_b200 import lmhead, synth
from tests import parity_harness as ph

pytestmark = pytest.mark.gpu

PATHS = (lmhead.CORAL_PATH_AUTO, lmhead.CORAL_PATH_STREAM, lmhead.CORAL_PATH_TCGEN05, lmhead.CORAL_PATH_SIMT_PLAIN,
         lmhead.CORAL_PATH_ADAPTIVE)


@pytest.mark.parametrize("seed", [3, 4])
def test_random_shapes_on_every_path(seed):
    rng = np.random.default_rng(seed)
    for case in range(40):
        H = int(rng.choice([64, 128, 256, 320, 512, 768, 1024]))
        N = int(rng.integers(1, 41))
        v = int(rng.integers(3, 301))
        M = int(rng.choice([1, 2, 3, 7, 8, 9, 16, 17, 31, 32, 33, 40, 64, 65, 100, 128, 129, 150, 200, 260]))
        kg = int(rng.integers(1, N + 1))
        kt = int(rng.integers(1, min(32, kg * v) + 1))
        zipf = float(rng.choice([0.0, 0.0, 1.5]))
        cfg = synth.HeadConfig("fuzz", H=H, V=v * N, N=N, k_groups=kg, k_tokens=kt, M=M, seed=int(rng.integers(0, 1000)),
                               w_std=0.05, zipf_s=zipf)
        W, gm, Wg, hb = synth.make_all(cfg)
        what = f"case {case}: H={H} N={N} v={v} M={M} kg={kg} kt={kt} zipf={zipf}"
        head = lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg), M, kg, 32)
        rows = np.unique(rng.integers(0, M, size=min(M, 6)))
        took_any = False
        for path in PATHS:
            head.set_path(path)
            try:
                out = ph.gpu_draft_numpy(head, hb, kg, kt)
            except lmhead.CoralError:
                continue                                   # the forced path cannot take this call
            took_any = True
            assert head.status() == 0, (what, path)
            rep = ph.compare(W, gm, Wg, hb[rows], kg, kt, {k: a[rows] for k, a in out.items()})
            assert rep.ok, (what, path, rep.errors[:2])
            if head.stats().path == lmhead.CORAL_PATH_SIMT_PLAIN:
                continue                                   # the plain path has neither records nor the Eq. 8 mode
            if N >= 2 and rng.random() < 0.5:              # the same call, vocab-sharded
                world = int(rng.integers(2, min(N, 5) + 1))
                gathered = torch.empty((world, M, 2 + 2 * kt), dtype=torch.int32, device="cuda")
                for r in range(world):
                    lmhead.coral_lmhead_set_group_shard(head.handle, r, world)
                    lmhead.coral_lmhead_draft_partial(head.handle, ph.to_dev_bf16(hb), kg, kt, gathered[r])
                lmhead.coral_lmhead_set_group_shard(head.handle, 0, 1)
                ids = torch.empty((M, kt), dtype=torch.int32, device="cuda")
                lps = torch.empty((M, kt), dtype=torch.float32, device="cuda")
                lmhead.coral_lmhead_merge_partials(gathered, kt, ids, lps)
                torch.cuda.synchronize()
                assert head.status() == 0, (what, path, "sharded")
                rep = ph.compare(W, gm, Wg, hb[rows], kg, kt,
                                 {"ids": ids.cpu().numpy()[rows], "logprobs": lps.cpu().numpy()[rows]})
                assert rep.ok, (what, path, f"world {world}", rep.errors[:2])
            if rng.random() < 0.3:                         # the same call in the Eq. 8 output mode
                lmhead.coral_lmhead_set_output_mode(head.handle, lmhead.CORAL_OUTPUT_FACTORISED)
                out = ph.gpu_draft_numpy(head, hb, kg, kt)
                lmhead.coral_lmhead_set_output_mode(head.handle, lmhead.CORAL_OUTPUT_JOINT)
                assert head.status() == 0, (what, path, "eq8")
                rep = ph.compare(W, gm, Wg, hb[rows], kg, kt, {k: a[rows] for k, a in out.items()}, factorised=True)
                assert rep.ok, (what, path, "eq8", rep.errors[:2])
        assert took_any, what
        head.close()
