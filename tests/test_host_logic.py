"""CPU-side checks: the C-ABI library builds, loads and exports every symbol the
header declares (no compute calls), argument checks that need no device, the
input generators, and the multi-rank bookkeeping of the bench on gloo ranks."""
import ctypes
import os
import re
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_2502_16880_b200 import build as cbuild
from paper_2502_16880_b200 import lmhead, synth


@pytest.fixture(scope="module")
def lib():
    cbuild.build_library()
    return lmhead.load_library()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "coral_lmhead.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(coral_(?:lmhead|tree|csra)_[a-z0-9_]+)\s*\(", header))
    assert {"coral_lmhead_create", "coral_lmhead_draft", "coral_lmhead_draft_ex", "coral_lmhead_destroy"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(lmhead._SIGNATURES), declared ^ set(lmhead._SIGNATURES)
    assert lmhead.coral_lmhead_version() == 1


def test_error_strings_and_host_only_argument_checks(lib):
    assert lmhead.coral_lmhead_error_string(0) == "ok"
    for code in range(-8, 0):
        assert lmhead.coral_lmhead_error_string(code) not in ("ok", "unknown status")
    ok = lmhead.make_config(4096, 128256, 64, 960, 8, 10)
    pb, wb = lmhead.coral_lmhead_query_sizes(ok)
    assert pb == 64 * 126 * 16 * 4096 * 2 and wb > 0 and wb % 256 == 0   # groups x 16-row items x 64-column blocks x 16 x 64 x 2
    for bad in [lmhead.make_config(4096, 128256, 63, 8, 8, 10),     # V % N != 0
                lmhead.make_config(4100, 128256, 64, 8, 8, 10),     # H % 8 != 0
                lmhead.make_config(4096, 128256, 64, 0, 8, 10),
                lmhead.make_config(4096, 128256, 64, 8, 65, 10),
                lmhead.make_config(4096, 128256, 64, 8, 8, 33),
                lmhead.make_config(4096, 512 * 300, 512, 8, 8, 10)]:
        with pytest.raises(lmhead.CoralError) as e:
            lmhead.coral_lmhead_query_sizes(bad)
        assert e.value.code == lmhead.CORAL_ERR_INVALID
    # NULL handle / NULL pointers never reach the device
    assert lib.coral_lmhead_draft(None, None, 1, 1, 1, None, None, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_create(None, ctypes.byref(ok), None, None, None, None, None, None) == lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_destroy(None) == 0


def test_generators_are_seeded_and_prefix_stable():
    cfg = synth.CONFIGS["tiny"]
    a, b = synth.make_hidden(cfg, 4), synth.make_hidden(cfg, 9)
    assert np.array_equal(a, b[:4])
    assert not np.array_equal(synth.make_hidden(cfg, 4, batch=1), a)
    gm = synth.make_group_map(cfg)
    assert np.all(np.bincount(gm, minlength=cfg.N) == cfg.v)
    assert np.array_equal(synth.make_w_gate(cfg), synth.make_w_gate(cfg))
    # bf16 rounding: nearest, ties to even
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5], np.float32)   # 1+2^-8 is a tie -> even (1.0); 1+3*2^-8 -> up
    assert synth.fp32_to_bf16_bits(x).tolist() == [0x3F80, 0x3F80, 0x3F82, 0xC020]
    w = synth.bf16_bits_to_fp32(synth.make_w_vocab(cfg))
    assert abs(float(w.std()) - 0.02) < 1e-3


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    ms, byts = bench.aggregate_over_ranks(dist, 10.0 + rank, 100.0 * (rank + 1))
    q.put((rank, ms, byts, bench.batches_for_rank(rank, world)))
    dist.destroy_process_group()


def test_two_rank_aggregation_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, byts, batches in res:
        assert ms == 11.0 and byts == 300.0          # max of times, sum of bytes
    assert not set(res[0][3]) & set(res[1][3])       # ranks draft for disjoint batches


def test_reference_arm_prints_contract_line():
    import json
    import subprocess
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--rows", "1"], capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stderr
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0


def test_parity_harness_accepts_the_oracle_and_rejects_planted_mistakes():
    """The comparison the GPU tests rely on, exercised on the CPU: the oracle's own result passes; a swapped id,
    an id outside the row's groups, a shifted log-prob and an unsorted row are each reported."""
    from oracle import lmhead_oracle as orc
    from tests import parity_harness as ph
    cfg = synth.CONFIGS["tiny"]
    W, gm, Wg, hb = synth.make_all(cfg)
    ref = orc.draft(W, gm, Wg, hb, cfg.k_groups, cfg.k_tokens)
    good = {"groups": ref.groups.copy(), "gate": ref.gate.astype(np.float32), "logits": ref.logits.astype(np.float32),
            "lse": ref.lse.astype(np.float32), "ids": ref.ids.copy(), "logprobs": ref.logprobs.astype(np.float32)}
    rep = ph.compare(W, gm, Wg, hb, cfg.k_groups, cfg.k_tokens, good)
    assert rep.ok and rep.tie_resolved_ids == 0 and rep.max_logprob_err < 1e-5

    def broken(**kw):
        bad = {k: v.copy() for k, v in good.items()}
        for k, fn in kw.items():
            fn(bad[k])
        return ph.compare(W, gm, Wg, hb, cfg.k_groups, cfg.k_tokens, bad)

    def swap_ids(a):
        a[1, [0, 5]] = a[1, [5, 0]]
    assert any("row 1 pos 0" in e for e in broken(ids=swap_ids).errors)
    inactive = int(np.setdiff1d(np.arange(cfg.V), ref.logit_tokens[2].ravel())[0])

    def foreign_id(a):
        a[2, 3] = inactive
    assert any("not in an active group" in e for e in broken(ids=foreign_id).errors)

    def shift_lp(a):
        a[3, 9] -= 0.01
    assert any("row 3 pos 9: logprob" in e for e in broken(logprobs=shift_lp).errors)

    def unsort(a):
        a[0, [2, 3]] = a[0, [3, 2]]
    assert broken(ids=unsort, logprobs=unsort).errors          # same pairs, wrong order

    def dup(a):
        a[0, 1] = a[0, 0]
    assert any("duplicate" in e for e in broken(ids=dup).errors)
