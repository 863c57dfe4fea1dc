"""The range-checked build (-DCORAL_CHECK_BOUNDS) stands in for a memory checker: every index the kernels
compute from the router's output is compared with the capacity of the array it indexes, and a violation sets
CORAL_ERR_BOUNDS instead of touching memory.  Here the draft step runs on that build, in a process of its
own (the library is chosen when the package is first imported), over shapes that exercise every kernel -
all three head paths, ragged groups, several passes per group, wide tensor-core entries, the many-row mode of
the tensor-core kernel, forced groups, the
two-layer router, vocab sharding - and must come out with status 0 and the oracle's results."""
import os
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = textwrap.dedent("""
    import numpy as np, torch
    from paper_2502_16880_b200 import lmhead, synth, build
    from tests import parity_harness as ph
    assert lmhead.LIB_PATH == build.LIB_CHECKED
    torch.cuda.set_device(0)
    shapes = [  # H, v, N, M, kg, kt, path
        (256, 256, 16, 4, 4, 10, lmhead.CORAL_PATH_STREAM), (256, 256, 16, 40, 16, 7, lmhead.CORAL_PATH_STREAM),
        (256, 256, 16, 128, 8, 10, lmhead.CORAL_PATH_STREAM), (768, 300, 6, 9, 2, 10, lmhead.CORAL_PATH_STREAM),
        (328, 300, 6, 13, 3, 5, lmhead.CORAL_PATH_SIMT_PLAIN), (256, 256, 16, 4, 4, 10, lmhead.CORAL_PATH_SIMT_PLAIN),
        (256, 256, 16, 200, 4, 10, lmhead.CORAL_PATH_TCGEN05), (256, 256, 16, 300, 8, 10, lmhead.CORAL_PATH_TCGEN05),
        (320, 300, 6, 400, 3, 5, lmhead.CORAL_PATH_TCGEN05), (256, 256, 16, 1200, 8, 10, lmhead.CORAL_PATH_TCGEN05),
        (256, 256, 16, 60, 16, 10, lmhead.CORAL_PATH_AUTO), (256, 256, 16, 100, 4, 10, lmhead.CORAL_PATH_ADAPTIVE),
        (4096, 300, 16, 1600, 8, 10, lmhead.CORAL_PATH_TCGEN05),      # 105 MB of gathered rows: batches taken in turn
    ]
    for H, v, N, M, kg, kt, path in shapes:
        cfg = synth.HeadConfig("chk", H=H, V=v * N, N=N, k_groups=kg, k_tokens=kt, M=M, seed=11, w_std=0.05)
        W, gm, Wg, hb = synth.make_all(cfg)
        head = lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), ph.to_dev_bf16(Wg), M, kg, 32)
        head.set_path(path)
        out = ph.gpu_draft_numpy(head, hb, kg, kt)
        assert head.status() == 0, (H, v, N, M, kg, kt, path)
        rows = np.unique(np.linspace(0, M - 1, min(M, 24)).astype(int))
        rep = ph.compare(W, gm, Wg, hb[rows], kg, kt, {k: a[rows] for k, a in out.items()})
        assert rep.ok, rep.errors
        if path == lmhead.CORAL_PATH_STREAM and M <= 40:        # vocab sharding, both ranks of a world of two
            for rank in range(2):
                lmhead.coral_lmhead_set_group_shard(head.handle, rank, 2)
                rec = torch.empty((M, 2 + 2 * kt), dtype=torch.int32, device="cuda")
                lmhead.coral_lmhead_draft_partial(head.handle, ph.to_dev_bf16(hb), kg, kt, rec)
                torch.cuda.synchronize()
                assert head.status() == 0
            lmhead.coral_lmhead_set_group_shard(head.handle, 0, 1)
        head.close()
    print("checked build: all cases status 0")
""")


@pytest.mark.gpu
def test_draft_step_on_the_range_checked_build():
    from paper_2502_16880_b200 import build
    lib = build.build_library(checked=True)
    env = dict(os.environ, CORAL_LMHEAD_LIB=lib, PYTHONPATH=ROOT)
    r = subprocess.run([sys.executable, "-c", CASES], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "all cases status 0" in r.stdout


def test_checked_build_exports_the_same_symbols():
    """CPU: the checked library builds and exports every entry point the binding declares."""
    import ctypes
    from paper_2502_16880_b200 import build, lmhead
    lib = ctypes.CDLL(build.build_library(checked=True))
    for name in lmhead._SIGNATURES:
        assert hasattr(lib, name), name
