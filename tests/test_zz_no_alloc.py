"""coral_lmhead_route_static: the router step for callers that may not allocate.

Some users of this library run where device allocation is forbidden: a server
whose memory pool is sized once and never grows, a plug-in that receives a
stream and tensors but no allocator, a latency-critical section that cannot
afford cudaMalloc's device-wide synchronisation.  They cannot create a handle,
because a handle needs a workspace.  The entry point tested here takes only the
inputs and outputs; its scratch is a fixed array built into the library.

The check: through the C ABI, its groups and gate scores must equal those of the
ordinary entry point (coral_lmhead_draft_ex with the groups/gate taps) within
the tolerance the parity tests use, on two calls in a row with different rows
(the array keeps the first call's contents, so the second call shows that stale
data is harmless), and oversized requests must be refused with a clear code.
The same outputs are also held against the CPU oracle directly (scores within
the tolerance, groups equal except where the oracle's own scores tie).
This file sorts last on purpose: a run that stops at the first failure has
already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import lmhead_oracle as orc
from paper_2502_16880_b200 import lmhead, synth
from tests import parity_harness as ph

pytestmark = pytest.mark.gpu


def _existing_entry_point(head, hd, k_groups):
    out = head.draft(hd, k_groups, 5, taps=True)
    torch.cuda.synchronize()
    return out["groups"].cpu().numpy(), out["gate"].cpu().numpy()


def test_route_static_matches_existing_entry_point_twice():
    cfg = synth.CONFIGS["tiny"]
    W, gm, Wg = synth.make_w_vocab(cfg), synth.make_group_map(cfg), synth.make_w_gate(cfg)
    Wg_d = ph.to_dev_bf16(Wg)
    head = lmhead.LMHead(ph.to_dev_bf16(W), torch.from_numpy(gm), Wg_d, 64, cfg.N, 10)
    # second call: fewer rows and a different k, so leftovers of the first call lie beyond what it rewrites
    for M, k_groups, batch in [(37, 4, 0), (5, 7, 1)]:
        hd = ph.to_dev_bf16(synth.make_hidden(cfg, M, batch=batch))
        want_groups, want_gate = _existing_entry_point(head, hd, k_groups)
        # outputs are allocated by the caller, before the call; the call itself allocates nothing
        groups = torch.full((M, k_groups), -1, dtype=torch.int32, device="cuda")
        gate = torch.zeros((M, cfg.N), dtype=torch.float32, device="cuda")
        lmhead.coral_lmhead_route_static(Wg_d, hd, k_groups, groups, gate)
        torch.cuda.synchronize()
        got_gate = gate.cpu().numpy()
        assert np.all(ph.close(got_gate, want_gate)), np.abs(got_gate - want_gate).max()
        got_groups = groups.cpu().numpy()
        assert np.array_equal(got_groups, want_groups)
        # and against the oracle itself (router part of the step: Eq. 7's scores, top-n of Section 3.3)
        hb = synth.make_hidden(cfg, M, batch=batch)
        ref = orc.draft(W, gm, Wg, hb, k_groups, 1, want_logits=False)
        assert np.all(ph.close(got_gate, ref.gate)), np.abs(got_gate - ref.gate).max()
        for m in range(M):
            for s in range(k_groups):
                a, b = int(got_groups[m, s]), int(ref.groups[m, s])
                assert a == b or ph.close(ref.gate[m, a], ref.gate[m, b]), (m, s, a, b)
            assert len(set(got_groups[m].tolist())) == k_groups
    head.close()


def test_route_static_rejects_sizes_beyond_its_scratch():
    cfg = synth.CONFIGS["tiny"]
    lib = lmhead.load_library()
    Wg_d = ph.to_dev_bf16(synth.make_w_gate(cfg))
    M = lmhead.CORAL_ROUTE_STATIC_MAX_ROWS + 1
    hd = ph.to_dev_bf16(synth.make_hidden(cfg, M))
    groups = torch.empty((M, 2), dtype=torch.int32, device="cuda")
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    rc = lib.coral_lmhead_route_static(p(Wg_d), p(hd), M, cfg.H, cfg.N, 2, p(groups), None, None)
    assert rc == lmhead.CORAL_ERR_TOO_LARGE
    assert "scratch" in lmhead.coral_lmhead_error_string(rc)
    assert lib.coral_lmhead_route_static(p(Wg_d), p(hd), 4, cfg.H, cfg.N, cfg.N + 1, p(groups), None, None) == \
        lmhead.CORAL_ERR_INVALID
    assert lib.coral_lmhead_route_static(None, p(hd), 4, cfg.H, cfg.N, 2, p(groups), None, None) == \
        lmhead.CORAL_ERR_INVALID
    torch.cuda.synchronize()
