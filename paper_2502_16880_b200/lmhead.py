"""Thin ctypes binding of the C ABI in include/coral_lmhead.h.

Argument marshalling only: every step of the draft path runs in the CUDA
library.  torch is used for device memory and streams.  There is no CPU
fallback: if the compiled library is missing, loading fails with an error.
The function names are those of the C ABI; `LMHead` is a small convenience
wrapper that owns the device buffers.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# CORAL_LMHEAD_LIB selects another build of the same library (the range-checked one, see build.py)
LIB_PATH = os.environ.get("CORAL_LMHEAD_LIB") or os.path.join(_PKG, "libcoral_lmhead.so")

CORAL_OK = 0
CORAL_ERR_INVALID = -1
CORAL_ERR_GROUPING = -2
CORAL_ERR_CUDA = -3
CORAL_ERR_NOMEM = -4
CORAL_ERR_TIMEOUT = -5
CORAL_ERR_BOUNDS = -6
CORAL_ERR_TOO_LARGE = -7
CORAL_ERR_NONFINITE = -8
CORAL_ROUTE_STATIC_MAX_ROWS = 64
CORAL_OUTPUT_JOINT, CORAL_OUTPUT_FACTORISED, CORAL_OUTPUT_FACTORISED_RENORM = 0, 1, 2
CORAL_PATH_AUTO, CORAL_PATH_STREAM, CORAL_PATH_TCGEN05, CORAL_PATH_SIMT_PLAIN, CORAL_PATH_ADAPTIVE = 0, 1, 2, 3, 4


class coral_lmhead_config(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("H", ctypes.c_int32), ("V", ctypes.c_int32),
                ("n_groups", ctypes.c_int32), ("max_M", ctypes.c_int32), ("max_k_groups", ctypes.c_int32),
                ("max_k_tokens", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class coral_lmhead_stats(ctypes.Structure):
    _fields_ = [("path", ctypes.c_int32), ("M", ctypes.c_int32), ("k_groups", ctypes.c_int32),
                ("k_tokens", ctypes.c_int32), ("groups_touched", ctypes.c_int32),
                ("kernel_launches", ctypes.c_int32), ("weight_bytes", ctypes.c_int64),
                ("algorithmic_bytes", ctypes.c_int64)]


_lib = None
_vp, _i = ctypes.c_void_p, ctypes.c_int

_SIGNATURES = {
    "coral_lmhead_version": (_i, []),
    "coral_lmhead_query_sizes": (_i, [ctypes.POINTER(coral_lmhead_config), ctypes.POINTER(ctypes.c_size_t),
                                      ctypes.POINTER(ctypes.c_size_t)]),
    "coral_lmhead_create": (_i, [ctypes.POINTER(_vp), ctypes.POINTER(coral_lmhead_config), _vp, _vp, _vp, _vp, _vp, _vp]),
    "coral_lmhead_draft": (_i, [_vp, _vp, _i, _i, _i, _vp, _vp, _vp]),
    "coral_lmhead_draft_ex": (_i, [_vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "coral_lmhead_draft_host": (_i, [_vp, _vp, _i, _i, _i, _vp, _vp, _vp]),
    "coral_lmhead_set_group_shard": (_i, [_vp, _i, _i]),
    "coral_lmhead_draft_partial": (_i, [_vp, _vp, _i, _i, _i, _vp, _vp]),
    "coral_lmhead_merge_partials": (_i, [_vp, _i, _i, _i, _vp, _vp, _vp]),
    "coral_lmhead_copy_floor": (_i, [_vp, ctypes.c_longlong, _i, _i, _vp]),
    "coral_lmhead_tc_issue_probe": (_i, [_vp, _i, _i, _i, _i, _vp, _vp]),
    "coral_lmhead_set_hot_groups": (_i, [_vp, _i]),
    "coral_csra_workspace_bytes": (_i, [_i, _i, _i, ctypes.POINTER(ctypes.c_size_t)]),
    "coral_csra_infonce": (_i, [_vp, _vp, _i, _i, _i, ctypes.c_float, _vp, _vp, _vp, _vp, _vp]),
    "coral_csra_status": (_i, [_vp, _vp]),
    "coral_lmhead_selftest_wait_expiry": (_i, [_vp, _vp]),
    "coral_lmhead_set_path": (_i, [_vp, _i]),
    "coral_lmhead_set_output_mode": (_i, [_vp, _i]),
    "coral_lmhead_set_router_mlp": (_i, [_vp, _vp, _vp]),
    "coral_lmhead_set_kernel_timing": (_i, [_vp, _i]),
    "coral_lmhead_head_kernel_ms": (_i, [_vp, ctypes.POINTER(ctypes.c_float)]),
    "coral_lmhead_stage_ms": (_i, [_vp] + [ctypes.POINTER(ctypes.c_float)] * 3),
    "coral_lmhead_status": (_i, [_vp, _vp]),
    "coral_lmhead_last_stats": (_i, [_vp, ctypes.POINTER(coral_lmhead_stats), _vp]),
    "coral_lmhead_route_static": (_i, [_vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp]),
    "coral_tree_expand": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp, _vp]),
    "coral_lmhead_error_string": (ctypes.c_char_p, [_i]),
    "coral_lmhead_destroy": (_i, [_vp]),
}


def load_library(path: str = LIB_PATH):
    """Load the compiled CUDA library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2502_16880_b200.build` "
                "(nvcc, sm_100a). There is no fallback path.")
        lib = ctypes.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


class CoralError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {coral_lmhead_error_string(code)} ({code})")


def _check(code: int, where: str) -> None:
    if code != CORAL_OK:
        raise CoralError(code, where)


def _dev_ptr(t, dtype=None, allow_none=True):
    if t is None:
        if allow_none:
            return None
        raise ValueError("tensor required")
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def make_config(H, V, n_groups, max_M, max_k_groups, max_k_tokens, shard=None) -> coral_lmhead_config:
    """shard = (rank, world): the handle stores and computes only the groups n with n % world == rank."""
    flags = 0 if shard is None else (int(shard[1]) & 0xFF) | ((int(shard[0]) & 0xFF) << 8)
    return coral_lmhead_config(ctypes.sizeof(coral_lmhead_config), H, V, n_groups, max_M, max_k_groups,
                               max_k_tokens, flags)


# ---- functions named as in the C ABI -------------------------------------------------
def coral_lmhead_version() -> int:
    return int(load_library().coral_lmhead_version())


def coral_lmhead_error_string(code: int) -> str:
    return load_library().coral_lmhead_error_string(int(code)).decode()


def coral_lmhead_query_sizes(cfg: coral_lmhead_config):
    pb, wb = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(load_library().coral_lmhead_query_sizes(ctypes.byref(cfg), ctypes.byref(pb), ctypes.byref(wb)),
           "coral_lmhead_query_sizes")
    return int(pb.value), int(wb.value)


def coral_lmhead_create(cfg, W_vocab, group_map_host, W_gate, packed_buf=None, workspace=None, stream=None):
    """W_vocab/W_gate: CUDA bf16 tensors; group_map_host: CPU int32 tensor [V]. Returns an opaque handle."""
    if group_map_host.is_cuda or group_map_host.dtype != torch.int32 or not group_map_host.is_contiguous():
        raise ValueError("group_map_host must be a contiguous CPU int32 tensor")
    if group_map_host.numel() != cfg.V:
        raise ValueError("group_map_host must have V entries")
    h = ctypes.c_void_p()
    _check(load_library().coral_lmhead_create(
        ctypes.byref(h), ctypes.byref(cfg), _dev_ptr(W_vocab, torch.bfloat16, False),
        ctypes.c_void_p(group_map_host.data_ptr()), _dev_ptr(W_gate, torch.bfloat16, False),
        _dev_ptr(packed_buf), _dev_ptr(workspace), _stream_ptr(stream)), "coral_lmhead_create")
    return h


def coral_lmhead_draft(handle, hidden, k_groups, k_tokens, out_ids, out_logprobs, stream=None):
    M = hidden.shape[0]
    _check(load_library().coral_lmhead_draft(
        handle, _dev_ptr(hidden, torch.bfloat16, False), M, int(k_groups), int(k_tokens),
        _dev_ptr(out_ids, torch.int32, False), _dev_ptr(out_logprobs, torch.float32, False), _stream_ptr(stream)),
        "coral_lmhead_draft")


def coral_lmhead_draft_ex(handle, hidden, k_groups, k_tokens, out_ids, out_logprobs, forced_groups=None,
                          out_groups=None, out_gate=None, out_logits=None, out_lse=None, stream=None):
    M = hidden.shape[0]
    _check(load_library().coral_lmhead_draft_ex(
        handle, _dev_ptr(hidden, torch.bfloat16, False), M, int(k_groups), int(k_tokens),
        _dev_ptr(forced_groups, torch.int32), _dev_ptr(out_groups, torch.int32), _dev_ptr(out_gate, torch.float32),
        _dev_ptr(out_logits, torch.float32), _dev_ptr(out_lse, torch.float32),
        _dev_ptr(out_ids, torch.int32, False), _dev_ptr(out_logprobs, torch.float32, False), _stream_ptr(stream)),
        "coral_lmhead_draft_ex")


def coral_lmhead_draft_host(handle, hidden_host, k_groups, k_tokens, out_ids_host, out_logprobs_host, stream=None):
    """Host (ideally pinned) buffers in and out; returns after the results are in host memory."""
    for t in (hidden_host, out_ids_host, out_logprobs_host):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("expected contiguous CPU tensors")
    M = hidden_host.shape[0]
    _check(load_library().coral_lmhead_draft_host(
        handle, ctypes.c_void_p(hidden_host.data_ptr()), M, int(k_groups), int(k_tokens),
        ctypes.c_void_p(out_ids_host.data_ptr()), ctypes.c_void_p(out_logprobs_host.data_ptr()),
        _stream_ptr(stream)), "coral_lmhead_draft_host")


def coral_lmhead_set_group_shard(handle, rank: int, world: int) -> None:
    _check(load_library().coral_lmhead_set_group_shard(handle, int(rank), int(world)), "coral_lmhead_set_group_shard")


def coral_lmhead_draft_partial(handle, hidden, k_groups, k_tokens, out_records, stream=None):
    """out_records: CUDA int32 tensor [M, 2 + 2 * k_tokens] (the per-row record of this GPU's groups)."""
    M = hidden.shape[0]
    if out_records.numel() != M * (2 + 2 * int(k_tokens)):
        raise ValueError("out_records must hold M x (2 + 2 k_tokens) words")
    _check(load_library().coral_lmhead_draft_partial(
        handle, _dev_ptr(hidden, torch.bfloat16, False), M, int(k_groups), int(k_tokens),
        _dev_ptr(out_records, torch.int32, False), _stream_ptr(stream)), "coral_lmhead_draft_partial")


def coral_lmhead_merge_partials(records, k_tokens, out_ids, out_logprobs, stream=None):
    """records: CUDA int32 tensor [world, M, 2 + 2 * k_tokens], rank-major as an all-gather leaves it."""
    world, M = records.shape[0], records.shape[1]
    _check(load_library().coral_lmhead_merge_partials(
        _dev_ptr(records, torch.int32, False), world, M, int(k_tokens), _dev_ptr(out_ids, torch.int32, False),
        _dev_ptr(out_logprobs, torch.float32, False), _stream_ptr(stream)), "coral_lmhead_merge_partials")


def draft_vocab_sharded(handle, hidden, k_groups, k_tokens, out_ids, out_logprobs, group=None, records=None,
                        gathered=None):
    """One vocab-sharded draft step on this rank of `group` (torch.distributed): this GPU's record per row,
    one all-gather of the records, the merge.  The handle must have been given this rank's shard with
    coral_lmhead_set_group_shard.  `records` [M, W] and `gathered` [world, M, W] (W = 2 + 2 k_tokens, int32)
    may be passed in to avoid allocating per call."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    M, W = hidden.shape[0], 2 + 2 * int(k_tokens)
    if records is None:
        records = torch.empty((M, W), dtype=torch.int32, device=hidden.device)
    if gathered is None:
        gathered = torch.empty((world, M, W), dtype=torch.int32, device=hidden.device)
    coral_lmhead_draft_partial(handle, hidden, k_groups, k_tokens, records)
    dist.all_gather_into_tensor(gathered.view(world * M, W), records.view(M, W), group=group)   # rank-major rows
    coral_lmhead_merge_partials(gathered, k_tokens, out_ids, out_logprobs)


def coral_lmhead_set_output_mode(handle, mode: int) -> None:
    _check(load_library().coral_lmhead_set_output_mode(handle, int(mode)), "coral_lmhead_set_output_mode")


def coral_lmhead_set_router_mlp(handle, W1=None, stream=None) -> None:
    """W1: CUDA bf16 [H, H] tensor of Eq. 7's first router layer, or None for the single-matrix gate."""
    _check(load_library().coral_lmhead_set_router_mlp(handle, _dev_ptr(W1, torch.bfloat16), _stream_ptr(stream)),
           "coral_lmhead_set_router_mlp")


def coral_lmhead_copy_floor(handle, nbytes: int, stream=None, in_flight: int = 0, repeats: int = 1) -> None:
    """Measurement aid: a do-nothing stream of the first `nbytes` of the packed head, `repeats` sweeps with
    `in_flight` 16 KiB copies outstanding per SM (0 = default); time it with events."""
    _check(load_library().coral_lmhead_copy_floor(handle, int(nbytes), int(in_flight), int(repeats),
                                                  _stream_ptr(stream)), "coral_lmhead_copy_floor")


def coral_lmhead_tc_issue_probe(handle, n: int, per_commit: int, issuers: int, rounds: int, out_ns, stream=None) -> None:
    """out_ns: CUDA int64 tensor of two words (issue time, completion time in ns of the first pair's first issuer)."""
    _check(load_library().coral_lmhead_tc_issue_probe(handle, int(n), int(per_commit), int(issuers), int(rounds),
                                                      _dev_ptr(out_ns, torch.int64, allow_none=False),
                                                      _stream_ptr(stream)), "coral_lmhead_tc_issue_probe")


def coral_csra_workspace_bytes(n: int, views: int, D: int) -> int:
    b = ctypes.c_size_t(0)
    _check(load_library().coral_csra_workspace_bytes(int(n), int(views), int(D), ctypes.byref(b)), "coral_csra_workspace_bytes")
    return int(b.value)


def coral_csra_infonce(Q, K, views, tau, workspace, out_loss, out_row_loss=None, out_logits=None, stream=None):
    """Q [n, D], K [views * n, D] CUDA bf16; workspace: CUDA uint8 tensor of coral_csra_workspace_bytes(n, views, D);
    out_loss [1] f32, out_row_loss [n] f32 or None, out_logits [n, views * n] f32 or None."""
    n, D = Q.shape
    if K.shape[0] != int(views) * n or K.shape[1] != D:
        raise ValueError("K must be [views * n, D]")
    _check(load_library().coral_csra_infonce(
        _dev_ptr(Q, torch.bfloat16, False), _dev_ptr(K, torch.bfloat16, False), n, int(views), D, float(tau),
        _dev_ptr(workspace, torch.uint8, False), _dev_ptr(out_row_loss, torch.float32),
        _dev_ptr(out_loss, torch.float32, False), _dev_ptr(out_logits, torch.float32), _stream_ptr(stream)),
        "coral_csra_infonce")


def coral_csra_status(workspace, stream=None) -> int:
    return int(load_library().coral_csra_status(_dev_ptr(workspace, torch.uint8, False), _stream_ptr(stream)))


def coral_lmhead_set_hot_groups(handle, n_hot: int) -> None:
    _check(load_library().coral_lmhead_set_hot_groups(handle, int(n_hot)), "coral_lmhead_set_hot_groups")


def coral_lmhead_selftest_wait_expiry(handle, stream=None) -> None:
    """Runs the kernels' bounded wait on a barrier nothing completes; coral_lmhead_status then reports a timeout."""
    _check(load_library().coral_lmhead_selftest_wait_expiry(handle, _stream_ptr(stream)),
           "coral_lmhead_selftest_wait_expiry")


def coral_lmhead_set_path(handle, path: int) -> None:
    _check(load_library().coral_lmhead_set_path(handle, int(path)), "coral_lmhead_set_path")


def coral_lmhead_set_kernel_timing(handle, on: bool) -> None:
    _check(load_library().coral_lmhead_set_kernel_timing(handle, int(bool(on))), "coral_lmhead_set_kernel_timing")


def coral_lmhead_head_kernel_ms(handle) -> float:
    ms = ctypes.c_float(0.0)
    _check(load_library().coral_lmhead_head_kernel_ms(handle, ctypes.byref(ms)), "coral_lmhead_head_kernel_ms")
    return float(ms.value)


def coral_lmhead_stage_ms(handle):
    """(route_ms, head_ms, merge_ms) of the last call made with kernel timing on."""
    a, b, c = ctypes.c_float(0.0), ctypes.c_float(0.0), ctypes.c_float(0.0)
    _check(load_library().coral_lmhead_stage_ms(handle, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "coral_lmhead_stage_ms")
    return float(a.value), float(b.value), float(c.value)


def coral_lmhead_status(handle, stream=None) -> int:
    return int(load_library().coral_lmhead_status(handle, _stream_ptr(stream)))


def coral_lmhead_last_stats(handle, stream=None) -> coral_lmhead_stats:
    s = coral_lmhead_stats()
    _check(load_library().coral_lmhead_last_stats(handle, ctypes.byref(s), _stream_ptr(stream)),
           "coral_lmhead_last_stats")
    return s


def coral_lmhead_route_static(W_gate, hidden, k_groups, out_groups, out_gate=None, stream=None) -> None:
    """Gate scores and top-k groups without a handle and without any allocation inside the library
    (for callers that are not allowed to allocate device memory); at most CORAL_ROUTE_STATIC_MAX_ROWS rows.
    The tensors passed in are the only memory the caller provides; scratch is built into the library."""
    N, H = W_gate.shape
    M = hidden.shape[0]
    _check(load_library().coral_lmhead_route_static(
        _dev_ptr(W_gate, torch.bfloat16, False), _dev_ptr(hidden, torch.bfloat16, False), M, H, N, int(k_groups),
        _dev_ptr(out_groups, torch.int32, False), _dev_ptr(out_gate, torch.float32), _stream_ptr(stream)),
        "coral_lmhead_route_static")


def coral_tree_expand(parent_scores, cand_ids, cand_logprobs, K, out_parent, out_token, out_score, stream=None):
    """parent_scores [n_seq, nodes] f32; cand_ids / cand_logprobs [n_seq, nodes, k_tokens] (or None); outputs [n_seq, K]."""
    n_seq, nodes = parent_scores.shape
    k_tokens = 1 if cand_logprobs is None else cand_logprobs.shape[-1]
    _check(load_library().coral_tree_expand(
        _dev_ptr(parent_scores, torch.float32, False), _dev_ptr(cand_ids, torch.int32), _dev_ptr(cand_logprobs, torch.float32),
        n_seq, nodes, k_tokens, int(K), _dev_ptr(out_parent, torch.int32, False), _dev_ptr(out_token, torch.int32, False),
        _dev_ptr(out_score, torch.float32, False), _stream_ptr(stream)), "coral_tree_expand")


def coral_lmhead_destroy(handle) -> None:
    _check(load_library().coral_lmhead_destroy(handle), "coral_lmhead_destroy")


# ---- convenience wrapper ---------------------------------------------------------------
class LMHead:
    """Owns the packed weights and workspace (torch allocations) of one handle."""

    def __init__(self, W_vocab, group_map_host, W_gate, max_M, max_k_groups, max_k_tokens=10, shard=None):
        V, H = W_vocab.shape
        N = W_gate.shape[0]
        self.cfg = make_config(H, V, N, max_M, max_k_groups, max_k_tokens, shard)
        pb, wb = coral_lmhead_query_sizes(self.cfg)
        dev = W_vocab.device
        self.packed = torch.empty(pb, dtype=torch.uint8, device=dev)
        self.workspace = torch.empty(wb, dtype=torch.uint8, device=dev)
        self.handle = coral_lmhead_create(self.cfg, W_vocab, group_map_host, W_gate, self.packed, self.workspace)
        self.device = dev

    def draft(self, hidden, k_groups, k_tokens, taps=False, forced_groups=None, stream=None):
        M = hidden.shape[0]
        dev = self.device
        ids = torch.empty((M, k_tokens), dtype=torch.int32, device=dev)
        lps = torch.empty((M, k_tokens), dtype=torch.float32, device=dev)
        if not taps and forced_groups is None:
            coral_lmhead_draft(self.handle, hidden, k_groups, k_tokens, ids, lps, stream)
            return ids, lps
        v = self.cfg.V // self.cfg.n_groups
        out = {
            "groups": torch.empty((M, k_groups), dtype=torch.int32, device=dev),
            "gate": torch.empty((M, self.cfg.n_groups), dtype=torch.float32, device=dev),
            "logits": torch.empty((M, k_groups, v), dtype=torch.float32, device=dev),
            "lse": torch.empty((M,), dtype=torch.float32, device=dev),
        }
        coral_lmhead_draft_ex(self.handle, hidden, k_groups, k_tokens, ids, lps, forced_groups=forced_groups,
                              out_groups=out["groups"], out_gate=out["gate"], out_logits=out["logits"],
                              out_lse=out["lse"], stream=stream)
        out["ids"], out["logprobs"] = ids, lps
        return out

    def set_path(self, path):
        coral_lmhead_set_path(self.handle, path)

    def status(self):
        return coral_lmhead_status(self.handle)

    def stats(self):
        return coral_lmhead_last_stats(self.handle)

    def close(self):
        if self.handle is not None:
            coral_lmhead_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
