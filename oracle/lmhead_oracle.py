"""ctypes loader for the CPU oracle (oracle/lmhead_oracle.c).

TEST INFRASTRUCTURE: imported only by the tests, the smoke check and the
bench's CPU-baseline leg.  It marshals numpy arrays to the C function and adds
no arithmetic of its own.  The product path never imports this module.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lmhead_oracle.c")
_LIB = os.path.join(_HERE, "liblmhead_oracle.so")
_lib = None


def build(force: bool = False, src: str = _SRC, out: str = _LIB) -> str:
    """Compile the oracle with gcc (no fast-math: fp64 sums in source order)."""
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-Wall", "-o", out, src, "-lm"]
        subprocess.run(cmd, check=True)
    return out


def _load(path: str | None = None):
    global _lib
    if path is not None:
        return _bind(ctypes.CDLL(path))
    if _lib is None:
        _lib = _bind(ctypes.CDLL(build()))
    return _lib


def _bind(lib):
    p = ctypes.c_void_p
    i = ctypes.c_int
    lib.coral_oracle_draft.restype = i
    lib.coral_oracle_draft.argtypes = [p, p, p, p, p, i, i, i, i, i, i, p, p, i, p, p, p, p, p, p, p, p, p]
    lib.coral_oracle_threads.restype = i
    return lib


def threads() -> int:
    return int(_load().coral_oracle_threads())


@dataclass
class OracleResult:
    gate: np.ndarray          # [M, N] f64
    groups: np.ndarray        # [M, k_groups] i32, selection order
    logits: np.ndarray        # [M, k_groups, v] f64, slot layout
    logit_tokens: np.ndarray  # [M, k_groups, v] i32
    lse: np.ndarray           # [M] f64
    group_lse: np.ndarray     # [M, k_groups] f64
    log_router: np.ndarray    # [M, N] f64
    ids: np.ndarray           # [M, k_tokens] i32
    logprobs: np.ndarray      # [M, k_tokens] f64


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def draft(W_vocab, group_map, W_gate, hidden, k_groups, k_tokens, *, W1=None, forced_groups=None,
          gate_override=None, factorised=False, want_logits=True, lib_path=None) -> OracleResult:
    """Run the oracle.  bf16 tensors are uint16 bit patterns (numpy).  factorised: False/0 joint log-softmax,
    True/1 Eq. 8, 2 Eq. 8 with p_router renormalised over the selected groups."""
    lib = _load(lib_path)
    W_vocab = np.ascontiguousarray(W_vocab, dtype=np.uint16)
    W_gate = np.ascontiguousarray(W_gate, dtype=np.uint16)
    hidden = np.ascontiguousarray(hidden, dtype=np.uint16)
    group_map = np.ascontiguousarray(group_map, dtype=np.int32)
    V, H = W_vocab.shape
    N = W_gate.shape[0]
    M = hidden.shape[0]
    if W_gate.shape[1] != H or hidden.shape[1] != H or group_map.shape != (V,):
        raise ValueError("shape mismatch")
    if W1 is not None:
        W1 = np.ascontiguousarray(W1, dtype=np.uint16)
        if W1.shape != (H, H):
            raise ValueError("W1 must be [H, H]")
    if forced_groups is not None:
        forced_groups = np.ascontiguousarray(forced_groups, dtype=np.int32)
        if forced_groups.shape != (M, k_groups):
            raise ValueError("forced_groups must be [M, k_groups]")
    if gate_override is not None:
        gate_override = np.ascontiguousarray(gate_override, dtype=np.float64)
        if gate_override.shape != (M, N):
            raise ValueError("gate_override must be [M, N]")
    v = V // max(N, 1)
    res = OracleResult(
        gate=np.zeros((M, N)), groups=np.zeros((M, k_groups), np.int32),
        logits=np.zeros((M, k_groups, v)) if want_logits else None,
        logit_tokens=np.zeros((M, k_groups, v), np.int32) if want_logits else None,
        lse=np.zeros(M), group_lse=np.zeros((M, k_groups)), log_router=np.zeros((M, N)),
        ids=np.zeros((M, k_tokens), np.int32), logprobs=np.zeros((M, k_tokens)))
    rc = lib.coral_oracle_draft(
        _ptr(W_vocab), _ptr(group_map), _ptr(W_gate), _ptr(W1), _ptr(hidden), H, V, N, M,
        int(k_groups), int(k_tokens), _ptr(forced_groups), _ptr(gate_override), int(factorised),
        _ptr(res.gate), _ptr(res.groups), _ptr(res.logits), _ptr(res.logit_tokens), _ptr(res.lse),
        _ptr(res.group_lse), _ptr(res.log_router), _ptr(res.ids), _ptr(res.logprobs))
    if rc != 0:
        raise ValueError(f"coral_oracle_draft failed with status {rc}")
    return res
