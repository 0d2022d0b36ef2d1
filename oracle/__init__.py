"""ctypes front end of the CPU oracle (moe_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests/, the smoke check and the benchmark's CPU-baseline / reference legs may
import this package.  It never imports the CUDA package, and vice versa.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "_moe_oracle.so")
_SRC = os.path.join(_HERE, "moe_oracle.c")
_lib = None


def build(force: bool = False) -> str:
    """gcc -O2 -fopenmp; no -ffast-math, so only the declared simd reductions reorder sums."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fopenmp-simd", "-shared", "-fPIC",
                               "-o", _SO, _SRC, "-lm"])
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.oracle_route.restype = ci
        lib.oracle_route.argtypes = [vp, ci, ci, ci, vp, vp]
        lib.oracle_permute.restype = ci
        lib.oracle_permute.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp]
        lib.oracle_expert_ffn.restype = None
        lib.oracle_expert_ffn.argtypes = [vp, vp, vp, ci, ci, ci, vp, vp]
        lib.oracle_moe_layer.restype = ci
        lib.oracle_moe_layer.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci] + [vp] * 10
        lib.oracle_moe_tokens.restype = ci
        lib.oracle_moe_tokens.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, ci, vp]
        i64p = ctypes.POINTER(ctypes.c_int64)
        lib.oracle_ep_descriptors.restype = ci
        lib.oracle_ep_descriptors.argtypes = [vp, ci, ci, ci, ci, ci, i64p, i64p, i64p]
        lib.oracle_permute_ep.restype = ci
        lib.oracle_permute_ep.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp, vp]
        lib.oracle_moe_tokens_ep.restype = ci
        lib.oracle_moe_tokens_ep.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, vp, ci, vp]
        lib.oracle_num_threads.restype = ci
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


@dataclass
class Routing:
    idx: np.ndarray       # [T,k] int32, descending logit, ties to the lowest index
    gates: np.ndarray     # [T,k] float32, softmax over the selected k
    counts: np.ndarray    # [E+S] int32
    offsets: np.ndarray   # [E+S+1] int32
    row_of: np.ndarray    # [T,k+S] int32
    token_of: np.ndarray  # [P] int32


def route(logits: np.ndarray, k: int):
    logits = _c(logits, np.float32)
    T, E = logits.shape
    idx = np.empty((T, k), np.int32)
    gates = np.empty((T, k), np.float32)
    rc = _load().oracle_route(_p(logits), T, E, k, _p(idx), _p(gates))
    if rc:
        raise ValueError(f"oracle_route failed: {rc} (-1 = non-finite logit, -2 = bad k)")
    return idx, gates


def permute(idx: np.ndarray, E: int, S: int = 0):
    idx = _c(idx, np.int32)
    T, k = idx.shape
    counts = np.empty(E + S, np.int32)
    offsets = np.empty(E + S + 1, np.int32)
    row_of = np.empty((T, k + S), np.int32)
    token_of = np.empty(T * (k + S), np.int32)
    rc = _load().oracle_permute(_p(idx), T, E, k, S, _p(counts), _p(offsets), _p(row_of),
                                _p(token_of))
    if rc:
        raise ValueError(f"oracle_permute failed: {rc}")
    return counts, offsets, row_of, token_of


def routing(logits: np.ndarray, k: int, S: int = 0) -> Routing:
    idx, gates = route(logits, k)
    counts, offsets, row_of, token_of = permute(idx, logits.shape[1], S)
    return Routing(idx, gates, counts, offsets, row_of, token_of)


def expert_ffn(x_row_bf16: np.ndarray, gate_up_e: np.ndarray, down_e: np.ndarray,
               acc_double: bool = False):
    """One row through one expert: returns (h [I], y [H]) fp32."""
    x_row_bf16 = _c(x_row_bf16, np.uint16)
    gate_up_e = _c(gate_up_e, np.uint16)
    down_e = _c(down_e, np.uint16)
    H = x_row_bf16.shape[0]
    I = down_e.shape[1]
    assert gate_up_e.shape == (2 * I, H) and down_e.shape == (H, I)
    h = np.empty(I, np.float32)
    y = np.empty(H, np.float32)
    _load().oracle_expert_ffn(_p(x_row_bf16), _p(gate_up_e), _p(down_e), H, I, int(acc_double),
                              _p(h), _p(y))
    return h, y


@dataclass
class LayerResult:
    routing: Routing
    out: np.ndarray                 # [T,H] fp32
    xe: Optional[np.ndarray] = None  # [P,H]
    h: Optional[np.ndarray] = None   # [P,I]
    y: Optional[np.ndarray] = None   # [P,H]


def moe_layer(x, logits, gate_up, down, k: int, S: int = 0, acc_double: bool = False,
              keep_intermediates: bool = False) -> LayerResult:
    """All five stages with materialised intermediates (small layers only)."""
    x = _c(x, np.uint16)
    logits = _c(logits, np.float32)
    gate_up = _c(gate_up, np.uint16)
    down = _c(down, np.uint16)
    T, H = x.shape
    E = logits.shape[1]
    EE, twoI, _ = gate_up.shape
    I = twoI // 2
    assert EE == E + S and down.shape == (EE, H, I)
    P = T * (k + S)
    idx = np.empty((T, k), np.int32)
    gates = np.empty((T, k), np.float32)
    counts = np.empty(EE, np.int32)
    offsets = np.empty(EE + 1, np.int32)
    row_of = np.empty((T, k + S), np.int32)
    token_of = np.empty(P, np.int32)
    out = np.empty((T, H), np.float32)
    xe = np.empty((P, H), np.float32) if keep_intermediates else None
    hb = np.empty((P, I), np.float32) if keep_intermediates else None
    y = np.empty((P, H), np.float32) if keep_intermediates else None
    rc = _load().oracle_moe_layer(_p(x), _p(logits), _p(gate_up), _p(down), T, H, I, E, k, S,
                                  int(acc_double), _p(idx), _p(gates), _p(counts), _p(offsets),
                                  _p(row_of), _p(token_of), _p(out), _p(xe), _p(hb), _p(y))
    if rc:
        raise ValueError(f"oracle_moe_layer failed: {rc}")
    return LayerResult(Routing(idx, gates, counts, offsets, row_of, token_of), out, xe, hb, y)


def moe_tokens(x, logits, gate_up, down, k: int, tokens, S: int = 0,
               acc_double: bool = False) -> np.ndarray:
    """out rows [n,H] fp32 of the listed tokens, each from the definition (no permutation)."""
    x = _c(x, np.uint16)
    logits = _c(logits, np.float32)
    gate_up = _c(gate_up, np.uint16)
    down = _c(down, np.uint16)
    tokens = _c(tokens, np.int32)
    T, H = x.shape
    E = logits.shape[1]
    EE, twoI, _ = gate_up.shape
    I = twoI // 2
    assert EE == E + S and down.shape == (EE, H, I)
    assert tokens.min(initial=0) >= 0 and tokens.max(initial=0) < T
    out = np.empty((tokens.shape[0], H), np.float32)
    rc = _load().oracle_moe_tokens(_p(x), _p(logits), _p(gate_up), _p(down), H, I, E, k, S,
                                   int(acc_double), _p(tokens), tokens.shape[0], _p(out))
    if rc:
        raise ValueError(f"oracle_moe_tokens failed: {rc}")
    return out


# ---------------------------------------------------------------------------- one EP rank's share

def ep_descriptors(idx: np.ndarray, E: int, ep_rank: int, ep_size: int):
    """(X_local, X_in, X_in_uniq) of Section 3.1 for one rank."""
    idx = _c(idx, np.int32)
    T, k = idx.shape
    a, b, c = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    rc = _load().oracle_ep_descriptors(_p(idx), T, E, k, ep_rank, ep_size, ctypes.byref(a), ctypes.byref(b),
                                       ctypes.byref(c))
    if rc:
        raise ValueError(f"oracle_ep_descriptors failed: {rc}")
    return a.value, b.value, c.value


def routing_ep(logits: np.ndarray, k: int, ep_rank: int, ep_size: int) -> Routing:
    """Global routing, permutation restricted to the rank's experts (row -1 for the other slots)."""
    idx, gates = route(logits, k)
    T, E = logits.shape
    counts = np.empty(E, np.int32)
    offsets = np.empty(E + 1, np.int32)
    row_of = np.empty((T, k), np.int32)
    token_of = np.full(T * k, -1, np.int32)
    rc = _load().oracle_permute_ep(_p(idx), T, E, k, ep_rank, ep_size, _p(counts), _p(offsets), _p(row_of),
                                   _p(token_of))
    if rc:
        raise ValueError(f"oracle_permute_ep failed: {rc}")
    return Routing(idx, gates, counts, offsets, row_of, token_of[:int(offsets[-1])].copy())


def moe_tokens_ep(x, logits, gate_up, down, k: int, tokens, ep_rank: int, ep_size: int,
                  acc_double: bool = False) -> np.ndarray:
    """Partial output rows [n,H] of the listed tokens for one rank (sum over its local experts)."""
    x = _c(x, np.uint16)
    logits = _c(logits, np.float32)
    gate_up = _c(gate_up, np.uint16)
    down = _c(down, np.uint16)
    tokens = _c(tokens, np.int32)
    T, H = x.shape
    E = logits.shape[1]
    I = gate_up.shape[1] // 2
    out = np.empty((tokens.shape[0], H), np.float32)
    rc = _load().oracle_moe_tokens_ep(_p(x), _p(logits), _p(gate_up), _p(down), H, I, E, k, ep_rank, ep_size,
                                      int(acc_double), _p(tokens), tokens.shape[0], _p(out))
    if rc:
        raise ValueError(f"oracle_moe_tokens_ep failed: {rc}")
    return out
