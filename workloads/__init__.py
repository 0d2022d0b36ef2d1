"""Seeded synthetic MoE-layer workloads (inputs only; no arithmetic of the method).

The paper measures on routing traces of trained models over public prompt sets
(its "Workloads" paragraph and Table 1).  Neither the data nor the weights are
available offline, so these generators stand in for them: same shapes (Table 1
rows where the shape is one of the paper's), bf16 activations ~N(0,1), bf16
weights ~N(0,0.02), fp32 router logits ~N(0,1), optionally plus a per-expert
bias that skews the expert load in a Zipf-like way.

Both the CPU oracle's tests and the CUDA path's tests draw their inputs from
here, so the two sides see bit-identical arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field, replace
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "_gen.so")
_SRC = os.path.join(_HERE, "gen.c")
_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into _gen.so next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"])
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        lib.wl_hash.restype = ctypes.c_uint64
        lib.wl_hash.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        for fn in (lib.wl_normal_f32, lib.wl_normal_bf16):
            fn.restype = None
            fn.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64,
                           ctypes.c_double, ctypes.c_double]
        lib.wl_normal_bf16_range.restype = None
        lib.wl_normal_bf16_range.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_uint64,
                                             ctypes.c_double, ctypes.c_double]
        lib.wl_add_row_bias_f32.restype = None
        lib.wl_add_row_bias_f32.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                            ctypes.c_void_p]
        _lib = lib
    return _lib


# --------------------------------------------------------------------------- configs

@dataclass(frozen=True)
class MoEConfig:
    """Shape of one synthetic MoE layer.  P = T*(k+S) token-expert rows."""
    name: str
    cfg_id: int          # enters the tensor seeds
    T: int               # tokens
    H: int               # hidden size
    I: int               # expert FFN width (SwiGLU: gate_up is [2I,H], down is [H,I])
    E: int               # routed experts
    k: int               # top-k
    S: int = 0           # always-on shared experts
    zipf_s: Optional[float] = None          # fixed skew exponent (None = uniform routing)
    zipf_range: Optional[tuple] = None      # per-layer skew drawn from U[lo,hi]
    layers: int = 1
    base_seed: int = 0

    @property
    def P(self) -> int:
        return self.T * (self.k + self.S)

    def with_T(self, T: int) -> "MoEConfig":
        return replace(self, T=T, name=f"{self.name}_T{T}")


CONFIGS: Dict[str, MoEConfig] = {
    # tiny layer the oracle evaluates in full
    "c1_tiny": MoEConfig("c1_tiny", 1, T=256, H=512, I=1024, E=8, k=2),
    # Mixtral-8x7B-shaped prefill layer
    "c2_mixtral": MoEConfig("c2_mixtral", 2, T=4096, H=4096, I=14336, E=8, k=2),
    # Qwen3-30B-A3B-shaped layer (Table 1 row), Zipf(1.2)-biased routing
    "c3_qwen3_30b": MoEConfig("c3_qwen3_30b", 3, T=8192, H=2048, I=768, E=128, k=8, zipf_s=1.2),
    # DeepSeek-V2-Lite-shaped layer (Table 1 row) with 2 shared experts, decode-like batches
    "c4_dsv2lite_T64": MoEConfig("c4_dsv2lite_T64", 4, T=64, H=2048, I=1408, E=64, k=6, S=2),
    "c4_dsv2lite_T256": MoEConfig("c4_dsv2lite_T256", 4, T=256, H=2048, I=1408, E=64, k=6, S=2),
    "c4_dsv2lite_T1024": MoEConfig("c4_dsv2lite_T1024", 4, T=1024, H=2048, I=1408, E=64, k=6, S=2),
    # 24 Qwen3-235B-A22B-shaped layers, fresh skew per layer
    "c5_qwen3_235b": MoEConfig("c5_qwen3_235b", 5, T=16384, H=4096, I=1536, E=128, k=8,
                               zipf_range=(0.8, 1.6), layers=24),
    # a quarter of one Qwen3-235B-shaped layer for profiler captures (the full layer holds 7.4 GB on the
    # device): a quarter of the experts AND a quarter of the tokens, so the rows per expert, the tile mix
    # and the bytes per token-expert pair stay those of the full layer while weights, activations and
    # FLOPs are each exactly a quarter
    "c5_quarter": MoEConfig("c5_quarter", 5, T=4096, H=4096, I=1536, E=32, k=8, zipf_range=(0.8, 1.6), layers=1),
}

# The other shapes of the paper's Table 1 (Qwen3-30B and DSv2-Lite are C3 / C4 above), at the
# paper's sequence lengths 2048 / 4096 / 8192 (and 16384), with a mild load skew (the paper's routing comes from
# trained routers on real prompts; a flat N(0,1) router would be unrealistically balanced).
for _i, (_n, _E, _k, _H, _I) in enumerate([("dsv3", 256, 8, 7168, 2048), ("phi35", 16, 2, 4096, 6400),
                                           ("qwen35_35b", 256, 8, 2048, 512), ("dsv2", 160, 6, 5120, 1536),
                                           ("qwen3_30b", 128, 8, 2048, 768), ("dsv2lite", 64, 6, 2048, 1408)]):
    # 16384 is the longest sequence of the paper's scheduler ablation (Section 5.6: 2k to 16k)
    for _T in (2048, 4096, 8192, 16384):
        CONFIGS[f"t1_{_n}_T{_T}"] = MoEConfig(f"t1_{_n}_T{_T}", 10 + _i, T=_T, H=_H, I=_I, E=_E, k=_k, zipf_s=0.5)

_T_X, _T_LOGITS, _T_GATE_UP, _T_DOWN, _T_PERM, _T_SKEW = 1, 2, 3, 4, 5, 6


def tensor_seed(cfg: MoEConfig, layer: int, tensor_id: int) -> int:
    return cfg.base_seed + 1000 * cfg.cfg_id + 16 * layer + tensor_id


def normal_f32(n: int, seed: int, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)
    _load().wl_normal_f32(out.ctypes.data, n, seed, mean, std)
    return out


def normal_bf16(n: int, seed: int, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    """Raw bf16 bit patterns as uint16."""
    out = np.empty(n, dtype=np.uint16)
    _load().wl_normal_bf16(out.ctypes.data, n, seed, mean, std)
    return out


def uniform01(seed: int, counter: int) -> float:
    return (_load().wl_hash(seed, counter) >> 11) * (1.0 / 9007199254740992.0)


def expert_permutation(E: int, seed: int) -> np.ndarray:
    """pi[e] = rank of expert e (0 = most loaded), from sorting hash values."""
    lib = _load()
    keys = np.array([lib.wl_hash(seed, e) for e in range(E)], dtype=np.uint64)
    order = np.argsort(keys, kind="stable")
    pi = np.empty(E, dtype=np.int64)
    pi[order] = np.arange(E)
    return pi


def layer_skew(cfg: MoEConfig, layer: int) -> Optional[float]:
    if cfg.zipf_s is not None:
        return float(cfg.zipf_s)
    if cfg.zipf_range is not None:
        lo, hi = cfg.zipf_range
        return lo + (hi - lo) * uniform01(tensor_seed(cfg, layer, _T_SKEW), 0)
    return None


def expert_bias(cfg: MoEConfig, layer: int) -> Optional[np.ndarray]:
    """b_e = -s * ln(pi(e)+1): added to N(0,1) logits so that the load is Zipf-like."""
    s = layer_skew(cfg, layer)
    if s is None:
        return None
    pi = expert_permutation(cfg.E, tensor_seed(cfg, layer, _T_PERM))
    return (-s * np.log(pi.astype(np.float64) + 1.0)).astype(np.float32)


def make_logits(cfg: MoEConfig, layer: int = 0) -> np.ndarray:
    lg = normal_f32(cfg.T * cfg.E, tensor_seed(cfg, layer, _T_LOGITS)).reshape(cfg.T, cfg.E)
    b = expert_bias(cfg, layer)
    if b is not None:
        _load().wl_add_row_bias_f32(lg.ctypes.data, cfg.T, cfg.E, b.ctypes.data)
    return lg


def make_x(cfg: MoEConfig, layer: int = 0) -> np.ndarray:
    """x as raw bf16 bits, [T,H] uint16.  The 24-layer stack reuses layer 0's x."""
    return normal_bf16(cfg.T * cfg.H, tensor_seed(cfg, 0, _T_X)).reshape(cfg.T, cfg.H)


def make_weights(cfg: MoEConfig):
    """(gate_up [E+S,2I,H], down [E+S,H,I]) raw bf16 bits; one layer's weights, reused."""
    EE = cfg.E + cfg.S
    gu = normal_bf16(EE * 2 * cfg.I * cfg.H, tensor_seed(cfg, 0, _T_GATE_UP), 0.0, 0.02)
    dn = normal_bf16(EE * cfg.H * cfg.I, tensor_seed(cfg, 0, _T_DOWN), 0.0, 0.02)
    return gu.reshape(EE, 2 * cfg.I, cfg.H), dn.reshape(EE, cfg.H, cfg.I)


def expert_weights(cfg: MoEConfig, e: int):
    """(gate_up[e] [2I,H], down[e] [H,I]) of one expert: the same values make_weights() puts at index
    e, produced without materialising the other experts (the streams are counter-based)."""
    lib = _load()
    n_gu, n_dn = 2 * cfg.I * cfg.H, cfg.H * cfg.I
    gu = np.empty(n_gu, dtype=np.uint16)
    dn = np.empty(n_dn, dtype=np.uint16)
    lib.wl_normal_bf16_range(gu.ctypes.data, e * n_gu, n_gu, tensor_seed(cfg, 0, _T_GATE_UP), 0.0, 0.02)
    lib.wl_normal_bf16_range(dn.ctypes.data, e * n_dn, n_dn, tensor_seed(cfg, 0, _T_DOWN), 0.0, 0.02)
    return gu.reshape(2 * cfg.I, cfg.H), dn.reshape(cfg.H, cfg.I)


@dataclass
class LayerInputs:
    cfg: MoEConfig
    x: np.ndarray          # [T,H] uint16 (bf16 bits)
    logits: np.ndarray     # [T,E] float32
    gate_up: np.ndarray    # [E+S,2I,H] uint16
    down: np.ndarray       # [E+S,H,I] uint16
    layer: int = 0
    extra: dict = field(default_factory=dict)


def make_inputs(cfg: MoEConfig, layer: int = 0, weights=None) -> LayerInputs:
    gu, dn = weights if weights is not None else make_weights(cfg)
    return LayerInputs(cfg, make_x(cfg, layer), make_logits(cfg, layer), gu, dn, layer)


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> 16) & 1
    return ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)


def stratified_token_sample(T: int, n: int, seed: int = 0) -> np.ndarray:
    """n distinct token indices: first, last, and one hashed pick per equal stratum."""
    n = min(n, T)
    lib = _load()
    picks = {0, T - 1}
    strata = max(n - 2, 0)
    for i in range(strata):
        lo = (i * T) // strata
        hi = max(((i + 1) * T) // strata, lo + 1)
        picks.add(lo + int(lib.wl_hash(seed, i) % (hi - lo)))
    return np.array(sorted(picks), dtype=np.int32)
