"""CPU restatement of the paper's scheduling cost model.  TEST INFRASTRUCTURE ONLY.

Follows Section 3 equation by equation, in the paper's notation, in IEEE fp32
(numpy float32 scalars: every operation is one correctly rounded fp32 operation,
no fused multiply-add), so that a device implementation that uses the same
operation order and round-to-nearest intrinsics must return the same plan.

Single-GPU reading of the workload terms (the paper counts only remote tokens,
which would be zero without peers): every token-expert pair moves through HBM,
so with P pairs, T tokens and B = 2H bytes per row
    W_comp     = P * 6*H*I              (Eq. 1, X_local + X_in = P)
    W_dispatch = (T + P) * B            (Eq. 2: each token read once, P rows written)
    W_combine  = (P + T) * B            (Eq. 3: P rows read, T rows written)
    W_comm     = W_dispatch + W_combine (Eq. 11's undefined symbol, as in Eq. 5)

Two further plan kinds, outside the paper (its movement crosses NVLink, so it never considers
them; on one GPU, where movement is an HBM copy that all SMs can do at full speed, they matter):
    kind 1, "dispatch on all SMs, then split": every SM dispatches, then c SMs combine chunk by
            chunk while N-c SMs run the GEMMs:
            T = W_disp/BW(N) + max(T_comp(c,K) + T_tail(c,K), W_comb/BW(c))
    kind 2, "phased": all SMs per phase, no spatial split (the paper's "w/o S+T" ablation as a
            candidate):  T = W_disp/BW(N) + W_comp/TFLOPS(N) + (1-alpha) * W_comb/BW(N)
    kind 3, "split with rejoin" (K = 1): c SMs dispatch while N-c run GEMM tiles; when the dispatch
            is done the c SMs join the GEMM queue for good; the final combine runs on all SMs:
            t_d = W_disp/BW(c),  W_during = min(t_d * TFLOPS(N-c), 2/3 W_comp)  (as Eq. 12; the 2/3 are
            the gate/up FLOPs, 4HI of 6HI per row, which the queue runs first: a dispatch that outlasts
            them holds the GEMM SMs up),
            T = t_d + max(0, W_comp - W_during)/TFLOPS(N) + (1-alpha) * W_comb/BW(N)
They take part in the arg-min only when CostTables.kinds has their bit set; ties go to the
paper's kind, then kinds 1, 2, 3 in that order, then to the smaller c, then to the smaller K.

Units: work in FLOPs / bytes, rates in FLOP/us and byte/us, times in us.
Parity: pinned by closed forms in tests/test_oracle_cost_model.py.  The values
the paper prints for its own runs (c*=40, K*=4 at 1.365 ms; 8.2 % gap; 0.54 us)
depend on calibration curves that exist only as figures: parity unpinned for
those, they are context only.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Sequence

import numpy as np

f32 = np.float32
K_CANDIDATES = (1, 2, 4, 8)
KIND_SPLIT, KIND_DISPATCH_ALL, KIND_PHASED, KIND_REJOIN = 0, 1, 2, 3


@dataclass
class CostTables:
    """Hardware input of the cost model (Figure 7: bandwidth / throughput curves)."""
    n_sm: int
    bw: np.ndarray        # [n_sm+1] float32, byte/us moved by c movement SMs (bw[0] unused)
    tflops: np.ndarray    # [n_sm+1] float32, FLOP/us delivered by n GEMM SMs (tflops[0] unused)
    eff_chunk: np.ndarray  # [4] float32, eff_chunk(K) for K = 1,2,4,8 (Eq. 9), eff_chunk[0] = 1
    alpha: float          # tile-level overlap ratio in [0,1) (Section 3.1)
    c_min: int = 2
    c_max: int = 74
    c_step: int = 2
    steal_workers: int = 0   # Eq. 14's N: workers that share W_steal (0 = n_sm; a build whose GEMM
                             # worker is an SM pair passes n_sm // 2 and counts tiles per pair)
    max_segments: int = 0    # a build that keeps a table of (chunk, expert) segments bounds the chunk
                             # count: candidates with K * n_experts > max_segments are skipped (0 = no bound)
    kinds: int = 1           # bit mask of the plan kinds in the arg-min: 1 = the paper's split (Eq. 15),
                             # 2 = dispatch on all SMs then split, 4 = phased, 8 = split with rejoin


@dataclass
class Plan:
    c: int
    K: int
    n_steal: int
    t_total: float
    kind: int = KIND_SPLIT


def workloads(T: int, P: int, H: int, I: int):
    """Eq. 1-3 under the single-GPU reading; fp32 like the device."""
    B = f32(2 * H)
    w_comp = f32(P) * f32(6.0) * f32(H) * f32(I)
    w_disp = f32(T + P) * B
    w_comb = f32(P + T) * B
    return w_comp, w_disp, w_comb


def workloads_ep(x_local: int, x_in: int, x_in_uniq: int, H: int, I: int):
    """Eq. 1-3 literally, for one expert-parallel rank: W_comp = (X_local + X_in) * 6HI,
    W_dispatch = X_in^uniq * B (each unique remote token is pulled once), W_combine = X_in * B."""
    B = f32(2 * H)
    w_comp = f32(x_local + x_in) * f32(6.0) * f32(H) * f32(I)
    w_disp = f32(x_in_uniq) * B
    w_comb = f32(x_in) * B
    return w_comp, w_disp, w_comb


def t_total(tab: CostTables, c: int, ki: int, w_comp, w_disp, w_comb) -> np.float32:
    """Eq. 15 with Eq. 9 (T_comp), Eq. 5 (T_comm) and Eq. 10 (T_tail)."""
    K = f32(K_CANDIDATES[ki])
    bw = f32(tab.bw[c])
    tf = f32(tab.tflops[tab.n_sm - c])
    t_comp = w_comp / (tf * f32(tab.eff_chunk[ki]))
    t_comm = (w_disp + w_comb) / bw
    t_tail = (f32(1.0) - f32(tab.alpha)) * (w_comb / (bw * K))
    return np.maximum(t_comp + t_tail, t_comm)


def t_total_dispatch_all(tab: CostTables, c: int, ki: int, w_comp, w_disp, w_comb) -> np.float32:
    """Kind 1: the dispatch runs on all N SMs first (W_disp / BW(N)); from then on the split of
    Eq. 15 with only the combine left as communication."""
    K = f32(K_CANDIDATES[ki])
    bw = f32(tab.bw[c])
    tf = f32(tab.tflops[tab.n_sm - c])
    t_disp = w_disp / f32(tab.bw[tab.n_sm])
    t_comp = w_comp / (tf * f32(tab.eff_chunk[ki]))
    t_tail = (f32(1.0) - f32(tab.alpha)) * (w_comb / (bw * K))
    t_comb = w_comb / bw
    return t_disp + np.maximum(t_comp + t_tail, t_comb)


def t_total_phased(tab: CostTables, w_comp, w_disp, w_comb) -> np.float32:
    """Kind 2: dispatch, GEMMs and combine one after the other, each on all N SMs."""
    bw = f32(tab.bw[tab.n_sm])
    tf = f32(tab.tflops[tab.n_sm])
    return (w_disp / bw + w_comp / tf) + (f32(1.0) - f32(tab.alpha)) * (w_comb / bw)


def t_total_rejoin(tab: CostTables, c: int, w_comp, w_disp, w_comb) -> np.float32:
    """Kind 3 (K = 1): the GEMM SMs' work during the dispatch as in Eq. 12, the rest on all N SMs."""
    n = tab.n_sm
    t_disp = w_disp / f32(tab.bw[c])
    w_during = np.minimum(t_disp * f32(tab.tflops[n - c]), w_comp * f32(0.6666667))
    w_rest = np.maximum(f32(0.0), w_comp - w_during)
    return (t_disp + w_rest / f32(tab.tflops[n])) + (f32(1.0) - f32(tab.alpha)) * (w_comb / f32(tab.bw[n]))


def candidates(tab: CostTables):
    c = tab.c_min
    while c <= tab.c_max and c <= tab.n_sm - 1:
        yield c
        c += tab.c_step


def n_steal(tab: CostTables, c: int, w_comp, w_disp, w_comb, n_tiles: int) -> int:
    """Eq. 11-14.  W_tile is the mean FLOPs of the n_tiles GEMM tiles of this layer,
    so n_steal = W_steal / (N * W_tile); rounded to nearest (half away from zero is
    impossible to hit exactly with these magnitudes; floor(x+0.5) is used), clamped
    to [0, n_tiles]."""
    if n_tiles <= 0:
        return 0
    t_comm = (w_disp + w_comb) / f32(tab.bw[c])                     # Eq. 11
    w_partial = t_comm * f32(tab.tflops[tab.n_sm - c])              # Eq. 12
    w_steal = np.maximum(f32(0.0), w_comp - w_partial)              # Eq. 13
    w_tile = w_comp / f32(n_tiles)
    if not (w_tile > 0):
        return 0
    ns = w_steal / (f32(tab.steal_workers or tab.n_sm) * w_tile)    # Eq. 14
    ns = int(np.floor(ns + f32(0.5)))
    return max(0, min(ns, n_tiles))


def plan(tab: CostTables, T: int, P: int, H: int, I: int, n_tiles_of_K: Sequence[int], w=None,
         n_experts: int = 0) -> Plan:
    """Eq. 16: argmin over the (c,K) grid, ties to the smaller c and then the smaller K;
    then the steal count at (c*,K*).  n_tiles_of_K[ki] = number of GEMM tiles of the
    layer when it is cut into K_CANDIDATES[ki] chunks.  w = (W_comp, W_disp, W_comb) overrides the
    single-GPU workload terms (used with workloads_ep).  n_experts (routed + shared) matters only
    with tab.max_segments.  Plan kinds beyond the paper's take part per tab.kinds; they come
    after the paper's kind in the candidate order, so ties go to the paper's.  The steal quota
    of Eq. 11-14 belongs to the paper's kind; the other kinds have none (0): in kind 1 the
    movement SMs are idle from the end of the dispatch on, in kind 2 there are no roles."""
    w_comp, w_disp, w_comb = w if w is not None else workloads(T, P, H, I)
    best = None
    evaluators = ((KIND_SPLIT, t_total), (KIND_DISPATCH_ALL, t_total_dispatch_all))
    for kind, fn in evaluators:
        if not (tab.kinds >> kind) & 1:
            continue
        for c in candidates(tab):
            for ki in range(len(K_CANDIDATES)):
                if tab.max_segments and K_CANDIDATES[ki] * n_experts > tab.max_segments:
                    continue
                t = fn(tab, c, ki, w_comp, w_disp, w_comb)
                if best is None or t < best[0]:
                    best = (t, c, ki, kind)
    if (tab.kinds >> KIND_PHASED) & 1:
        t = t_total_phased(tab, w_comp, w_disp, w_comb)
        if best is None or t < best[0]:
            best = (t, tab.n_sm, 0, KIND_PHASED)
    if (tab.kinds >> KIND_REJOIN) & 1:
        for c in candidates(tab):
            t = t_total_rejoin(tab, c, w_comp, w_disp, w_comb)
            if best is None or t < best[0]:
                best = (t, c, 0, KIND_REJOIN)
    t, c, ki, kind = best
    steal = n_steal(tab, c, w_comp, w_disp, w_comb, n_tiles_of_K[ki]) if kind == KIND_SPLIT else 0
    return Plan(c, K_CANDIDATES[ki], steal, float(t), kind)
