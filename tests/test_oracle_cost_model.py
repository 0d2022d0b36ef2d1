"""Pins for the CPU restatement of the scheduling cost model (Section 3, Eq. 1-16).

With toy hardware curves BW(c) = b*c and TFLOPS(n) = f*n the model has closed-form
answers (derived by hand below, not by re-evaluating the same formula), limiting cases
and monotonicity properties; a dropped term, a swapped table or a wrong tie-break fails
at least one of them.
"""
import math

import numpy as np
import pytest

from oracle import cost_model as cm


def _toy(n_sm=148, b=50.0e3, f=10.0e6, eff=(1.0, 1.0, 1.0, 1.0), alpha=0.0, **kw):
    idx = np.arange(n_sm + 1, dtype=np.float32)
    return cm.CostTables(n_sm, (b * idx).astype(np.float32), (f * idx).astype(np.float32),
                         np.array(eff, np.float32), alpha, **kw)


def test_workload_terms_eq1_to_eq3():
    T, k, H, I = 4096, 2, 4096, 14336
    P = T * k
    w_comp, w_disp, w_comb = cm.workloads(T, P, H, I)
    # Eq. 1: 6HI FLOPs per token-expert pair = 2 FLOPs x (gate HxI + up HxI + down IxH)
    assert math.isclose(float(w_comp), P * 2 * (3 * H * I), rel_tol=1e-6)
    # B = 2H bytes per bf16 row
    assert math.isclose(float(w_disp), (T + P) * H * 2, rel_tol=1e-6)
    assert math.isclose(float(w_comb), (P + T) * H * 2, rel_tol=1e-6)


def test_balance_point_closed_form():
    """alpha=0, K=1 forced (eff_chunk(K>1) tiny).  In the compute-dominated branch
    T_total(c) = A/(N-c) + C/c with A = W_comp/f, C = W_comb/b, whose minimum over real c
    is at c/(N-c) = sqrt(C/A)."""
    N = 148
    T, P, H, I = 8192, 65536, 2048, 768
    b, f = 40.0e3, 8.0e6
    tab = _toy(N, b, f, eff=(1.0, 1e-3, 1e-3, 1e-3), c_min=1, c_max=N - 1, c_step=1)
    w_comp, w_disp, w_comb = (float(v) for v in cm.workloads(T, P, H, I))
    r = math.sqrt((w_comb / b) / (w_comp / f))
    c_real = N * r / (1 + r)
    # the branch assumption holds at the optimum: T_comp > W_disp / BW
    assert (w_comp / (f * (N - c_real))) > w_disp / (b * c_real)
    p = cm.plan(tab, T, P, H, I, [100, 100, 100, 100])
    assert p.K == 1
    assert abs(p.c - c_real) <= 1.0
    # and the reported time is the closed-form value at the chosen c
    assert math.isclose(p.t_total, w_comp / (f * (N - p.c)) + w_comb / (b * p.c), rel_tol=1e-5)


def test_limits_compute_only_and_movement_only():
    N = 148
    # huge bandwidth: movement is free, time = W_comp / TFLOPS(N-c), increasing in c => c_min
    p = cm.plan(_toy(N, b=1e12, f=1e6), 4096, 8192, 4096, 14336, [10] * 4)
    assert p.c == 2
    # huge compute rate: time = T_comm = W_comm / BW(c), decreasing in c => c_max
    p = cm.plan(_toy(N, b=1e3, f=1e15), 4096, 8192, 4096, 14336, [10] * 4)
    assert p.c == 74


def test_chunk_count_tradeoff():
    T, P, H, I = 8192, 65536, 2048, 768
    # no chunking penalty: the tail shrinks with 1/K (Eq. 10), so the largest K wins
    assert cm.plan(_toy(eff=(1, 1, 1, 1)), T, P, H, I, [10] * 4).K == 8
    # prohibitive penalty for K>1 (Eq. 9): K = 1
    assert cm.plan(_toy(eff=(1, .01, .01, .01)), T, P, H, I, [10] * 4).K == 1
    # alpha -> 1 removes the tail, so chunking cannot help and any penalty selects K = 1
    assert cm.plan(_toy(eff=(1, .99, .98, .97), alpha=0.999999), T, P, H, I, [10] * 4).K == 1


def test_tail_term_uses_combine_bytes_only():
    """Eq. 10 scales W_combine, not W_comm: with alpha=0, K=1 and T_comp -> 0 both branches
    of the max are movement terms and T_total = max(W_comb, W_disp + W_comb)/BW = W_comm/BW."""
    tab = _toy(b=1.0, f=1e30)
    w_comp, w_disp, w_comb = cm.workloads(1000, 8000, 1024, 512)
    t = cm.t_total(tab, 10, 0, w_comp, w_disp, w_comb)
    assert math.isclose(float(t), float(w_disp + w_comb) / 10.0, rel_tol=1e-6)
    # alpha halves the tail; with a large T_comp the total moves by exactly that amount
    tab0 = _toy(b=1.0, f=1.0, alpha=0.0)
    tab5 = _toy(b=1.0, f=1.0, alpha=0.5)
    d = float(cm.t_total(tab0, 10, 0, w_comp, w_disp, w_comb)) - float(cm.t_total(tab5, 10, 0, w_comp, w_disp, w_comb))
    assert math.isclose(d, 0.5 * float(w_comb) / 10.0, rel_tol=1e-3)


def test_ties_go_to_smaller_c_then_smaller_K():
    N = 148
    flat = np.full(N + 1, 5.0e6, np.float32)
    tab = cm.CostTables(N, flat.copy(), flat.copy(), np.ones(4, np.float32), 0.999999999)
    # alpha rounds to 1 in fp32: no tail, flat curves => every (c,K) has the same T_total
    p = cm.plan(tab, 1024, 8192, 2048, 1408, [7] * 4)
    assert (p.c, p.K) == (tab.c_min, 1)


def test_steal_count_limits():
    N = 148
    T, P, H, I = 4096, 8192, 4096, 14336
    w = cm.workloads(T, P, H, I)
    # W_comp = 0 (no pairs) => nothing to steal (Eq. 13)
    assert cm.n_steal(_toy(), 10, np.float32(0), w[1], w[2], 1000) == 0
    # infinitely fast movement: t_comm -> 0, W_steal = W_comp, n_steal = n_tiles / N (Eq. 14)
    assert cm.n_steal(_toy(b=1e20), 10, *w, 14800) == 100
    # very slow movement: the compute SMs finish everything meanwhile => 0
    assert cm.n_steal(_toy(b=1e-3), 10, *w, 14800) == 0
    # half-way: choose b so that W_partial = W_comp / 2 at c = 10
    f = 10.0e6
    t_half = float(w[0]) / 2 / (f * (N - 10))
    b = float(w[1] + w[2]) / t_half / 10
    assert abs(cm.n_steal(_toy(b=b, f=f), 10, *w, 14800) - 50) <= 1


@pytest.mark.parametrize("T,P,H,I", [(4096, 8192, 4096, 14336), (8192, 65536, 2048, 768), (64, 512, 2048, 1408)])
def test_more_movement_cost_never_lowers_c(T, P, H, I):
    last = 0
    for b in [1e6, 3e5, 1e5, 3e4, 1e4, 3e3, 1e3]:       # falling bandwidth per SM
        p = cm.plan(_toy(b=b, f=8e6, eff=(1, .9, .8, .7)), T, P, H, I, [64] * 4)
        assert p.c >= last
        last = p.c
