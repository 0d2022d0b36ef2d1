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


def test_steal_count_with_pair_workers():
    """A build whose GEMM worker is an SM pair divides W_steal among N/2 workers and counts pair
    tiles (Eq. 14 with N = pairs).  Closed forms: infinitely fast movement leaves all of W_comp to
    share, so every worker gets n_tiles / (N/2) tiles; when W_partial is exactly half of W_comp the
    quota is half of that; the pair quota is twice the per-SM quota for the same tile count."""
    N = 148
    T, P, H, I = 4096, 8192, 4096, 14336
    w = cm.workloads(T, P, H, I)
    n_tiles = 7400                       # 100 per pair
    assert cm.n_steal(_toy(b=1e20, steal_workers=N // 2), 10, *w, n_tiles) == n_tiles // (N // 2) == 100
    assert cm.n_steal(_toy(b=1e20), 10, *w, n_tiles) == n_tiles // N == 50
    f = 10.0e6
    t_half = float(w[0]) / 2 / (f * (N - 10))
    b = float(w[1] + w[2]) / t_half / 10
    assert abs(cm.n_steal(_toy(b=b, f=f, steal_workers=N // 2), 10, *w, n_tiles) - 50) <= 1
    # slow movement: nothing is left to steal, whatever the worker count
    assert cm.n_steal(_toy(b=1e-3, steal_workers=N // 2), 10, *w, n_tiles) == 0
    # a non-integer share rounds to nearest: 7437 / 74 = 100.5 -> 101 (floor(x + 0.5)), 7436 / 74 = 100.49 -> 100
    assert cm.n_steal(_toy(b=1e20, steal_workers=N // 2), 10, *w, 7437) == 101
    assert cm.n_steal(_toy(b=1e20, steal_workers=N // 2), 10, *w, 7436) == 100


def test_segment_table_bound_removes_large_chunk_counts():
    """With a bound on (chunk, expert) segments, K * n_experts > bound is not a candidate: without a
    chunking penalty the model wants K = 8, and gets the largest K that fits."""
    T, P, H, I = 8192, 65536, 2048, 512
    free = _toy(eff=(1, 1, 1, 1))
    assert cm.plan(free, T, P, H, I, [10] * 4, n_experts=256).K == 8
    bound = _toy(eff=(1, 1, 1, 1), max_segments=1024)
    assert cm.plan(bound, T, P, H, I, [10] * 4, n_experts=256).K == 4      # 8 * 256 > 1024
    assert cm.plan(bound, T, P, H, I, [10] * 4, n_experts=128).K == 8
    assert cm.plan(bound, T, P, H, I, [10] * 4, n_experts=600).K == 1


def test_phased_plan_wins_when_movement_is_cheap_by_the_gemm_rate_ratio():
    """Movement -> 0: every kind's time is its GEMM time, W_comp / TFLOPS(n).  The phased plan runs
    the GEMMs on all N SMs, the best split on N - c_min, so the phased plan wins and the ratio of
    the two times is TFLOPS(N) / TFLOPS(N - c_min)."""
    N = 148
    T, P, H, I = 4096, 8192, 4096, 14336
    split_only = _toy(N, b=1e15, f=1e6)
    both = _toy(N, b=1e15, f=1e6, kinds=1 | 4)
    p0 = cm.plan(split_only, T, P, H, I, [10] * 4)
    p2 = cm.plan(both, T, P, H, I, [10] * 4)
    assert (p0.kind, p0.c) == (cm.KIND_SPLIT, 2)
    assert (p2.kind, p2.c, p2.K, p2.n_steal) == (cm.KIND_PHASED, N, 1, 0)
    assert math.isclose(p0.t_total / p2.t_total, N / (N - 2), rel_tol=1e-5)      # toy TFLOPS(n) = f * n


def test_phased_plan_loses_when_movement_dominates_and_overlaps():
    """Linear toy curves, alpha = 0, K = 1 forced.  By hand: phased = W_disp/(bN) + A/N + W_comb/(bN)
    with A = W_comp/f; the split at c takes max(A/(N-c) + W_comb/(bc), (W_disp+W_comb)/(bc)).  For
    three bandwidths the plan must be the smaller of the hand-written phased time and the hand-written
    minimum over c, and must say which kind it is."""
    N = 148
    T, P, H, I = 8192, 65536, 2048, 768
    w_comp, w_disp, w_comb = (float(v) for v in cm.workloads(T, P, H, I))
    f = 8.0e6
    A = w_comp / f
    for b in (2.0e3, 2.0e4, 2.0e5):
        tab = _toy(N, b=b, f=f, eff=(1.0, 1e-3, 1e-3, 1e-3), kinds=1 | 4, c_min=2, c_max=N - 2, c_step=2)
        hand_phased = w_disp / (b * N) + A / N + w_comb / (b * N)
        hand_split = min(max(A / (N - c) + w_comb / (b * c), (w_disp + w_comb) / (b * c)) for c in range(2, N - 1, 2))
        p = cm.plan(tab, T, P, H, I, [10] * 4)
        assert math.isclose(p.t_total, min(hand_phased, hand_split), rel_tol=1e-5)
        assert (p.kind == cm.KIND_PHASED) == (hand_phased < hand_split)


def test_dispatch_all_kind_closed_form_and_tie_order():
    """Kind 1 at (c, K): W_disp/BW(N) + max(T_comp + T_tail, W_comb/BW(c)).  With a huge GEMM rate
    it is W_disp/(bN) + W_comb/(bc), minimal at c_max; the paper's kind gives (W_disp+W_comb)/(b c_max),
    which is larger whenever c_max < N, so kind 1 wins; with identical times the paper's kind is kept."""
    N = 148
    T, P, H, I = 1000, 8000, 1024, 512
    w_comp, w_disp, w_comb = (float(v) for v in cm.workloads(T, P, H, I))
    b = 1.0e3
    tab = _toy(N, b=b, f=1e30, kinds=1 | 2)
    p = cm.plan(tab, T, P, H, I, [10] * 4)
    assert (p.kind, p.c, p.n_steal) == (cm.KIND_DISPATCH_ALL, 74, 0)
    assert math.isclose(p.t_total, w_disp / (b * N) + w_comb / (b * 74), rel_tol=1e-5)
    # no movement cost at all and flat curves: every candidate of every kind ties -> paper's kind, c_min, K = 1
    flat = np.full(N + 1, 5.0e6, np.float32)
    tabf = cm.CostTables(N, np.full(N + 1, 1e30, np.float32), flat, np.ones(4, np.float32), 0.0, kinds=7)
    pf = cm.plan(tabf, T, P, H, I, [10] * 4)
    assert (pf.kind, pf.c, pf.K) == (cm.KIND_SPLIT, 2, 1)


def test_rejoin_kind_closed_forms():
    """Kind 3: t_d = W_disp/BW(c); the N-c GEMM SMs do t_d*TFLOPS(N-c) meanwhile; the rest runs on N SMs.
    (a) With LINEAR curves the time does not depend on c and equals the phased time: by hand
        t_d + (A*f - f*(N-c)*t_d)/(f*N) = A/N + t_d*c/N = A/N + W_disp/(b*N), A = W_comp/f.  Phased comes
        first in the candidate order, so it keeps the tie.
    (b) With a concave GEMM curve, TFLOPS(n) = F*sqrt(n/N), the time is t_d*(1 - sqrt((N-c)/N)) + W_comp/F
        + tail while the GEMMs outlast the dispatch: less than the phased time, minimal at some c that
        the hand formula gives.
    (c) Slow dispatch: only the gate/up tiles (2/3 of the FLOPs) can run meanwhile; T = t_d + the down tiles
        on N SMs + the combine tail."""
    N = 148
    T, P, H, I = 8192, 65536, 2048, 768
    w_comp, w_disp, w_comb = (float(v) for v in cm.workloads(T, P, H, I))
    b, f = 40.0e3, 8.0e6
    lin = _toy(N, b, f, kinds=8)
    A = w_comp / f
    for c in (24, 32, 74):        # (with these the dispatch ends before 2/3 of the GEMM work is done: c/(N-c) > 0.147)
        t = float(cm.t_total_rejoin(lin, c, *cm.workloads(T, P, H, I)))
        assert math.isclose(t, A / N + w_disp / (b * N) + w_comb / (b * N), rel_tol=1e-5)
    # two dispatch SMs: only the gate/up tiles (2/3 of the work) can run meanwhile, the down tiles follow on N SMs
    t2 = float(cm.t_total_rejoin(lin, 2, *cm.workloads(T, P, H, I)))
    assert math.isclose(t2, w_disp / (b * 2) + (A / 3) / N + w_comb / (b * N), rel_tol=1e-5)
    both = _toy(N, b, f, kinds=4 | 8)
    assert cm.plan(both, T, P, H, I, [10] * 4).kind == cm.KIND_PHASED
    # (b) TFLOPS(n) = F * sqrt(n / N)
    idx = np.arange(N + 1, dtype=np.float64)
    F = 1.2e9
    conc = cm.CostTables(N, (b * idx).astype(np.float32), (F * np.sqrt(idx / N)).astype(np.float32),
                         np.ones(4, np.float32), 0.0, kinds=4 | 8)
    p = cm.plan(conc, T, P, H, I, [10] * 4)
    assert p.kind == cm.KIND_REJOIN and p.K == 1 and p.n_steal == 0
    hand = lambda c: (w_disp / (b * c)) * (1.0 - math.sqrt((N - c) / N)) + w_comp / F + w_comb / (b * N) \
        if (w_disp / (b * c)) * F * math.sqrt((N - c) / N) < 2 * w_comp / 3 else w_disp / (b * c) + w_comp / (3 * F) + w_comb / (b * N)
    best_c = min(range(2, 75, 2), key=hand)
    assert math.isclose(p.t_total, hand(best_c), rel_tol=1e-4) and abs(p.c - best_c) <= 2
    phased = w_disp / (b * N) + w_comp / F + w_comb / (b * N)
    assert p.t_total < phased
    # (c) two dispatch SMs at a crawl: the other 146 finish the GEMMs long before
    slow = _toy(N, b=10.0, f=1e9, kinds=8, c_min=2, c_max=2)
    p = cm.plan(slow, T, P, H, I, [10] * 4)
    assert math.isclose(p.t_total, w_disp / 20.0 + (w_comp / 3) / (1e9 * N) + w_comb / (10.0 * N), rel_tol=1e-5)
