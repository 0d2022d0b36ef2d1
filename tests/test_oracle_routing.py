"""Pins for the oracle's routing stages: select (top-k), gates, counts/offsets, permutation.

Every check compares the oracle with something that is not the oracle: a full stable
sort, a library softmax / bincount / argsort, crafted inputs whose answer is known by
construction, or an invariant of the definition.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl


def _brute_topk(logits, k):
    """Full stable sort by (-logit, index): numpy's stable argsort on the negated logits
    keeps the lower index first among equal keys (and -0.0 == 0.0 compare equal)."""
    order = np.argsort(-logits.astype(np.float64), axis=1, kind="stable")
    return order[:, :k].astype(np.int32)


@pytest.mark.parametrize("T,E,k", [(1, 1, 1), (7, 8, 2), (33, 64, 6), (50, 128, 8), (16, 5, 5), (9, 256, 8)])
def test_topk_matches_full_stable_sort(T, E, k):
    lg = wl.normal_f32(T * E, seed=11 + T + E).reshape(T, E)
    idx, _ = oracle.route(lg, k)
    np.testing.assert_array_equal(idx, _brute_topk(lg, k))


def test_topk_ties_go_to_lowest_index():
    E, k = 16, 4
    # all-equal row => 0..k-1
    lg = np.zeros((1, E), np.float32)
    idx, g = oracle.route(lg, k)
    np.testing.assert_array_equal(idx[0], np.arange(k))
    np.testing.assert_allclose(g[0], 1.0 / k, rtol=1e-7)
    # duplicated maxima at 9 and 3 => 3 first, then 9; then the tied runners-up 0,1
    lg = np.full((1, E), -1.0, np.float32)
    lg[0, 9] = 2.0
    lg[0, 3] = 2.0
    idx, _ = oracle.route(lg, k)
    np.testing.assert_array_equal(idx[0], [3, 9, 0, 1])
    # +0.0 and -0.0 are a tie: lowest index wins regardless of sign bit
    lg = np.full((1, E), -5.0, np.float32)
    lg[0, 7] = 0.0
    lg[0, 2] = -0.0
    idx, _ = oracle.route(lg, 2)
    np.testing.assert_array_equal(idx[0], [2, 7])


def test_topk_k_equals_E_is_stable_argsort_and_gates_are_softmax():
    T, E = 12, 10
    lg = wl.normal_f32(T * E, seed=5).reshape(T, E)
    lg[3, 4] = lg[3, 8]  # a tie inside
    idx, g = oracle.route(lg, E)
    np.testing.assert_array_equal(idx, _brute_topk(lg, E))
    # k = E: gates (scattered back to expert order) are the library softmax over all logits
    sm = torch.softmax(torch.from_numpy(lg).double(), dim=1).numpy()
    got = np.zeros_like(sm)
    np.put_along_axis(got, idx.astype(np.int64), g.astype(np.float64), axis=1)
    np.testing.assert_allclose(got, sm, rtol=2e-6, atol=1e-9)


def test_topk_against_library_topk_on_tie_free_input():
    T, E, k = 64, 128, 8
    lg = wl.normal_f32(T * E, seed=77).reshape(T, E)
    assert all(len(np.unique(r)) == E for r in lg)  # tie-free, so library order is defined
    idx, g = oracle.route(lg, k)
    tv, ti = torch.topk(torch.from_numpy(lg), k, dim=1, largest=True, sorted=True)
    np.testing.assert_array_equal(idx, ti.numpy().astype(np.int32))
    # gates = renormalised full softmax restricted to the selected k
    full = torch.softmax(torch.from_numpy(lg).double(), dim=1)
    sel = torch.gather(full, 1, ti)
    ref = (sel / sel.sum(dim=1, keepdim=True)).numpy()
    np.testing.assert_allclose(g, ref, rtol=3e-6)


def test_gate_properties():
    T, E, k = 40, 32, 6
    lg = wl.normal_f32(T * E, seed=3).reshape(T, E)
    idx, g = oracle.route(lg, k)
    np.testing.assert_allclose(g.sum(axis=1), 1.0, atol=1e-6)
    assert (np.diff(g, axis=1) <= 0).all()  # descending logit => descending gate
    # k = 1 => gate exactly 1
    _, g1 = oracle.route(lg, 1)
    assert (g1 == 1.0).all()
    # adding a constant per token changes neither the selection nor (up to rounding) the gates;
    # a power-of-two shift of small logits is exact in fp32 differences only approximately,
    # so compare with a tolerance
    idx2, g2 = oracle.route(lg + np.float32(8.0), k)
    np.testing.assert_array_equal(idx, idx2)
    np.testing.assert_allclose(g, g2, rtol=2e-5)


def test_nonfinite_logits_are_rejected():
    lg = np.zeros((2, 4), np.float32)
    lg[1, 2] = np.nan
    with pytest.raises(ValueError):
        oracle.route(lg, 2)
    lg[1, 2] = np.inf
    with pytest.raises(ValueError):
        oracle.route(lg, 2)


@pytest.mark.parametrize("T,E,k,S", [(1, 4, 2, 0), (37, 8, 2, 0), (100, 64, 6, 2), (257, 128, 8, 0), (5, 3, 3, 1)])
def test_counts_offsets_permutation(T, E, k, S):
    lg = wl.normal_f32(T * E, seed=100 + T).reshape(T, E)
    r = oracle.routing(lg, k, S)
    P = T * (k + S)
    # experts of a token are distinct
    assert all(len(set(row)) == k for row in r.idx)
    # counts = bincount (library), sum = T*k over routed experts; shared experts see every token
    np.testing.assert_array_equal(r.counts[:E], np.bincount(r.idx.ravel(), minlength=E))
    assert r.counts[:E].sum() == T * k
    assert (r.counts[E:] == T).all()
    # offsets = exclusive prefix sum, monotone, last = P
    np.testing.assert_array_equal(r.offsets, np.concatenate([[0], np.cumsum(r.counts)]))
    assert r.offsets[-1] == P
    # row_of is a bijection onto [0,P) and token_of inverts it
    flat = r.row_of.ravel()
    np.testing.assert_array_equal(np.sort(flat), np.arange(P))
    np.testing.assert_array_equal(r.token_of[r.row_of], np.repeat(np.arange(T)[:, None], k + S, 1))
    # equals a stable counting sort of the flattened (t, slot) list keyed by expert
    keys = np.concatenate([r.idx, np.tile(np.arange(E, E + S, dtype=np.int32), (T, 1))], axis=1).ravel()
    order = np.argsort(keys, kind="stable")           # order[row] = flat (t,slot) index
    np.testing.assert_array_equal(r.token_of, (order // (k + S)).astype(np.int32))
    inv = np.empty(P, np.int64)
    inv[order] = np.arange(P)
    np.testing.assert_array_equal(flat, inv)
    # tokens ascend inside every expert segment, and every row of a segment belongs to it
    for e in range(E + S):
        seg = r.token_of[r.offsets[e]:r.offsets[e + 1]]
        assert (np.diff(seg) > 0).all()
        if e < E:
            assert all(e in r.idx[t] for t in seg)


def test_row_of_definition_brute_force_tiny():
    """row_of[t,j] = offsets[e] + #{t' < t : e in idx[t']} evaluated literally."""
    T, E, k = 23, 5, 2
    lg = wl.normal_f32(T * E, seed=9).reshape(T, E)
    r = oracle.routing(lg, k)
    for t in range(T):
        for j in range(k):
            e = r.idx[t, j]
            before = sum(1 for tp in range(t) if e in r.idx[tp])
            assert r.row_of[t, j] == r.offsets[e] + before


def test_zipf_bias_skews_load_like_the_planning_table():
    """The skewed config's generator: a dozen huge experts, many tiny ones, load sums to T*k."""
    cfg = wl.CONFIGS["c3_qwen3_30b"]
    lg = wl.make_logits(cfg)
    r = oracle.routing(lg, cfg.k)
    c = np.sort(r.counts)[::-1]
    assert c.sum() == cfg.T * cfg.k
    assert c[0] > 0.9 * cfg.T            # the most loaded expert sees nearly every token
    assert (c < 128).sum() > 60          # most experts get less than one 128-row tile
    assert np.median(c) < 100
