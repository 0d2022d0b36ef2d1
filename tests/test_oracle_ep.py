"""Pins for the oracle's expert-parallel share: the partial outputs of all ranks add up to the
full layer, the workload descriptors equal a set-based count, the restricted permutation is the
full one with the other experts removed."""
import numpy as np
import pytest

import oracle
from oracle import cost_model as cm
import workloads as wl


def _layer(T=96, H=64, I=96, E=16, k=4, seed=5):
    x = wl.normal_bf16(T * H, seed).reshape(T, H)
    lg = wl.normal_f32(T * E, seed + 1).reshape(T, E)
    gu = wl.normal_bf16(E * 2 * I * H, seed + 2, 0.0, 0.05).reshape(E, 2 * I, H)
    dn = wl.normal_bf16(E * H * I, seed + 3, 0.0, 0.05).reshape(E, H, I)
    return x, lg, gu, dn


@pytest.mark.parametrize("R", [1, 2, 4])
def test_partial_outputs_of_all_ranks_sum_to_the_full_layer(R):
    x, lg, gu, dn = _layer()
    T, k = x.shape[0], 4
    toks = np.arange(T, dtype=np.int32)
    full = oracle.moe_tokens(x, lg, gu, dn, k, toks, acc_double=True)
    parts = [oracle.moe_tokens_ep(x, lg, gu, dn, k, toks, r, R, acc_double=True) for r in range(R)]
    np.testing.assert_allclose(sum(parts), full, rtol=2e-6, atol=2e-7)
    if R == 1:
        np.testing.assert_allclose(parts[0], full, rtol=1e-6, atol=1e-8)
    # a token without an expert on the rank gets exactly zero
    idx, _ = oracle.route(lg, k)
    for r in range(R):
        lo, hi = r * (16 // R), (r + 1) * (16 // R)
        none = ~((idx >= lo) & (idx < hi)).any(axis=1)
        assert (parts[r][none] == 0).all()


def test_descriptors_match_a_set_based_count():
    T, E, k, R = 200, 32, 6, 4
    lg = wl.normal_f32(T * E, 9).reshape(T, E)
    idx, _ = oracle.route(lg, k)
    Ts = (T + R - 1) // R
    tot_pairs = 0
    for r in range(R):
        xl, xi, xu = oracle.ep_descriptors(idx, E, r, R)
        lo, hi = r * (E // R), (r + 1) * (E // R)
        pairs = [(t, e) for t in range(T) for e in idx[t] if lo <= e < hi]
        own = lambda t: t // Ts == r
        assert xl == sum(1 for t, _ in pairs if own(t))
        assert xi == sum(1 for t, _ in pairs if not own(t))
        assert xu == len({t for t, _ in pairs if not own(t)})
        assert xu <= xi
        tot_pairs += xl + xi
    assert tot_pairs == T * k                       # every pair lives on exactly one rank
    # R = 1: nothing is remote
    assert oracle.ep_descriptors(idx, E, 0, 1) == (T * k, 0, 0)


def test_restricted_permutation_is_the_full_one_without_the_other_experts():
    T, E, k, R = 150, 16, 4, 4
    lg = wl.normal_f32(T * E, 13).reshape(T, E)
    full = oracle.routing(lg, k)
    for r in range(R):
        ep = oracle.routing_ep(lg, k, r, R)
        lo, hi = r * (E // R), (r + 1) * (E // R)
        np.testing.assert_array_equal(ep.idx, full.idx)
        np.testing.assert_array_equal(ep.gates, full.gates)          # gates stay normalised over all k
        np.testing.assert_array_equal(ep.counts[lo:hi], full.counts[lo:hi])
        assert ep.counts[:lo].sum() == 0 and ep.counts[hi:].sum() == 0
        local = (full.idx >= lo) & (full.idx < hi)
        assert (ep.row_of[~local] == -1).all()
        # local rows keep their order: same token sequence per expert, shifted to start at 0
        np.testing.assert_array_equal(ep.row_of[local], full.row_of[:, :k][local] - full.offsets[lo])
        np.testing.assert_array_equal(ep.token_of, full.token_of[full.offsets[lo]:full.offsets[hi]])


def test_ep_workload_terms_follow_eq1_to_eq3_literally():
    w_comp, w_disp, w_comb = cm.workloads_ep(1000, 3000, 1200, 4096, 1536)
    assert np.isclose(float(w_comp), 4000 * 6 * 4096 * 1536, rtol=1e-6)
    assert np.isclose(float(w_disp), 1200 * 2 * 4096, rtol=1e-6)      # unique remote tokens only
    assert np.isclose(float(w_comb), 3000 * 2 * 4096, rtol=1e-6)      # one result per remote pair
    # no remote tokens: the communication terms vanish and the model degenerates to compute only
    _, d0, c0 = cm.workloads_ep(1000, 0, 0, 4096, 1536)
    assert float(d0) == 0.0 and float(c0) == 0.0
