"""The value checks of the large GPU parity cases compare sampled output rows.  The sample is built
from the oracle's routing (tests/parity.py: coverage_token_sample); these CPU tests check, by brute
force over the routing, that it reaches what it claims to reach."""
import numpy as np
import pytest

import oracle
import workloads as wl
from parity import coverage_token_sample


def _reached(ref, cfg, toks, block_m):
    """(experts, (expert, m-block) pairs) touched by the rows of the sampled tokens, from the
    definition: row r of expert e lies in m-block (r - offsets[e]) // block_m."""
    experts, blocks = set(), set()
    for t in toks:
        for j in range(cfg.k + cfg.S):
            r = int(ref.row_of[t, j])
            e = int(ref.idx[t, j]) if j < cfg.k else cfg.E + (j - cfg.k)
            assert ref.offsets[e] <= r < ref.offsets[e + 1] and ref.token_of[r] == t
            experts.add(e)
            blocks.add((e, (r - int(ref.offsets[e])) // block_m))
    return experts, blocks


@pytest.mark.parametrize("name", ["c3_qwen3_30b", "c4_dsv2lite_T1024", "t1_qwen35_35b_T2048"])
def test_full_sample_reaches_every_expert_segment_end_and_m_block(name):
    cfg = wl.CONFIGS[name]
    ref = oracle.routing(wl.make_logits(cfg), cfg.k, cfg.S)
    toks, cov = coverage_token_sample(ref, cfg, 16, None, 128, seed=cfg.cfg_id)
    assert len(set(toks.tolist())) == len(toks) and (np.diff(toks) > 0).all()
    experts, blocks = _reached(ref, cfg, toks, 128)
    nonempty = {e for e in range(cfg.E + cfg.S) if ref.counts[e] > 0}
    assert experts == nonempty
    all_blocks = {(e, m) for e in nonempty for m in range((int(ref.counts[e]) + 127) // 128)}
    assert blocks == all_blocks
    # first and last row of every routed expert's segment
    tokset = set(toks.tolist())
    for e in range(cfg.E):
        if ref.counts[e] > 0:
            assert int(ref.token_of[ref.offsets[e]]) in tokset
            assert int(ref.token_of[ref.offsets[e + 1] - 1]) in tokset
    assert cov["experts"] == len(nonempty) and cov["m_blocks"] == len(all_blocks) == cov["m_blocks_total"]
    assert cov["tiny_experts"] == cov["tiny_experts_total"]


def test_budget_keeps_the_strata_and_prefers_small_experts():
    cfg = wl.CONFIGS["c3_qwen3_30b"]
    ref = oracle.routing(wl.make_logits(cfg), cfg.k, cfg.S)
    toks, cov = coverage_token_sample(ref, cfg, 8, 40, 128, seed=3)
    assert len(toks) == 40 and 0 in toks and cfg.T - 1 in toks
    # the smallest non-empty experts' end rows come first after the strata
    smallest = [e for e in np.argsort(ref.counts[:cfg.E], kind="stable") if ref.counts[e] > 0][:8]
    for e in smallest:
        assert int(ref.token_of[ref.offsets[e]]) in set(toks.tolist())
