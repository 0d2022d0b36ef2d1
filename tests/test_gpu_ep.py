"""GPU parity of the expert-parallel share (one rank of an EP group modelled on one GPU): global
routing, rows only for the experts hosted on the rank, remote tokens staged once, partial outputs.
Checked against the oracle's per-rank functions; the outputs of all ranks must add up to the layer."""
import numpy as np
import pytest
import torch

import oracle
from oracle import cost_model as cm
import workloads as wl
import paper_2609_21483_b200 as pk
from parity import bf16_to_np, check_values, coverage_token_sample, to_dev

pytestmark = pytest.mark.gpu


def _check_rank(moe, inp, r, R, tokens=None):
    cfg = inp.cfg
    ref = oracle.routing_ep(inp.logits, cfg.k, r, R)
    got = {k: v.cpu().numpy() for k, v in moe.routing(cfg.T).items()}
    np.testing.assert_array_equal(got["topk_idx"], ref.idx)
    np.testing.assert_allclose(got["gates"], ref.gates, rtol=1e-5)
    np.testing.assert_array_equal(got["counts"], ref.counts)
    np.testing.assert_array_equal(got["offsets"], ref.offsets)
    np.testing.assert_array_equal(got["row_of"], ref.row_of)
    n_rows = int(ref.offsets[-1])
    np.testing.assert_array_equal(got["token_of"][:n_rows], ref.token_of)
    xl, xi, xu = oracle.ep_descriptors(ref.idx, cfg.E, r, R)
    d = moe.ep_descriptors()
    assert (d["x_local"], d["x_in"], d["x_in_uniq"]) == (xl, xi, xu)
    return ref, (xl, xi, xu)


def test_every_rank_of_a_small_group_and_their_sum():
    cfg = wl.MoEConfig("ep_small", 93, T=1000, H=512, I=768, E=32, k=4, zipf_s=0.8)
    inp = wl.make_inputs(cfg)
    x, lg, gu, dn = to_dev(inp)
    moe = pk.WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    full = moe.forward(x, lg).float().clone()
    moe.check()
    R = 4
    toks = np.arange(cfg.T, dtype=np.int32)
    total = torch.zeros_like(full)
    for r in range(R):
        moe.set_expert_parallel(r, R)
        bits = None
        for sched in [(pk.SCHED_AUTO, 0, 1, 0), (pk.SCHED_SERIAL, 0, 1, 0), (pk.SCHED_FIXED, 12, 2, 3)]:
            moe.set_schedule(*sched)
            out = moe.forward(x, lg)
            moe.check()
            if bits is None:
                bits = out.view(torch.int16).clone()
            assert torch.equal(out.view(torch.int16), bits), f"rank {r}: schedule {sched} changed the output bits"
        _check_rank(moe, inp, r, R)
        ref = oracle.moe_tokens_ep(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, toks, r, R)
        check_values(bf16_to_np(out), ref, f"rank {r}")
        # tokens without an expert on this rank come back as exact zeros
        idx = moe.routing(cfg.T)["topk_idx"].cpu().numpy()
        lo, hi = r * (cfg.E // R), (r + 1) * (cfg.E // R)
        none = torch.from_numpy(~((idx >= lo) & (idx < hi)).any(axis=1)).cuda()
        assert (out[none] == 0).all() and bool(none.any())
        total += out.float()
    # the partial outputs of all ranks add up to the layer (each was rounded to bf16 once more)
    err = (total - full).abs()
    assert bool((err <= 3e-2 + 3e-2 * full.abs()).all())
    assert float(torch.linalg.norm(total - full) / torch.linalg.norm(full)) < 8e-3
    # back to the plain layer
    moe.set_expert_parallel(0, 1)
    moe.set_schedule(pk.SCHED_AUTO)
    again = moe.forward(x, lg)
    moe.check()
    assert torch.equal(again.float(), full)
    moe.close()


def test_plan_uses_the_paper_s_workload_terms_in_ep_mode():
    cfg = wl.MoEConfig("ep_plan", 94, T=2048, H=1024, I=512, E=64, k=6, zipf_s=1.0)
    inp = wl.make_inputs(cfg)
    x, lg, gu, dn = to_dev(inp)
    moe = pk.WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    geo = moe.geometry()
    N, R, r = geo["n_sm"], 4, 2
    moe.set_expert_parallel(r, R)
    idx_f = np.arange(N + 1, dtype=np.float64)
    bw = (3.0e4 * idx_f).astype(np.float32); bw[0] = bw[1]
    tf = (1.2e9 * np.sqrt(idx_f / N)).astype(np.float32); tf[0] = tf[1]
    eff = np.array([1.0, 0.8, 0.6, 0.4], np.float32)
    moe.set_cost_tables(bw, tf, eff, 0.7, 2, N // 2, 2)
    moe.forward(x, lg)
    moe.check()
    ref, (xl, xi, xu) = _check_rank(moe, inp, r, R)
    # GEMM tiles of the rank for K = 1,2,4,8 from the restricted routing
    nblk = (cfg.T + geo["route_block"] - 1) // geo["route_block"]
    lo, hi = r * (cfg.E // R), (r + 1) * (cfg.E // R)
    fine = np.zeros((8, cfg.E), np.int64)
    for t in range(cfg.T):
        f = ((t // geo["route_block"]) * 8) // nblk
        for e in ref.idx[t]:
            if lo <= e < hi:
                fine[f, e] += 1
    nt = cfg.I // geo["tile_n0"] + (cfg.H + geo["tile_n1"] - 1) // geo["tile_n1"]
    tiles = []
    for K in (1, 2, 4, 8):
        g = 8 // K
        tiles.append(sum(int(((fine[j * g:(j + 1) * g].sum(0) + geo["gemm_tile_m"] - 1) // geo["gemm_tile_m"]).sum())
                         for j in range(K)) * nt)
    for kinds in (7, 15, 1):      # the default kinds, all four, the paper's split alone
        moe.set_model_options(kinds, -1)
        moe.forward(x, lg)
        moe.check()
        tab = cm.CostTables(N, bw, tf, eff, 0.7, 2, N // 2, 2, steal_workers=N // 2, max_segments=1024, kinds=kinds)
        want = cm.plan(tab, cfg.T, 0, cfg.H, cfg.I, tiles, w=cm.workloads_ep(xl, xi, xu, cfg.H, cfg.I), n_experts=cfg.E)
        got = moe.plan()
        assert (got["kind"], got["c"], got["K"], got["n_steal"]) == (want.kind, want.c, want.K, want.n_steal), (got, want)
    moe.close()


def test_c5_shaped_rank_share_sampled():
    """Config 5's optional mode: 32 local experts of 128, 4 token shards, rank 0, sampled tokens."""
    cfg = wl.CONFIGS["c5_qwen3_235b"]
    inp = wl.make_inputs(cfg)
    x, lg, gu, dn = to_dev(inp)
    moe = pk.WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    moe.set_expert_parallel(0, 4)
    out = moe.forward(x, lg)
    moe.check()
    _, (xl, xi, xu) = _check_rank(moe, inp, 0, 4)
    assert xu <= xi and xl + xi > 0
    # a sample that reaches every local expert's first and last row and every local m-block
    toks, cov = coverage_token_sample(oracle.routing_ep(inp.logits, cfg.k, 0, 4), cfg, 8, None,
                                      moe.geometry()["block_m"], seed=5)
    print(f"[coverage] c5 rank 0 of 4: {cov}")
    assert cov["experts"] == cov["experts_nonempty"] and cov["m_blocks"] == cov["m_blocks_total"], cov
    ref = oracle.moe_tokens_ep(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, toks, 0, 4)
    check_values(bf16_to_np(out[torch.from_numpy(toks).long().cuda()]), ref, "c5 rank 0")
    moe.close()


@pytest.mark.parametrize("seed", range(16))
def test_random_groups_shapes_and_ranks(seed):
    """Seeded random EP groups: one rank's routing, descriptors and partial output against the oracle."""
    rng = np.random.default_rng(7000 + seed)
    R = int(rng.choice([2, 4, 8]))
    E = R * int(rng.choice([1, 2, 4, 8]))
    k = int(rng.integers(1, min(E, 8) + 1))
    T = int(rng.choice([1, 5, 64, 130, 300, 700]))
    H = int(rng.choice([128, 256, 640]))
    I = int(rng.choice([128, 384]))
    zipf = [None, 1.0, 3.0][int(rng.integers(0, 3))]
    cfg = wl.MoEConfig(f"ep_rand{seed}", 300 + seed, T=T, H=H, I=I, E=E, k=k, zipf_s=zipf)
    inp = wl.make_inputs(cfg)
    x, lg, gu, dn = to_dev(inp)
    moe = pk.WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    r = int(rng.integers(0, R))
    moe.set_expert_parallel(r, R)
    if rng.random() < 0.5:
        K = int(rng.choice([1, 2, 4]))
        moe.set_schedule(pk.SCHED_FIXED, int(rng.integers(2, 60)), K, int(rng.integers(0, 20)))
    out = moe.forward(x, lg)
    moe.check()
    _check_rank(moe, inp, r, R)
    ref = oracle.moe_tokens_ep(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, np.arange(cfg.T, dtype=np.int32), r, R)
    if np.abs(ref).max() > 0:
        check_values(bf16_to_np(out), ref, f"seed {seed} rank {r}/{R}")
    else:
        assert bool((out == 0).all())
    moe.close()


@pytest.mark.parametrize("T", [50, 64, 128])
def test_small_batch_every_rank_routing_descriptors_and_output(T):
    """Batches on both sides of the limit below which every CTA routes the batch for itself (remote tokens
    are then staged from the masks in shared memory): permutation, workload descriptors and partial output
    of every rank of a group of 4, in every schedule."""
    cfg = wl.MoEConfig(f"ep_small_batch_T{T}", 95, T=T, H=256, I=384, E=16, k=4, zipf_s=1.0)
    inp = wl.make_inputs(cfg)
    x, lg, gu, dn = to_dev(inp)
    moe = pk.WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    R = 4
    toks = np.arange(cfg.T, dtype=np.int32)
    for r in range(R):
        moe.set_expert_parallel(r, R)
        ref = oracle.moe_tokens_ep(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, toks, r, R)
        for sched in [(pk.SCHED_AUTO, 0, 1, 0), (pk.SCHED_SERIAL, 0, 1, 0), (pk.SCHED_FIXED, 12, 2, 3)]:
            moe.set_schedule(*sched)
            out = moe.forward(x, lg)
            moe.check()
            _check_rank(moe, inp, r, R)
            if np.abs(ref).max() > 0:
                check_values(bf16_to_np(out), ref, f"T {T} rank {r} schedule {sched}")
            else:
                assert bool((out == 0).all())
    moe.close()
