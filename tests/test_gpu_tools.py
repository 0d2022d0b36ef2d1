"""GPU checks of the measurement tools: the in-kernel timeline and the calibration of the cost
model's tables (both go through the C ABI)."""
import numpy as np
import pytest
import torch

import workloads as wl
import paper_2609_21483_b200 as pk
from parity import to_dev

pytestmark = pytest.mark.gpu


def test_timeline_accounts_for_every_tile_exactly_once():
    """Every dispatch tile (m-block), every combine tile and every (m-block, n-tile) GEMM epilogue
    appears exactly once in the trace, whatever the schedule; tracing does not change the output."""
    cfg = wl.MoEConfig("trace", 91, T=1000, H=512, I=768, E=16, k=4, zipf_s=1.0)
    inp = wl.make_inputs(cfg)
    x, lg, gu, dn = to_dev(inp)
    moe = pk.WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    ref = moe.forward(x, lg).clone()
    moe.check()
    geo = moe.geometry()
    counts = moe.routing(cfg.T)["counts"].cpu().numpy()
    moe.enable_trace(4096)
    for sched in [(pk.SCHED_AUTO, 0, 1, 0), (pk.SCHED_SERIAL, 0, 1, 0), (pk.SCHED_FIXED, 10, 2, 3)]:
        moe.set_schedule(*sched)
        out = moe.forward(x, lg)
        moe.check()
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
        ev = np.concatenate([a for a in moe.read_trace() if len(a)])
        kind, ident = ev[:, 2] >> 24, ev[:, 2] & 0xFFFFFF
        K = moe.plan()["K"]
        # m-blocks: per (chunk, expert) segment ceil(rows/128); recompute from the routing
        nblk = (cfg.T + geo["route_block"] - 1) // geo["route_block"]
        idx = moe.routing(cfg.T)["topk_idx"].cpu().numpy()
        seg = np.zeros((K, cfg.E), np.int64)
        for t in range(cfg.T):
            j = (((t // geo["route_block"]) * 8) // nblk) // (8 // K)
            seg[j, idx[t]] += 1
        n_mb = int(((seg + geo["block_m"] - 1) // geo["block_m"]).sum())
        disp = np.sort(ident[kind == 4])
        np.testing.assert_array_equal(disp, np.arange(n_mb))
        comb = np.sort(ident[kind == 7])
        ct = geo["combine_tile"]          # halved until every SM has a combine tile
        while ct > 1 and (cfg.T + ct - 1) // ct < geo["n_sm"]:
            ct //= 2
        np.testing.assert_array_equal(comb, np.arange((cfg.T + ct - 1) // ct))
        nt = cfg.I // geo["tile_n0"] + (cfg.H + geo["tile_n1"] - 1) // geo["tile_n1"]
        epi = ident[kind == 6]
        # regular tiles report once per m-block and n-tile; a swapped (unpaired) m-block is finished
        # by both CTAs of its pair and reports twice
        odd = int((((seg + geo["block_m"] - 1) // geo["block_m"]) % 2).sum())
        assert len(epi) == (n_mb + odd) * nt
        assert set(epi.tolist()) == set(range(n_mb))
        assert (ev[:, 1].astype(np.int64) - ev[:, 0].astype(np.int64) >= 0).mean() > 0.99   # 32-bit wrap aside
    assert counts.sum() == cfg.T * cfg.k
    moe.close()


def test_calibration_produces_usable_tables_and_auto_follows_them():
    from paper_2609_21483_b200 import calibrate
    cfg = wl.CONFIGS["c4_dsv2lite_T1024"]
    moe, (x, lg), tab = calibrate.calibrate(cfg, verbose=False)
    n = tab["n_sm"]
    assert tab["bw"].shape == (n + 1,) and tab["tflops"].shape == (n + 1,)
    assert (np.diff(tab["bw"][1:n // 2]) >= 0).all()            # more movement SMs never move less
    assert 0 < tab["bw"][2] < tab["bw"][n // 2]
    assert tab["eff_chunk"][0] == 1.0 and (np.diff(tab["eff_chunk"]) <= 1e-6).all()
    assert 0.0 <= tab["alpha"] < 1.0
    moe.enable_trace(0)
    moe.set_cost_tables(tab["bw"], tab["tflops"], tab["eff_chunk"], tab["alpha"], tab["c_min"], tab["c_max"],
                        tab["c_step"])
    moe.set_schedule(pk.SCHED_AUTO)
    moe.set_model_options(1 << pk.PLAN_SPLIT, -1)         # the paper's plan kind alone
    moe.forward(x, lg)
    moe.check()
    p = moe.plan()
    assert p["kind"] == pk.PLAN_SPLIT
    assert 2 <= p["c"] <= n // 2 and p["c"] % 2 == 0 and p["K"] in (1, 2, 4, 8) and p["t_total_us"] > 0
    moe.set_model_options(7, -1)                          # the default kinds: the phased plan reports c = n_sm
    moe.forward(x, lg)
    moe.check()
    q = moe.plan()
    assert q["t_total_us"] <= p["t_total_us"] and (q["c"] == n) == (q["kind"] == pk.PLAN_PHASED)
    moe.close()


def test_grid_sweep_compares_the_model_s_pick_with_the_forced_grid():
    """The (c, K) sweep of the accuracy experiment (Section 5.5) on a small shape: every grid point is
    the paper's split forced to one (c, K) with the steal count Eq. 11-14 give at that c; the model's
    own pick must be one of the candidates and its gap to the measured optimum finite."""
    from paper_2609_21483_b200 import calibrate
    cfg = wl.CONFIGS["c4_dsv2lite_T256"]
    moe, xl, tab = calibrate.calibrate(cfg, verbose=False)
    rep = calibrate.grid_sweep(moe, xl, cfg, tab, verbose=False, c_points=(4, 16, 48), reps=2)
    assert rep["grid_points"] in (3 * 4, 4 * 4)          # the model's pick joins the grid when it is not on it
    assert rep["plan"]["kind"] == pk.PLAN_SPLIT and 2 <= rep["plan"]["c"] <= tab["n_sm"] // 2
    assert np.isfinite(rep["selection_gap"]) and rep["selection_gap"] >= 0.0
    assert rep["best_us"] > 0 and rep["pick_us"] >= rep["best_us"]
    # the steal quota moves with c: fewer movement SMs finish later, so less is left to steal
    steals = {c: rep["steal_of"][f"{c},1"] for c in (4, 16, 48)}
    assert steals[4] <= steals[16] <= steals[48]
    assert rep["auto_us"] > 0 and rep["serial_us"] > 0
    moe.close()


@pytest.mark.gpu
def test_utilisation_report_from_the_kernel_timeline():
    """The paper's spatial split overlaps movement with tensor-core work; with barriers between the
    phases nothing overlaps."""
    from paper_2609_21483_b200 import timeline
    cfg = wl.CONFIGS["c3_qwen3_30b"].with_T(4096)
    auto, trace = timeline.run(cfg, "split")
    serial, _ = timeline.run(cfg, "serial")
    for rep in (auto, serial):
        assert 0.0 < rep["sm_busy"] <= 1.0 and 0.0 < rep["tensor_active"] <= 1.0
        assert rep["overlap_ratio"] <= min(rep["movement_active"], rep["tensor_active"]) + 1e-9
        assert rep["gemm_TFLOPs"] > 0 and rep["dispatch_GBps"] > 0 and rep["combine_GBps"] > 0
    assert auto["overlap_ratio"] > 0.05
    assert serial["overlap_ratio"] < 0.01
    txt = timeline.ascii_timeline(trace, width=60).splitlines()
    assert len(txt) == auto["n_cta"] + 1 and any("G" in l for l in txt[1:])
