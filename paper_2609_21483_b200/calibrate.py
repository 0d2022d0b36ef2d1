"""Calibration of the cost model's hardware tables on the GPU at hand, and the (c, K) grid sweep.

The paper's cost model is fed measured hardware tables: movement bandwidth and GEMM throughput, each
as a function of the number of SMs given to it (Section 3, Figures 4 and 7), an overlap ratio alpha
(Section 3.1) and a chunking efficiency eff_chunk(K) (Section 3.2.1, Figure 9a).  This module measures them for one layer shape
from the kernel's own timeline:

  BW(c)        movement bytes of dispatch / time the c movement SMs needed for it, while the other
               SMs run GEMM tiles (forced schedule c, K=1, no stealing)
  TFLOPS(n)    useful FLOPs of the GEMM tiles finished after dispatch ended / that time span, with
               n = N - c GEMM SMs (same runs)
  eff_chunk(K) useful GEMM FLOP rate at K chunks / the rate at K=1, both after dispatch has ended
               (a quarter of the SMs dispatch, then every SM works on the GEMM queue)
  alpha        1 - tail * BW(c) / W_combine, tail = time from the last GEMM tile to the kernel end

and can sweep the whole (c, K) grid to compare the model's pick with the measured optimum
(Section 5.5's accuracy experiment).

    python -m paper_2609_21483_b200.calibrate --config c3_qwen3_30b [--grid]
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

C_POINTS = (2, 4, 8, 12, 16, 24, 32, 48, 64, 74)
K_POINTS = (1, 2, 4, 8)


def _events(moe):
    rows = []
    for cta, a in enumerate(moe.read_trace()):
        for r in a:
            rows.append((cta, int(r[0]), int(r[1]), int(r[2]) >> 24, int(r[2]) & 0xFFFFFF, int(r[3])))
    ev = np.array(rows, dtype=np.int64)
    t0 = ev[:, 1].min()
    ev[:, 1] -= t0
    ev[:, 2] -= t0
    ev[:, 2] = np.where(ev[:, 2] < ev[:, 1], ev[:, 2] + (1 << 32), ev[:, 2])
    return ev


def timeline(moe, x, lg, H, I):
    """Runs one traced forward; returns a dict of windows (us) and padded GEMM FLOPs over time."""
    import torch
    moe.forward(x, lg)
    moe.forward(x, lg)
    torch.cuda.synchronize()
    moe.check()
    ev = _events(moe)
    us = lambda v: v / 1e3
    d = ev[ev[:, 3] == 4]
    e6 = ev[ev[:, 3] == 6]
    typ = e6[:, 5] >> 16
    flops = 2.0 * 128 * 256 * np.where((typ == 0) | (typ == 3), H, I)      # gemm0 (regular, swapped) : gemm1
    out = {"end": us(ev[:, 2].max()), "gemm_first": us(e6[:, 1].min()), "gemm_last": us(e6[:, 2].max()),
           "gemm_ends": us(e6[:, 2]), "gemm_flops": flops}
    if len(d):
        out["disp_start"], out["disp_end"] = us(d[:, 1].min()), us(d[:, 2].max())
    return out


def calibrate(cfg, layer=0, verbose=True):
    import torch
    import workloads as wl
    import paper_2609_21483_b200 as pk

    inp = wl.make_inputs(cfg, layer)
    as_bf16 = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()
    x, gu, dn = as_bf16(inp.x), as_bf16(inp.gate_up), as_bf16(inp.down)
    lg = torch.from_numpy(inp.logits).cuda()
    moe = pk.WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    moe.enable_trace(16384)
    N = moe.geometry()["n_sm"]
    P = cfg.P
    w_comp = P * 6.0 * cfg.H * cfg.I
    w_disp = (cfg.T + P) * 2.0 * cfg.H
    w_comb = (P + cfg.T) * 2.0 * cfg.H

    bw_pts, tf_pts, alpha_pts = {}, {}, []
    for c in C_POINTS:
        if c > N - 2:
            continue
        moe.set_schedule(pk.SCHED_FIXED, c, 1, 0)
        tl = timeline(moe, x, lg, cfg.H, cfg.I)
        padded = tl["gemm_flops"].sum()
        useful = w_comp / padded
        t_disp = tl["disp_end"] - tl["disp_start"]
        bw_pts[c] = w_disp / t_disp                                   # byte/us
        after = tl["gemm_ends"] > tl["disp_end"]
        span = tl["gemm_last"] - tl["disp_end"]
        if after.sum() > 10 and span > 0:
            tf_pts[N - c] = tl["gemm_flops"][after].sum() * useful / span   # FLOP/us
        tail = tl["end"] - tl["gemm_last"]
        alpha_pts.append(1.0 - tail * bw_pts[c] / w_comb)
        if verbose:
            print(f"c={c:3d}: dispatch {t_disp:8.1f} us -> BW {bw_pts[c]/1e3:8.1f} GB/s; "
                  f"GEMM on {N-c:3d} SMs {tf_pts.get(N-c, float('nan'))/1e6:8.1f} TFLOP/s; tail {tail:6.1f} us; "
                  f"layer {tl['end']:8.1f} us", flush=True)

    eff = []
    base = None
    for K in K_POINTS:
        if K * (cfg.E + cfg.S) > 1024:
            eff.append(eff[-1] * 0.8)
            continue
        # a quarter of the SMs dispatch quickly, then everybody works on the GEMM queue: the rate of
        # useful FLOPs after dispatch ended is the chunked GEMM throughput
        moe.set_schedule(pk.SCHED_FIXED, N // 4, K, 1 << 20)
        tl = timeline(moe, x, lg, cfg.H, cfg.I)
        after = tl["gemm_ends"] > tl["disp_end"]
        rate = tl["gemm_flops"][after].sum() * (w_comp / tl["gemm_flops"].sum()) / (tl["gemm_last"] - tl["disp_end"])
        base = rate if base is None else base
        eff.append(float(min(1.0, rate / base)))
        if verbose:
            print(f"K={K}: GEMM rate {rate/1e6:8.1f} TFLOP/s -> eff_chunk {eff[-1]:.3f}; layer {tl['end']:8.1f} us", flush=True)

    def interp(pts, n_max):
        xs = np.array(sorted(pts))
        # more SMs are never modelled as slower than fewer (the extra ones could stay idle): measured
        # rates of a small layer saturate and then wobble with the noise
        ys = np.maximum.accumulate(np.array([pts[v] for v in xs]))
        grid = np.arange(n_max + 1, dtype=np.float64)
        out = np.interp(grid, np.concatenate([[0], xs]), np.concatenate([[0], ys]))
        out[0] = out[1]
        return out.astype(np.float32)

    tables = {"n_sm": N, "bw": interp(bw_pts, N), "tflops": interp(tf_pts, N),
              "eff_chunk": np.array(eff, np.float32),
              "alpha": float(np.clip(np.median(alpha_pts), 0.0, 0.99)),
              "c_min": 2, "c_max": N // 2, "c_step": 2}
    return moe, (x, lg), tables


def grid_sweep(moe, xl, cfg, tables, verbose=True, c_points=C_POINTS, reps=3):
    """Measured layer time for every (c, K) of a grid of the paper's split plans, the model's pick
    and the selection gap (the paper reports 8.2 % on its hardware).

    A grid point is AUTO with the candidate set cut down to that one (c, K): the device then runs the
    paper's split at (c, K) with the steal count Eq. 11-14 give at that c, without the elastic
    stealing and the first dispatch wave.  The model's pick is AUTO over the whole grid under the same
    restrictions."""
    import torch
    import paper_2609_21483_b200 as pk
    x, lg = xl
    moe.enable_trace(0)
    res, steal_of = {}, {}
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def time_it(n=5):
        moe.forward(x, lg)
        ev0.record()
        for _ in range(n):
            moe.forward(x, lg)
        ev1.record()
        torch.cuda.synchronize()
        moe.check()
        return ev0.elapsed_time(ev1) / n * 1e3

    def tables_for(c_min, c_max, c_step, only_K=None):
        eff = np.array(tables["eff_chunk"], np.float32)
        if only_K is not None:      # every other chunk count priced out of the arg-min
            eff = np.array([1.0 if K == only_K else 1e-6 for K in K_POINTS], np.float32)
        moe.set_cost_tables(tables["bw"], tables["tflops"], eff, tables["alpha"], c_min, c_max, c_step)

    moe.set_schedule(pk.SCHED_AUTO)
    tables_for(tables["c_min"], tables["c_max"], tables["c_step"])
    moe.set_model_options(7, -1)
    t_auto = time_it()
    plan_auto = moe.plan()
    moe.set_model_options(1 << pk.PLAN_SPLIT, 0)
    time_it(1)
    plan = moe.plan()
    n_sm = tables["n_sm"]
    # the model's own pick is a grid point like the others, measured in the same sweeps: two sweeps in
    # opposite order, so that the clock state the previous points leave behind (a slow K = 8 point lets
    # the part cool down) hits every point from both sides
    cs = sorted({c for c in c_points if c <= n_sm - 2 and c % 2 == 0} | {plan["c"]})
    pts = [(c, K) for c in cs for K in K_POINTS if K * (cfg.E + cfg.S) <= 1024]
    acc = {pt: 0.0 for pt in pts}
    for sweep in (pts, pts[::-1]):
        for c, K in sweep:
            tables_for(c, c, 2, only_K=K)
            acc[(c, K)] += time_it(reps)
            got = moe.plan()
            assert (got["c"], got["K"]) == (c, K), (got, c, K)
            steal_of[f"{c},{K}"] = got["n_steal"]
    res = {pt: v / 2 for pt, v in acc.items()}
    t_pick = res[(plan["c"], plan["K"])]
    tables_for(tables["c_min"], tables["c_max"], tables["c_step"])
    best = min(res, key=res.get)
    moe.set_model_options(7, -1)
    moe.set_schedule(pk.SCHED_SERIAL)
    t_serial = time_it()
    # what the in-kernel search costs: set-up time with and without it, from the timeline
    def setup_us(mode, *a):
        moe.set_schedule(mode, *a)
        moe.enable_trace(4096)
        moe.forward(x, lg)
        moe.forward(x, lg)
        ev = _events(moe)
        moe.enable_trace(0)
        e = ev[ev[:, 3] == 2]
        return float(((e[:, 2] - e[:, 1]) / 1e3).mean())
    su_auto, su_fixed = setup_us(pk.SCHED_AUTO), setup_us(pk.SCHED_FIXED, plan["c"], plan["K"], plan["n_steal"])
    moe.set_schedule(pk.SCHED_AUTO)
    if verbose:
        print("grid (us):")
        for c in cs:
            print(f"  c={c:3d} " + " ".join(f"K={K}:{res.get((c, K), float('nan')):8.1f} (steal {steal_of.get(f'{c},{K}', '-')})"
                                            for K in K_POINTS))
        print(f"AUTO (all plan kinds) {plan_auto} -> {t_auto:.1f} us; measured optimum of the split grid {best} -> "
              f"{res[best]:.1f} us; AUTO vs that {100 * (t_auto / res[best] - 1):+.1f} %; SERIAL {t_serial:.1f} us")
        print(f"model's split pick {plan}: {t_pick:.1f} us, selection gap inside the grid {100 * (t_pick / res[best] - 1):.1f} %; "
              f"set-up {su_auto:.2f} us with the search, {su_fixed:.2f} us without")
    return {"workload": cfg.name, "auto_us": t_auto, "plan_auto": plan_auto, "plan": plan, "best": list(best),
            "best_us": res[best], "pick_us": t_pick, "selection_gap": t_pick / res[best] - 1,
            "auto_vs_best": t_auto / res[best] - 1, "serial_us": t_serial, "setup_us_auto": su_auto,
            "setup_us_fixed": su_fixed, "grid_points": len(res), "steal_of": steal_of}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c3_qwen3_30b")
    ap.add_argument("--layer", type=int, default=0)
    ap.add_argument("--grid", action="store_true")
    ap.add_argument("--out", default="")
    args = ap.parse_args()
    import workloads as wl
    cfg = wl.CONFIGS[args.config]
    moe, xl, tables = calibrate(cfg, args.layer)
    print("alpha", tables["alpha"], "eff_chunk", tables["eff_chunk"].tolist())
    if args.grid:
        print(json.dumps(grid_sweep(moe, xl, cfg, tables)))
    if args.out:
        with open(args.out, "w") as f:
            json.dump({k: (v.tolist() if isinstance(v, np.ndarray) else v) for k, v in tables.items()}, f)
    moe.close()


if __name__ == "__main__":
    main()
