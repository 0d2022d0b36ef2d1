"""Utilisation report from the kernel's own timeline.

The paper's profiling window opens when routing is done and closes when the last combine is; over it
the paper reports SM activity, link utilisation, tensor-core activity and an overlap ratio: the share
of the window in which data movement and tensor-core work are both under way (Section 5.4, Figure 11;
Figure 8 draws the SMs' roles over time).  On one GPU the movement is the dispatch and combine traffic through
HBM.  The kernel records one event per tile and per CTA (weave_moe_set_trace); this module turns
the records into the same quantities:

  sm_busy          mean over CTAs of the fraction of the window covered by that CTA's tiles
                   (set-up, dispatch, GEMM main loops and epilogues, combine; waits are idle)
  movement_active  fraction of the window with at least one dispatch or combine tile live
  tensor_active    fraction of the window with at least one GEMM main loop live
  overlap_ratio    fraction of the window with both (the paper's definition)
  mean_ctas_*      time-averaged number of CTAs in each role (how wide the overlap is)
  *_GBps, gemm_TFLOPs   payload rates over the time each kind of work was live

    python -m paper_2609_21483_b200.timeline --config c4_dsv2lite_T1024 [--sched auto|serial|fixed:c:K:steal]
                                            [--ascii timeline.txt]

analyse() is plain numpy over the event arrays, so it is testable without a GPU.
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

# event kinds written by the kernel
EV_ROUTE, EV_SETUP, EV_FIXUP, EV_DISPATCH, EV_CLAIM, EV_EPILOGUE, EV_COMBINE, EV_WAIT_CHUNK, EV_BARRIER = range(1, 10)
EV_MMA = 11
_BUSY_KINDS = (EV_SETUP, EV_FIXUP, EV_DISPATCH, EV_EPILOGUE, EV_COMBINE, EV_MMA)


def flatten(trace):
    """list (one per CTA) of [n,4] uint32 records -> int64 array [m,6] = cta, start, end, kind, id, extra
    with times in ns relative to the first event (the counter's low 32 bits may wrap once)."""
    rows = []
    for cta, a in enumerate(trace):
        a = np.asarray(a, dtype=np.uint32).reshape(-1, 4).astype(np.int64)
        if len(a):
            rows.append(np.column_stack([np.full(len(a), cta), a[:, 0], a[:, 1], a[:, 2] >> 24, a[:, 2] & 0xFFFFFF, a[:, 3]]))
    if not rows:
        return np.zeros((0, 6), np.int64)
    ev = np.concatenate(rows)
    # the records hold the low 32 bits of a ns counter: take every stamp as a signed distance (within
    # +-2.1 s) from one reference stamp, which undoes a wrap in the middle of the kernel
    ref = ev[0, 1]
    for col in (1, 2):
        ev[:, col] = ((ev[:, col] - ref + (1 << 31)) % (1 << 32)) - (1 << 31)
    t0 = ev[:, 1].min()
    ev[:, 1] -= t0
    ev[:, 2] -= t0
    return ev


def _coverage(starts, ends, breaks):
    """number of intervals [start, end) covering each segment between consecutive breakpoints"""
    cnt = np.zeros(len(breaks), np.int64)
    np.add.at(cnt, np.searchsorted(breaks, starts), 1)
    np.add.at(cnt, np.searchsorted(breaks, ends), -1)
    return np.cumsum(cnt)[:-1]


def _busy_intervals(ev, n_cta):
    """(cta, start, end) of everything that counts as work.  A GEMM main loop is recorded by the pair's
    leader (even CTA) and keeps both CTAs' tensor cores busy; the time it waited for a free accumulator
    (extra, ns) is not work."""
    out = []
    for kind in _BUSY_KINDS:
        e = ev[ev[:, 3] == kind]
        if not len(e):
            continue
        if kind == EV_MMA:
            s = np.minimum(e[:, 1] + e[:, 5], e[:, 2])
            out.append(np.column_stack([e[:, 0], s, e[:, 2]]))
            peer = e[:, 0] + 1
            ok = peer < n_cta
            out.append(np.column_stack([peer[ok], s[ok], e[ok, 2]]))
        else:
            out.append(e[:, :3])
    return np.concatenate(out) if out else np.zeros((0, 3), np.int64)


def analyse(trace, shape=None):
    """trace: what WeaveMoE.read_trace() returns.  shape: optional dict with T, H, I, k, S for the rates."""
    n_cta = len(trace)
    ev = flatten(trace)
    if not len(ev):
        raise ValueError("empty trace")
    setup = ev[ev[:, 3] == EV_SETUP]
    route = ev[ev[:, 3] == EV_ROUTE]
    w0 = int(setup[:, 1].min()) if len(setup) else (int(route[:, 2].max()) if len(route) else 0)
    w1 = int(ev[:, 2].max())
    window = max(w1 - w0, 1)

    busy = _busy_intervals(ev, n_cta)
    busy[:, 1] = np.clip(busy[:, 1], w0, w1)
    busy[:, 2] = np.clip(busy[:, 2], w0, w1)
    per_cta = np.zeros(n_cta)
    for c in range(n_cta):
        b = busy[busy[:, 0] == c]
        if len(b):
            br = np.unique(np.concatenate([b[:, 1], b[:, 2]]))
            cov = _coverage(b[:, 1], b[:, 2], br)
            per_cta[c] = (np.diff(br) * (cov > 0)).sum() / window

    mv = ev[(ev[:, 3] == EV_DISPATCH) | (ev[:, 3] == EV_COMBINE)]
    mm = ev[ev[:, 3] == EV_MMA]
    mm_s = np.minimum(mm[:, 1] + mm[:, 5], mm[:, 2])
    breaks = np.unique(np.concatenate([[w0, w1], np.clip(mv[:, 1], w0, w1), np.clip(mv[:, 2], w0, w1),
                                       np.clip(mm_s, w0, w1), np.clip(mm[:, 2], w0, w1)]))
    seg = np.diff(breaks)
    n_mv = _coverage(np.clip(mv[:, 1], w0, w1), np.clip(mv[:, 2], w0, w1), breaks)
    n_mm = _coverage(np.clip(mm_s, w0, w1), np.clip(mm[:, 2], w0, w1), breaks)
    rep = {
        "n_cta": n_cta,
        "window_us": window / 1e3,
        "routing_us": w0 / 1e3,
        "sm_busy": float(per_cta.mean()),
        "sm_busy_min": float(per_cta.min()),
        "movement_active": float((seg * (n_mv > 0)).sum() / window),
        "tensor_active": float((seg * (n_mm > 0)).sum() / window),
        "overlap_ratio": float((seg * ((n_mv > 0) & (n_mm > 0))).sum() / window),
        "mean_ctas_moving": float((seg * n_mv).sum() / window),
        "mean_ctas_gemm": float((seg * n_mm).sum() * 2 / window),
        "events": int(len(ev)),
    }
    if shape is not None:
        T, H, I = shape["T"], shape["H"], shape["I"]
        P = T * (shape["k"] + shape.get("S", 0))
        us = lambda kind: _union_us(ev[ev[:, 3] == kind])
        td, tc, tg = us(EV_DISPATCH), us(EV_COMBINE), (seg * (n_mm > 0)).sum() / 1e3
        if td > 0:
            rep["dispatch_GBps"] = 2.0 * P * H * 2 / td / 1e3        # every row read once and written once
        if tc > 0:
            rep["combine_GBps"] = (P + T) * H * 2.0 / tc / 1e3
        if tg > 0:
            rep["gemm_TFLOPs"] = P * 6.0 * H * I / tg / 1e6
    return rep


def _union_us(e):
    if not len(e):
        return 0.0
    br = np.unique(np.concatenate([e[:, 1], e[:, 2]]))
    return float((np.diff(br) * (_coverage(e[:, 1], e[:, 2], br) > 0)).sum() / 1e3)


def ascii_timeline(trace, width=120):
    """One text row per CTA: what it mostly did in each of `width` equal slices of the kernel
    (R routing, s set-up, D dispatch, G GEMM, C combine, '.' idle or waiting)."""
    n_cta = len(trace)
    ev = flatten(trace)
    end = int(ev[:, 2].max())
    edges = np.linspace(0, end, width + 1)
    classes = [("R", (EV_ROUTE,)), ("s", (EV_SETUP, EV_FIXUP)), ("D", (EV_DISPATCH,)), ("G", (EV_MMA, EV_EPILOGUE)),
               ("C", (EV_COMBINE,))]
    occ = np.zeros((len(classes), n_cta, width))
    for ci, (_, kinds) in enumerate(classes):
        for kind in kinds:
            e = ev[ev[:, 3] == kind]
            if kind == EV_MMA and len(e):
                peer = e.copy()
                peer[:, 0] += 1
                e = np.concatenate([e, peer[peer[:, 0] < n_cta]])
            for cta, s, t in e[:, :3]:
                a, b = np.searchsorted(edges, [s, t], side="right") - 1
                for w in range(max(a, 0), min(b, width - 1) + 1):
                    occ[ci, cta, w] += max(0.0, min(t, edges[w + 1]) - max(s, edges[w]))
    lines = [f"one column = {end / width / 1e3:.1f} us; R routing, s set-up, D dispatch, G GEMM, C combine, . idle"]
    slice_ns = end / width
    for c in range(n_cta):
        row = []
        for w in range(width):
            ci = int(np.argmax(occ[:, c, w]))
            row.append(classes[ci][0] if occ[ci, c, w] > 0.25 * slice_ns else ".")
        lines.append(f"{c:3d} " + "".join(row))
    return "\n".join(lines)


def run(cfg, sched="auto", layer=0, events_per_cta=16384):
    """One traced forward of a seeded workload; returns (report, trace)."""
    import torch
    import workloads as wl
    import paper_2609_21483_b200 as pk

    inp = wl.make_inputs(cfg, layer)
    as_bf16 = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()
    moe = pk.WeaveMoE(as_bf16(inp.gate_up), as_bf16(inp.down), cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    if sched == "serial":
        moe.set_schedule(pk.SCHED_SERIAL)
    elif sched == "split":          # AUTO restricted to the paper's plan kind (a spatial split)
        moe.set_model_options(1 << pk.PLAN_SPLIT, -1)
    elif sched.startswith("fixed"):
        _, c, K, s = sched.split(":")
        moe.set_schedule(pk.SCHED_FIXED, int(c), int(K), int(s))
    x, lg = as_bf16(inp.x), torch.from_numpy(inp.logits).cuda()
    for _ in range(3):
        moe.forward(x, lg)
    moe.enable_trace(events_per_cta)
    moe.forward(x, lg)
    moe.forward(x, lg)
    torch.cuda.synchronize()
    moe.check()
    trace = moe.read_trace()
    rep = analyse(trace, {"T": cfg.T, "H": cfg.H, "I": cfg.I, "k": cfg.k, "S": cfg.S})
    rep["plan"] = moe.plan()
    rep["workload"], rep["sched"] = cfg.name, sched
    return rep, trace


def main(argv=None):
    import workloads as wl
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--config", default="c4_dsv2lite_T1024")
    ap.add_argument("--sched", default="auto", help="auto | split | serial | fixed:c:K:steal")
    ap.add_argument("--ascii", default=None, help="write the per-CTA text timeline to this file")
    a = ap.parse_args(argv)
    rep, trace = run(wl.CONFIGS[a.config], a.sched)
    print(json.dumps(rep))
    if a.ascii:
        with open(a.ascii, "w") as f:
            f.write(ascii_timeline(trace) + "\n")


if __name__ == "__main__":
    main()
