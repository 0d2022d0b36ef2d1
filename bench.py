#!/usr/bin/env python
"""Benchmark of the MoE-layer megakernel: layer latency, tokens/s, fraction of the layer roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

A step is one pass of the whole hot path (routing, dispatch, grouped SwiGLU GEMMs, combine: one
kernel launch per layer) over one batch of seeded synthetic input.  The default workload is the
largest single-GPU configuration: a stack of 24 Qwen3-235B-A22B-shaped layers (T=16384, H=4096,
I=1536, E=128, top-8, a fresh routing skew per layer), one step = 24 launches.  One JSON line is
printed by rank 0; with the default workload it also carries a `per_config` list with the other
configurations of record (Mixtral-shaped, Qwen3-30B-shaped, DSv2-Lite-shaped decode batches, the
tiny layer), each with its burst-window and sustained-run roofline fractions and the scheduler
ablation.

With --gpus N > 1 the script starts N ranks of itself under torch.distributed.run (or runs as one of
them when it was started that way): every rank runs an independent replica of the layer on its own
GPU (the path has no cross-GPU exchange step on one node: "replicas only"); the value is the number
of tokens all ranks processed divided by the slowest rank's device time.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"
DEFAULT_CONFIG = "c5_qwen3_235b"
PER_CONFIG = ["c2_mixtral", "c3_qwen3_30b", "c4_dsv2lite_T64", "c4_dsv2lite_T256", "c4_dsv2lite_T1024", "c1_tiny"]

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the megakernel, from the ncu
# captures summarised under profiles/ (None = not captured).  The Qwen3-235B-shaped layer's figure is
# the mean of three launches captured whole with the time and DRAM counters only (one pass).
NCU_DRAM_BYTES_PER_LAUNCH = {"c2_mixtral": 4.297e9, "c3_qwen3_30b": 2.603e9, "c5_qwen3_235b": 11.2e9,
                             "c5_quarter": 2.991e9}


def load_peaks():
    """Measured roofline denominators (MEASURED_PEAKS.json beside this file), else the documented fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def layer_work(cfg, active_experts=None):
    """Algorithmic FLOPs and bytes of one layer (per launch).
    FLOPs = P * 6*H*I (Eq. 1).  Bytes = what the method itself moves, each intermediate written
    once and read once: logits, routing, dispatch (T rows read, P written), gemm0 reads P rows and
    the weights, h written and read, y written and read, out written."""
    T, H, I, E, k, S = cfg.T, cfg.H, cfg.I, cfg.E, cfg.k, cfg.S
    P = T * (k + S)
    ea = (E + S) if active_experts is None else active_experts
    flops = P * 6.0 * H * I
    weights = ea * 3.0 * H * I * 2
    act = (4.0 * T * E + 8.0 * T * k + (T + P) * 2.0 * H + P * 2.0 * H + 2 * P * 2.0 * I + 2 * P * 2.0 * H
           + T * 2.0 * H)
    return {"flops": flops, "bytes": weights + act, "weights_bytes": weights, "act_bytes": act,
            "movement_bytes": (T + P) * 2.0 * H + (P + T) * 2.0 * H}


def roofline_of(work, layer_s, peaks, window):
    """Roofline entry of one layer time.  window = "burst" (a timed region well under half a second that
    starts from idle clocks: compared with the burst bf16 peak) or "sustained" (a back-to-back run of
    seconds under the power cap: compared with the sustained bf16 peak).  The bound is decided with the
    peak of the same window; the HBM copy bandwidth has one measured figure."""
    tf_peak = peaks["bf16_tflops_sustained"] if window == "sustained" else peaks["bf16_tflops"]
    t_flops = work["flops"] / (tf_peak * 1e12)
    t_bytes = work["bytes"] / (peaks["hbm_gbs"] * 1e9)
    if t_flops >= t_bytes:
        bound, achieved, peak, unit = "tensor", work["flops"] / layer_s / 1e12, tf_peak, "TFLOP/s"
    else:
        bound, achieved, peak, unit = "hbm", work["bytes"] / layer_s / 1e9, peaks["hbm_gbs"], "GB/s"
    return {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            "window": window, "layer_roofline_us": max(t_flops, t_bytes) * 1e6}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.idx}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [s.strip() for s in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [s for s, p in zip(sm, pw) if p > 0.5 * max(pw)] or sm
        return {"sm_mhz": float(np.median(busy)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "power_w_max": float(max(pw)), "samples": len(sm)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def aggregate_max(value: float, world: int, use_cuda: bool) -> float:
    """Max over ranks of a per-rank time (all-reduce MAX); identity for one process."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device="cuda" if use_cuda else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(tokens_per_rank_step: int, steps: int, world: int, max_seconds: float) -> float:
    return tokens_per_rank_step * steps * world / max_seconds


def launch_ranks(n: int, argv) -> int:
    """Starts n ranks of this script on this node under torch.distributed.run and returns its exit code."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def launcher_selftest(args):
    """The multi-rank plumbing without a GPU: gloo ranks, the slowest rank's time decides, rank 0
    prints the line.  Used by the CPU tests to exercise `--gpus N` as a user starts it."""
    import torch.distributed as dist
    rank, world, _ = dist_env()
    if world > 1:
        dist.init_process_group("gloo")
    sec = aggregate_max(1.0 + rank, world, use_cuda=False)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"launcher_selftest": True, "n_gpus": world, "max_seconds": sec,
                          "value": whole_job_throughput(4096, args.steps, world, sec)}), flush=True)


def host_weights_for(cfg, wl, oracle, logits, toks):
    """Host weight arrays for the oracle in which only the experts the sampled tokens use are filled
    in (zero pages that are never touched cost no memory), so that 20 GB layers stay benchable."""
    idx, _ = oracle.route(np.ascontiguousarray(logits[toks]), cfg.k)
    need = sorted(set(idx.ravel().tolist()) | set(range(cfg.E, cfg.E + cfg.S)))
    EE = cfg.E + cfg.S
    gu = np.zeros((EE, 2 * cfg.I, cfg.H), np.uint16)
    dn = np.zeros((EE, cfg.H, cfg.I), np.uint16)
    for e in need:
        gu[e], dn[e] = wl.expert_weights(cfg, e)
    return gu, dn


def cpu_sample_size(oracle, wl, inp, cfg, seconds: float) -> int:
    """How many tokens the oracle gets through in about `seconds` on this host: time a probe of
    8 tokens, scale, clamp to [8, T]."""
    probe = wl.stratified_token_sample(cfg.T, 8, seed=99)
    t0 = time.perf_counter()
    oracle.moe_tokens(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, probe, cfg.S)
    per_tok = max((time.perf_counter() - t0) / len(probe), 1e-6)
    return int(min(cfg.T, max(8, seconds / per_tok)))


# --------------------------------------------------------------------------------------- reference arm

def run_reference(args):
    """The reference arm of this tier is the CPU oracle as it stands, timed on the host cores on
    a bounded token sample of the same workload (rank 0 only)."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    import oracle
    import workloads as wl
    cfg = wl.CONFIGS[args.config]
    oracle.build(); wl.build()
    L = cfg.layers
    x_h = wl.make_x(cfg)
    lgs = [wl.make_logits(cfg, l) for l in range(L)]
    probe = wl.stratified_token_sample(cfg.T, 8, seed=99)
    inp = wl.LayerInputs(cfg, x_h, lgs[0], *host_weights_for(cfg, wl, oracle, lgs[0], probe))
    # per step and layer: full-T routing plus the sampled tokens' FFN/combine; the whole run is bounded
    budget = max(2.0, min(args.cpu_seconds, 120.0 / max(args.steps + 1, 1)))
    n = args.ref_tokens if args.ref_tokens > 0 else max(8, cpu_sample_size(oracle, wl, inp, cfg, budget) // L)
    toks = wl.stratified_token_sample(cfg.T, n, seed=cfg.cfg_id)
    need_logits = np.concatenate([lg[toks] for lg in lgs])
    idx, _ = oracle.route(np.ascontiguousarray(need_logits), cfg.k)
    EE = cfg.E + cfg.S
    gu = np.zeros((EE, 2 * cfg.I, cfg.H), np.uint16)
    dn = np.zeros((EE, cfg.H, cfg.I), np.uint16)
    for e in sorted(set(idx.ravel().tolist()) | set(range(cfg.E, EE))):
        gu[e], dn[e] = wl.expert_weights(cfg, e)
    for _ in range(max(args.warmup, 0) and 1):
        oracle.moe_tokens(x_h, lgs[0], gu, dn, cfg.k, toks[:1], cfg.S)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for l in range(L):
            oracle.routing(lgs[l], cfg.k, cfg.S)
            oracle.moe_tokens(x_h, lgs[l], gu, dn, cfg.k, toks, cfg.S)
    dt = time.perf_counter() - t0
    val = len(toks) * L * args.steps / dt
    cores = oracle.num_threads()
    sample = (f"{len(toks)} stratified tokens of T={cfg.T} per layer x {L} layer(s) per step (full-T routing + "
              f"per-token FFN/combine), {args.steps} steps, {dt:.1f} s")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "I": cfg.I, "E": cfg.E, "top_k": cfg.k,
                       "shared": cfg.S, "layers": L},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------- our arm

class Layer:
    """Device tensors and the handle of one workload."""

    def __init__(self, cfg, args, weights=None):
        import torch
        import workloads as wl
        import paper_2609_21483_b200 as pk
        self.cfg, self.pk, self.torch = cfg, pk, torch
        as_bf16 = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
        EE = cfg.E + cfg.S
        if weights is None:
            gu = torch.empty((EE, 2 * cfg.I, cfg.H), dtype=torch.bfloat16, device="cuda")
            dn = torch.empty((EE, cfg.H, cfg.I), dtype=torch.bfloat16, device="cuda")
            for e in range(EE):      # expert by expert: the host never holds the whole (up to 20 GB) tensor
                g_e, d_e = wl.expert_weights(cfg, e)
                gu[e].copy_(as_bf16(g_e))
                dn[e].copy_(as_bf16(d_e))
            weights = (gu, dn)
        self.weights = weights
        self.x_h = as_bf16(wl.make_x(cfg)).pin_memory()
        self.x = self.x_h.cuda()
        self.L = cfg.layers
        self.logits_h = [torch.from_numpy(wl.make_logits(cfg, l)).pin_memory() for l in range(self.L)]
        self.logits = [t.cuda() for t in self.logits_h]
        self.out = torch.empty_like(self.x)
        self.out_h = [torch.empty_like(self.x_h).pin_memory() for _ in range(2)]
        self.moe = pk.WeaveMoE(weights[0], weights[1], cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
        if args.sms:
            self.moe.set_sm_count(args.sms)
        if args.ep > 1:
            self.moe.set_expert_parallel(args.ep_rank, args.ep)
        geo = self.moe.geometry()
        self.fixed_c = max(2, int(round(0.15 * geo["n_sm"])))
        self.stream = torch.cuda.current_stream()

    # the schedules of the ablation (Section 5.6): (mode, c, K, steal), plan kinds, elastic switch
    def schedules(self):
        pk = self.pk
        return {
            "auto": ((pk.SCHED_AUTO, 0, 1, 0), 7, -1),                    # the model over its default plan kinds
            "auto_split": ((pk.SCHED_AUTO, 0, 1, 0), 1, -1),              # the paper's plan kind only
            "fixed": ((pk.SCHED_FIXED, self.fixed_c, 1, 0), 7, 0),        # static 15 % split, nothing else
            "fixed_elastic": ((pk.SCHED_FIXED, self.fixed_c, 1, 0), 7, 1),  # ... plus elastic stealing and the first dispatch wave
            "serial": ((pk.SCHED_SERIAL, 0, 1, 0), 7, -1),                # phases separated by grid barriers
        }

    def set(self, name):
        sched, kinds, elastic = self.schedules()[name]
        self.moe.set_schedule(*sched)
        self.moe.set_model_options(kinds, elastic)

    def step_dev(self):
        for l in range(self.L):
            self.moe.forward(self.x, self.logits[l], self.out)

    def step_host(self):
        # the call a user makes for a stream of batches from host memory: inputs and outputs cross
        # PCIe every layer call; the copies overlap the neighbouring calls' kernels
        for l in range(self.L):
            self.moe.forward_host_pipelined(self.x_h, self.logits_h[l], self.out_h[l % 2])

    def timed(self, fn, steps, warmup, world=1, host_path=False):
        torch = self.torch
        for _ in range(warmup):
            fn()
        if host_path:
            self.moe.host_wait()
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()
        if host_path:
            # the last output copy runs on the library's copy stream: wall clock around the whole
            # region, bracketed by full synchronisation (device events on one stream would miss it)
            t0 = time.perf_counter()
            for _ in range(steps):
                fn()
            self.moe.host_wait()
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            if world > 1:
                torch.distributed.barrier()
            return dt
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(self.stream)
        for _ in range(steps):
            fn()
        ev1.record(self.stream)
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        return ev0.elapsed_time(ev1) * 1e-3

    def sustained(self, step_s, seconds=2.0, local=0):
        """Layer time of a back-to-back run of at least `seconds` (after 0.3 s of the same load), with
        the clocks sampled during it: the figure to hold against the sustained peak."""
        n_warm = max(1, int(0.3 / step_s))
        n = max(2, int(np.ceil(seconds / step_s)))
        for _ in range(n_warm):
            self.step_dev()
        sampler = ClockSampler(local)
        sampler.start()
        sec = self.timed(self.step_dev, n, 0)
        clocks = sampler.stop()
        return sec / n / self.L, sec, clocks

    def ablation(self, step_s, rounds=4):
        """The schedules take turns.  The part runs under its power cap and the clock follows the last
        ~50 ms of load, so a schedule measured right after a slow (cool) one looks faster: each
        measurement is preceded by ~50 ms of its own schedule, and the order changes from round to
        round so that every schedule follows a different predecessor each time (round r walks the list
        with stride r + 1: with five schedules the four strides give four different predecessors)."""
        names = list(self.schedules())
        n = len(names)
        n_abl = max(2, min(5, int(0.25 / step_s) + 1))
        warm = max(1, min(20, int(0.05 / step_s) + 1))
        tot = {nm: 0.0 for nm in names}
        for r in range(rounds):
            stride = r % (n - 1) + 1
            for j in range(n):
                name = names[(2 * r + j * stride) % n]
                self.set(name)
                tot[name] += self.timed(self.step_dev, n_abl, warm)
        res = {nm + "_us_per_layer": s / (n_abl * rounds) / self.L * 1e6 for nm, s in tot.items()}
        res["fixed_c"] = self.fixed_c
        self.set("auto")
        self.moe.check()
        return res

    def close(self):
        self.moe.close()


def measure_side_config(name, args, peaks, weights_cache):
    """One entry of `per_config`: burst-window and sustained layer times with their roofline
    fractions, the plan, the scheduler ablation."""
    import torch
    import workloads as wl
    cfg = wl.CONFIGS[name]
    key = (cfg.cfg_id, cfg.H, cfg.I, cfg.E, cfg.S)
    lay = Layer(cfg, args, weights_cache.get(key))
    weights_cache.clear()
    weights_cache[key] = lay.weights
    lay.set("auto")
    n_burst = 10
    sec = lay.timed(lay.step_dev, n_burst, 3)
    if sec / n_burst < 5e-4:
        # a layer of tens of microseconds: ten launches are over before the host has queued them, and the
        # figure would be the host's launch rate; 200 launches (still a burst window) keep the queue full
        n_burst = 200
        sec = lay.timed(lay.step_dev, n_burst, 20)
    lay.moe.check()
    step_s = sec / n_burst
    plan = lay.moe.plan()
    work = layer_work(cfg)
    burst = roofline_of(work, step_s / lay.L, peaks, "burst")
    sus_layer_s, sus_sec, clocks = lay.sustained(step_s, seconds=args.sustain_seconds, local=args.local)
    sus = roofline_of(work, sus_layer_s, peaks, "sustained")
    entry = {"workload": cfg.name, "T": cfg.T, "layer_us": step_s / lay.L * 1e6, "frac": burst["frac"],
             "bound": burst["bound"], "layer_roofline_us": burst["layer_roofline_us"],
             "layer_us_sustained": sus_layer_s * 1e6, "frac_sustained": sus["frac"], "bound_sustained": sus["bound"],
             "sustained_run_s": sus_sec, "sm_mhz_sustained": clocks.get("sm_mhz"), "reasons": clocks.get("reasons"),
             "plan": plan, "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(cfg.name),
             "ablation": lay.ablation(step_s) if not args.no_ablation else {}}
    lay.close()
    del lay
    torch.cuda.empty_cache()
    return entry


def run_ours(args):
    import torch
    import workloads as wl
    import paper_2609_21483_b200 as pk

    rank, world, local = dist_env()
    if args.gpus > 1 and world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus}: started as one of {world} ranks")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    args.local = local
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pk.load()
    wl.build()

    cfg = wl.CONFIGS[args.config]
    lay = Layer(cfg, args)
    L = lay.L
    lay.set(args.sched)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.05)
    sec = lay.timed(lay.step_dev, args.steps, args.warmup, world)
    lay.moe.check()
    plan = lay.moe.plan() if rank == 0 else None
    sec_max = aggregate_max(sec, world, True)
    clocks = sampler.stop() if rank == 0 else None
    step_s = sec_max / args.steps
    if rank == 0 and (clocks.get("samples") or 0) < 5:
        # the timed region was too short for nvidia-smi's sampling period: repeat the same steps
        # (untimed) for about half a second with the sampler running, and say so
        probe = ClockSampler(local)
        probe.start()
        t_end = time.perf_counter() + 0.6
        while time.perf_counter() < t_end:
            lay.step_dev()
            torch.cuda.synchronize()
        clocks = probe.stop()
        clocks["note"] = "timed region shorter than the sampling period; sampled over an untimed 0.6 s repeat of the same steps"
    e2e_steps = max(1, min(args.steps, 10))
    sec_e2e = aggregate_max(lay.timed(lay.step_host, e2e_steps, 3, world, host_path=True), world, True)
    lay.moe.check()

    peaks = load_peaks()
    work = layer_work(cfg)
    ep_desc = None
    if args.ep > 1:
        # the rank computes only its own pairs: scale the algorithmic work by its share of the pairs
        ep_desc = lay.moe.ep_descriptors()
        share = (ep_desc["x_local"] + ep_desc["x_in"]) / float(cfg.P)
        work = {k: v * share for k, v in work.items()}
    layer_s = step_s / L
    # which peak the timed region is held against: the burst figure for a region well under half a second
    # (it starts from idle clocks), the sustained one for a back-to-back run under the power cap
    window = "sustained" if sec_max >= 0.5 else "burst"
    roof = roofline_of(work, layer_s, peaks, window)
    roof["traffic"] = NCU_DRAM_BYTES_PER_LAUNCH.get(cfg.name)
    roof["peak_source"] = f"{peaks['source']} ({window} window: timed region {sec_max:.2f} s)"
    roof["flops_per_launch"], roof["bytes_per_launch"] = work["flops"], work["bytes"]
    # the other window, from its own run: never one window's time over the other window's peak
    sustained = burst = None
    if rank == 0 and world == 1 and not args.no_ablation:
        if window == "burst":
            s_layer, s_sec, s_clk = lay.sustained(step_s, seconds=args.sustain_seconds, local=local)
            sustained = dict(roofline_of(work, s_layer, peaks, "sustained"), layer_us=s_layer * 1e6, run_s=s_sec,
                             sm_mhz=s_clk.get("sm_mhz"))
        else:
            torch.cuda.synchronize()
            time.sleep(1.0)                                   # let the clocks recover
            n_b = max(1, int(0.3 / step_s))
            b_sec = lay.timed(lay.step_dev, n_b, 0)
            burst = dict(roofline_of(work, b_sec / n_b / L, peaks, "burst"), layer_us=b_sec / n_b / L * 1e6, run_s=b_sec)
    roof["other_window"] = sustained or burst

    ablation = lay.ablation(step_s) if (rank == 0 and not args.no_ablation and world == 1) else {}

    cpu_base = None
    if rank == 0 and not args.no_cpu_baseline and args.ep <= 1:
        import oracle
        oracle.build()
        lg0 = lay.logits_h[0].numpy()
        probe = wl.stratified_token_sample(cfg.T, 8, seed=99)
        inp = wl.LayerInputs(cfg, wl.make_x(cfg), lg0, *host_weights_for(cfg, wl, oracle, lg0, probe))
        n = args.ref_tokens if args.ref_tokens > 0 else cpu_sample_size(oracle, wl, inp, cfg, args.cpu_seconds)
        toks = wl.stratified_token_sample(cfg.T, n, seed=cfg.cfg_id)
        inp.gate_up, inp.down = host_weights_for(cfg, wl, oracle, lg0, toks)
        t0 = time.perf_counter()
        oracle.routing(inp.logits, cfg.k, cfg.S)
        oracle.moe_tokens(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, toks, cfg.S)
        dt = time.perf_counter() - t0
        cpu_base = {"value": len(toks) / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                    "sample": f"{len(toks)} stratified tokens of T={cfg.T}, layer 0 of {L} (full-T routing + per-token "
                              f"FFN/combine) in {dt:.1f} s"}
        del inp

    lay.close()
    weights_cache = {}
    del lay
    torch.cuda.empty_cache()
    per_config = []
    if rank == 0 and world == 1 and args.per_config and args.ep <= 1:
        for name in PER_CONFIG:
            if name != cfg.name:
                per_config.append(measure_side_config(name, args, peaks, weights_cache))

    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return

    xb = cfg.T * cfg.H * 2
    line = {
        "metric": METRIC, "value": whole_job_throughput(cfg.T * L, args.steps, world, sec_max), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "I": cfg.I, "E": cfg.E, "top_k": cfg.k,
                   "shared": cfg.S, "layers": L, "sched": args.sched, "parallelism": f"replicas x{world}",
                   "l2_policy": "inputs larger than L2 (weights %.2f GB streamed every layer)" % (work["weights_bytes"] / 1e9)},
        "layer_us": layer_s * 1e6,
        "layer_roofline_us": roof["layer_roofline_us"],
        "roofline": roof,
        "e2e": {"value": whole_job_throughput(cfg.T * L, e2e_steps, world, sec_e2e), "unit": UNIT,
                "h2d_bytes_per_step": (xb + cfg.T * cfg.E * 4) * L, "d2h_bytes_per_step": xb * L},
        "gpu_launches": args.steps * L,
        "clocks": clocks,
        "plan": plan,
        "expert_parallel": ({"ep_size": args.ep, "ep_rank": args.ep_rank, **ep_desc,
                             "note": "work and roofline scaled by this rank's share of the token-expert pairs (last layer's routing)"}
                            if ep_desc else None),
        "ablation": ablation,
        "per_config": per_config,
        "cpu_baseline": cpu_base,
        "paper_context": "paper reports 2.89x geomean MoE-layer speedup over 5 systems on 4xH100 (EP=4); no 1-GPU or B200 number",
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default=DEFAULT_CONFIG)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sched", default="auto", choices=["auto", "auto_split", "fixed", "fixed_elastic", "serial"])
    ap.add_argument("--ref-tokens", type=int, default=0,
                    help="tokens in the CPU oracle's timed sample (0 = sized for --cpu-seconds of work)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--sustain-seconds", type=float, default=2.0,
                    help="length of the back-to-back run behind every sustained-window figure")
    ap.add_argument("--ep", type=int, default=1, help="model one rank of an expert-parallel group of this size")
    ap.add_argument("--ep-rank", type=int, default=0)
    ap.add_argument("--sms", type=int, default=0, help="SMs the kernel may occupy (0 = all; even)")
    ap.add_argument("--no-ablation", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--per-config", dest="per_config", action="store_true", default=None,
                    help="also measure the other configurations of record (default with the default workload)")
    ap.add_argument("--no-per-config", dest="per_config", action="store_false")
    ap.add_argument("--launcher-selftest", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.per_config is None:
        args.per_config = args.config == DEFAULT_CONFIG
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "ours" or args.launcher_selftest):
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    if args.launcher_selftest:
        launcher_selftest(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
