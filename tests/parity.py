"""Shared helper of the GPU parity tests: run the CUDA layer through its C ABI on a seeded
workload, evaluate the CPU oracle on the same arrays, compare.

Bars: routing indices, counts, offsets and the permutation bit-exact; gates to 1e-5 relative;
outputs |gpu - ref| <= 2e-2 + 2e-2*|ref| per element and relative L2 <= 5e-3 against the fp32
oracle.  Large layers are checked on a stratified token sample (each output row depends only on
its own token, its routing and the weights, so a sampled row is checked exactly).
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import workloads as wl
from paper_2609_21483_b200 import WeaveMoE

ABS_TOL, REL_TOL, L2_TOL, GATE_RTOL = 2e-2, 2e-2, 5e-3, 1e-5


def to_dev(inp: wl.LayerInputs, dev="cuda"):
    x = torch.from_numpy(inp.x.view(np.int16)).view(torch.bfloat16).to(dev)
    lg = torch.from_numpy(inp.logits).to(dev)
    gu = torch.from_numpy(inp.gate_up.view(np.int16)).view(torch.bfloat16).to(dev)
    dn = torch.from_numpy(inp.down.view(np.int16)).view(torch.bfloat16).to(dev)
    return x, lg, gu, dn


def bf16_to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def check_routing(moe: WeaveMoE, inp: wl.LayerInputs):
    cfg = inp.cfg
    ref = oracle.routing(inp.logits, cfg.k, cfg.S)
    r = {k: v.cpu().numpy() for k, v in moe.routing(cfg.T).items()}
    np.testing.assert_array_equal(r["topk_idx"], ref.idx)
    np.testing.assert_allclose(r["gates"], ref.gates, rtol=GATE_RTOL, atol=1e-9)
    np.testing.assert_array_equal(r["counts"], ref.counts)
    np.testing.assert_array_equal(r["offsets"], ref.offsets)
    np.testing.assert_array_equal(r["row_of"], ref.row_of[:, :cfg.k])
    np.testing.assert_array_equal(r["token_of"], ref.token_of)
    return ref


def check_values(out_gpu: np.ndarray, ref: np.ndarray, what=""):
    assert np.isfinite(out_gpu).all(), f"{what}: non-finite output"
    err = np.abs(out_gpu - ref)
    bound = ABS_TOL + REL_TOL * np.abs(ref)
    worst = float((err - bound).max())
    l2 = float(np.linalg.norm(out_gpu - ref) / max(np.linalg.norm(ref), 1e-30))
    assert worst <= 0, f"{what}: element bound exceeded by {worst:.3e} (max err {err.max():.3e})"
    assert l2 <= L2_TOL, f"{what}: relative L2 {l2:.3e} > {L2_TOL}"
    return l2


def oracle_rows(inp: wl.LayerInputs, tokens=None):
    """fp32 oracle output rows: the whole layer if tokens is None, else the listed tokens."""
    cfg = inp.cfg
    if tokens is None:
        return oracle.moe_layer(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, cfg.S).out
    return oracle.moe_tokens(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, tokens, cfg.S)


def run_case(cfg: wl.MoEConfig, sched=None, n_sample=None, layer=0, inp=None, dev_tensors=None, moe=None,
             max_tokens=None):
    """sched: None (AUTO) or (mode, c, K, steal).  Returns (moe, out tensor, relative L2)."""
    inp = inp if inp is not None else wl.make_inputs(cfg, layer)
    x, lg, gu, dn = dev_tensors if dev_tensors is not None else to_dev(inp)
    if moe is None:
        moe = WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=max_tokens or cfg.T)
    if sched is not None:
        moe.set_schedule(*sched)
    out = moe.forward(x, lg)
    moe.check()
    check_routing(moe, inp)
    if n_sample is None:
        l2 = check_values(bf16_to_np(out), oracle_rows(inp), cfg.name)
    else:
        toks = wl.stratified_token_sample(cfg.T, n_sample, seed=cfg.cfg_id)
        l2 = check_values(bf16_to_np(out[torch.from_numpy(toks).long().to(out.device)]),
                          oracle_rows(inp, toks), cfg.name)
    return moe, out, l2


def stream_weights_to_dev(cfg: wl.MoEConfig, dev="cuda"):
    """Device weights of a layer too large to build on the host in one piece: generated and copied
    expert by expert (the generator is counter-based, so the values equal make_weights())."""
    EE = cfg.E + cfg.S
    gu = torch.empty((EE, 2 * cfg.I, cfg.H), dtype=torch.bfloat16, device=dev)
    dn = torch.empty((EE, cfg.H, cfg.I), dtype=torch.bfloat16, device=dev)
    for e in range(EE):
        g, d = wl.expert_weights(cfg, e)
        gu[e].copy_(torch.from_numpy(g.view(np.int16)).view(torch.bfloat16))
        dn[e].copy_(torch.from_numpy(d.view(np.int16)).view(torch.bfloat16))
    return gu, dn


def run_case_streamed(cfg: wl.MoEConfig, n_sample: int, sched=None):
    """Like run_case for shapes whose weights do not fit comfortably on the host: the oracle gets
    zero-initialised weight arrays (untouched pages cost nothing) in which only the experts of the
    sampled tokens are filled in."""
    x_h, lg_h = wl.make_x(cfg), wl.make_logits(cfg)
    x = torch.from_numpy(x_h.view(np.int16)).view(torch.bfloat16).cuda()
    lg = torch.from_numpy(lg_h).cuda()
    gu, dn = stream_weights_to_dev(cfg)
    moe = WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    if sched is not None:
        moe.set_schedule(*sched)
    out = moe.forward(x, lg)
    moe.check()
    inp = wl.LayerInputs(cfg, x_h, lg_h, None, None)
    check_routing(moe, inp)
    toks = wl.stratified_token_sample(cfg.T, n_sample, seed=cfg.cfg_id)
    idx, _ = oracle.route(lg_h[toks], cfg.k)
    need = sorted(set(idx.ravel().tolist()) | set(range(cfg.E, cfg.E + cfg.S)))
    EE = cfg.E + cfg.S
    gu_h = np.zeros((EE, 2 * cfg.I, cfg.H), np.uint16)
    dn_h = np.zeros((EE, cfg.H, cfg.I), np.uint16)
    for e in need:
        gu_h[e], dn_h[e] = wl.expert_weights(cfg, e)
    ref = oracle.moe_tokens(x_h, lg_h, gu_h, dn_h, cfg.k, toks, cfg.S)
    l2 = check_values(bf16_to_np(out[torch.from_numpy(toks).long().to(out.device)]), ref, cfg.name)
    return moe, out, l2
