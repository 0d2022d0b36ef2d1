"""Shared helper of the GPU parity tests: run the CUDA layer through its C ABI on a seeded
workload, evaluate the CPU oracle on the same arrays, compare.

Bars: routing indices, counts, offsets and the permutation bit-exact; gates to 1e-5 relative;
outputs |gpu - ref| <= 2e-2 + 2e-2*|ref| per element and relative L2 <= 5e-3 against the fp32
oracle.  Large layers are checked on a token sample (each output row depends only on its own token, its
routing and the weights, so a sampled row is checked exactly).  The sample is built from the
ORACLE's routing so that it reaches every part of the expert-major layout: the first and the last
row of every non-empty expert, a row in every 128-row m-block, and token strata.
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


def coverage_token_sample(ref, cfg: wl.MoEConfig, n_strata: int = 16, budget=None, block_m: int = 128, seed: int = 0):
    """Tokens whose output rows, together, touch every part of the expert-major buffers.

    ref = the oracle's routing of the layer.  In this order of priority: the tokens of the first
    and the last row of every non-empty expert, experts with the fewest rows first (a segment's
    last rows sit in its ragged, unpaired m-block); the token of one hashed row inside every
    m-block (block_m consecutive rows of one expert's segment); n_strata tokens spread over the
    batch (first, last, one per stratum).  budget caps the number of tokens (None = all of them;
    the strata are always kept).  Returns (sorted token array, coverage dict)."""
    E, S = cfg.E, cfg.S
    counts, offsets, token_of = ref.counts, ref.offsets, ref.token_of      # (routing_ep: other ranks' counts are 0)
    strata = [int(t) for t in wl.stratified_token_sample(cfg.T, n_strata, seed=seed)]
    ordered = []
    routed = [e for e in np.argsort(counts[:E], kind="stable") if counts[e] > 0]
    for e in routed:
        ordered.append(int(token_of[offsets[e]]))
        ordered.append(int(token_of[offsets[e + 1] - 1]))
    h = (seed * 2654435761 + 12345) & 0xFFFFFFFFFFFFFFFF
    for e in list(routed) + list(range(E, E + S)):
        for r0 in range(int(offsets[e]), int(offsets[e + 1]), block_m):
            n = min(block_m, int(offsets[e + 1]) - r0)
            h = (h * 6364136223846793005 + 1442695040888963407) & 0xFFFFFFFFFFFFFFFF      # 64-bit LCG
            ordered.append(int(token_of[r0 + (h >> 33) % n]))
    picks, seen = [], set()
    for t in strata + ordered:
        if t not in seen:
            seen.add(t)
            picks.append(t)
    if budget is not None:
        picks = picks[:max(budget, len(set(strata)))]
    toks = np.array(sorted(picks), dtype=np.int32)
    # what the sample reaches: every (token, slot) row of a sampled token is value-checked
    rows = ref.row_of[toks].ravel()
    rows = rows[rows >= 0]          # an expert-parallel rank has rows only for its own experts
    exp_of_row = np.searchsorted(offsets, rows, side="right") - 1
    mb_id = set()
    for r, e in zip(rows.tolist(), exp_of_row.tolist()):
        mb_id.add((e, (r - int(offsets[e])) // block_m))
    n_mb = int(sum((int(c) + block_m - 1) // block_m for c in counts))
    tiny = [e for e in range(E) if 0 < counts[e] <= 32]
    cov = {"tokens": int(len(toks)), "experts": len(set(exp_of_row.tolist())),
           "experts_nonempty": int((counts > 0).sum()), "m_blocks": len(mb_id), "m_blocks_total": n_mb,
           "tiny_experts": len(set(exp_of_row.tolist()) & set(tiny)), "tiny_experts_total": len(tiny)}
    return toks, cov


def oracle_rows(inp: wl.LayerInputs, tokens=None):
    """fp32 oracle output rows: the whole layer if tokens is None, else the listed tokens."""
    cfg = inp.cfg
    if tokens is None:
        return oracle.moe_layer(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, cfg.S).out
    return oracle.moe_tokens(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k, tokens, cfg.S)


def run_case(cfg: wl.MoEConfig, sched=None, n_sample=None, layer=0, inp=None, dev_tensors=None, moe=None,
             max_tokens=None, budget=None, require_full_coverage=False):
    """sched: None (AUTO) or (mode, c, K, steal).  n_sample: None = the whole output is compared,
    else the number of token strata of a coverage sample (see coverage_token_sample; budget caps
    it).  Returns (moe, out tensor, relative L2)."""
    inp = inp if inp is not None else wl.make_inputs(cfg, layer)
    x, lg, gu, dn = dev_tensors if dev_tensors is not None else to_dev(inp)
    if moe is None:
        moe = WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=max_tokens or cfg.T)
    if sched is not None:
        moe.set_schedule(*sched)
    out = moe.forward(x, lg)
    moe.check()
    ref = check_routing(moe, inp)
    if n_sample is None:
        l2 = check_values(bf16_to_np(out), oracle_rows(inp), cfg.name)
    else:
        toks, cov = coverage_token_sample(ref, cfg, n_sample, budget, moe.geometry()["block_m"], seed=cfg.cfg_id)
        print(f"[coverage] {cfg.name} layer {layer}: {cov}")
        if require_full_coverage:
            assert cov["experts"] == cov["experts_nonempty"] and cov["m_blocks"] == cov["m_blocks_total"], cov
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


def oracle_rows_streamed(cfg: wl.MoEConfig, x_h, lg_h, toks, max_experts_per_group: int = 64):
    """Oracle rows of the listed tokens for a layer whose weights are too large to hold on the host
    in one piece: the tokens are taken in groups that need at most max_experts_per_group experts;
    each group gets zero-initialised weight arrays (untouched pages cost nothing) in which only
    its experts are filled in."""
    idx, _ = oracle.route(np.ascontiguousarray(lg_h[toks]), cfg.k)
    EE = cfg.E + cfg.S
    shared = list(range(cfg.E, EE))
    out = np.empty((len(toks), cfg.H), np.float32)
    i = 0
    while i < len(toks):
        need, j = set(shared), i
        while j < len(toks) and len(need | set(idx[j].tolist())) <= max(max_experts_per_group, cfg.k + cfg.S):
            need |= set(idx[j].tolist())
            j += 1
        gu_h = np.zeros((EE, 2 * cfg.I, cfg.H), np.uint16)
        dn_h = np.zeros((EE, cfg.H, cfg.I), np.uint16)
        for e in sorted(need):
            gu_h[e], dn_h[e] = wl.expert_weights(cfg, e)
        out[i:j] = oracle.moe_tokens(x_h, lg_h, gu_h, dn_h, cfg.k, toks[i:j], cfg.S)
        del gu_h, dn_h
        i = j
    return out


def run_case_streamed(cfg: wl.MoEConfig, n_sample: int, sched=None, budget=None, max_experts_per_group: int = 64):
    """Like run_case for shapes whose weights do not fit comfortably on the host (see
    oracle_rows_streamed)."""
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
    rt = check_routing(moe, inp)
    toks, cov = coverage_token_sample(rt, cfg, n_sample, budget, moe.geometry()["block_m"], seed=cfg.cfg_id)
    print(f"[coverage] {cfg.name}: {cov}")
    ref = oracle_rows_streamed(cfg, x_h, lg_h, toks, max_experts_per_group)
    l2 = check_values(bf16_to_np(out[torch.from_numpy(toks).long().to(out.device)]), ref, cfg.name)
    return moe, out, l2
