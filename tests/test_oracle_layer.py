"""Pins for the oracle's value stages: dispatch, gemm0 + silu_mul, gemm1, combine.

Checked against library fp64 matmuls (torch), closed forms with identity-like experts,
special cases whose answer is known by construction, and a per-token brute force that
uses no permutation at all.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl


def _rand_layer(T, H, I, E, S, seed):
    EE = E + S
    x = wl.normal_bf16(T * H, seed).reshape(T, H)
    lg = wl.normal_f32(T * E, seed + 1).reshape(T, E)
    gu = wl.normal_bf16(EE * 2 * I * H, seed + 2, 0.0, 0.05).reshape(EE, 2 * I, H)
    dn = wl.normal_bf16(EE * H * I, seed + 3, 0.0, 0.05).reshape(EE, H, I)
    return x, lg, gu, dn


def _torch_ffn(xf, gu_e, dn_e):
    """Textbook SwiGLU MLP in fp64 with library matmuls: rows [0,I) of gate_up are the gate."""
    I = dn_e.shape[1]
    a = xf @ gu_e.T                       # [n, 2I]
    h = torch.nn.functional.silu(a[:, :I]) * a[:, I:]
    return h, h @ dn_e.T


def _t64(bits):
    return torch.from_numpy(wl.bf16_bits_to_f32(bits)).double()


def test_dense_swiglu_matches_library_matmul():
    """E=1, k=1: gate is 1 and the layer is a dense SwiGLU MLP."""
    T, H, I = 9, 96, 160
    x, lg, gu, dn = _rand_layer(T, H, I, 1, 0, seed=21)
    res = oracle.moe_layer(x, lg, gu, dn, k=1, keep_intermediates=True)
    h_ref, y_ref = _torch_ffn(_t64(x), _t64(gu[0]), _t64(dn[0]))
    assert (res.routing.gates == 1.0).all()
    np.testing.assert_allclose(res.h, h_ref.numpy(), rtol=2e-5, atol=2e-6)
    np.testing.assert_allclose(res.out, y_ref.numpy(), rtol=2e-5, atol=2e-6)
    # single-row entry point agrees with the same library computation
    h1, y1 = oracle.expert_ffn(x[4], gu[0], dn[0])
    np.testing.assert_allclose(h1, h_ref[4].numpy(), rtol=2e-5, atol=2e-6)
    np.testing.assert_allclose(y1, y_ref[4].numpy(), rtol=2e-5, atol=2e-6)


def test_gate_half_is_the_one_that_gets_silu():
    """Swapping the halves of gate_up must change the result (silu(a)*b != silu(b)*a)."""
    H, I = 32, 48
    x, _, gu, dn = _rand_layer(1, H, I, 1, 0, seed=4)
    _, y = oracle.expert_ffn(x[0], gu[0], dn[0])
    swapped = np.concatenate([gu[0][I:], gu[0][:I]], axis=0)
    _, y2 = oracle.expert_ffn(x[0], swapped, dn[0])
    assert np.abs(y - y2).max() > 1e-3
    # and the un-swapped one is the library's silu(gate)*up
    _, y_ref = _torch_ffn(_t64(x[:1]), _t64(gu[0]), _t64(dn[0]))
    np.testing.assert_allclose(y, y_ref[0].numpy(), rtol=2e-5, atol=2e-6)


def test_fp32_and_fp64_accumulation_agree():
    T, H, I, E, k = 24, 256, 384, 4, 2
    x, lg, gu, dn = _rand_layer(T, H, I, E, 0, seed=8)
    a = oracle.moe_layer(x, lg, gu, dn, k).out
    b = oracle.moe_layer(x, lg, gu, dn, k, acc_double=True).out
    rel = np.linalg.norm(a - b) / np.linalg.norm(b)
    assert rel < 2e-6


@pytest.mark.parametrize("T,H,I,E,k,S", [(17, 64, 96, 4, 2, 0), (40, 128, 64, 16, 4, 2), (5, 32, 32, 3, 3, 1)])
def test_layer_matches_library_reference(T, H, I, E, k, S):
    """Whole layer vs a torch fp64 computation that never permutes: loop tokens, loop experts."""
    x, lg, gu, dn = _rand_layer(T, H, I, E, S, seed=31 + T)
    res = oracle.moe_layer(x, lg, gu, dn, k, S, keep_intermediates=True)
    r = res.routing
    xf = _t64(x)
    ref = torch.zeros(T, H, dtype=torch.float64)
    for t in range(T):
        for j in range(k):
            e = int(r.idx[t, j])
            _, y = _torch_ffn(xf[t:t + 1], _t64(gu[e]), _t64(dn[e]))
            ref[t] += float(r.gates[t, j]) * y[0]
        for s in range(S):
            _, y = _torch_ffn(xf[t:t + 1], _t64(gu[E + s]), _t64(dn[E + s]))
            ref[t] += y[0]
    np.testing.assert_allclose(res.out, ref.numpy(), rtol=3e-5, atol=3e-6)
    # dispatch is a bit copy: Xe[row] = x[token_of[row]]
    np.testing.assert_array_equal(res.xe, wl.bf16_bits_to_f32(x)[r.token_of])
    # intermediate y rows belong to the expert of their segment
    for e in range(E + S):
        rows = np.arange(r.offsets[e], r.offsets[e + 1])
        if len(rows):
            _, y = _torch_ffn(xf[r.token_of[rows]], _t64(gu[e]), _t64(dn[e]))
            np.testing.assert_allclose(res.y[rows], y.numpy(), rtol=3e-5, atol=3e-6)


def test_identity_like_experts_closed_form():
    """H = I, x[:,0] = 1, gate projection = beta * (column 0), up = identity,
    down[e] = d_e * identity  =>  out[t] = x[t] * silu(beta) * sum_j g[t,j] * d_{e_j}."""
    T, H, E, k = 50, 64, 8, 3
    I = H
    x = wl.normal_bf16(T * H, 1).reshape(T, H).copy()
    x[:, 0] = wl.f32_to_bf16_bits(np.array([1.0], np.float32))[0]
    lg = wl.normal_f32(T * E, 2).reshape(T, E)
    beta = 1.0
    one = wl.f32_to_bf16_bits(np.array([1.0], np.float32))[0]
    gu = np.zeros((E, 2 * I, H), np.uint16)
    gu[:, :I, 0] = wl.f32_to_bf16_bits(np.array([beta], np.float32))[0]
    gu[:, I + np.arange(I), np.arange(H)] = one
    d = wl.f32_to_bf16_bits(np.linspace(0.5, 2.25, E).astype(np.float32))     # bf16-exact steps of 0.25
    dn = np.zeros((E, H, I), np.uint16)
    for e in range(E):
        dn[e, np.arange(H), np.arange(I)] = d[e]
    res = oracle.moe_layer(x, lg, gu, dn, k)
    s = beta / (1.0 + np.exp(-beta))
    dv = wl.bf16_bits_to_f32(d).astype(np.float64)
    w = (res.routing.gates.astype(np.float64) * dv[res.routing.idx]).sum(axis=1)
    ref = wl.bf16_bits_to_f32(x).astype(np.float64) * s * w[:, None]
    np.testing.assert_allclose(res.out, ref, rtol=3e-6, atol=1e-7)


def test_identical_experts_make_routing_irrelevant():
    """All experts equal => out = FFN(x) for every token (needs sum of gates = 1 and a
    correct permutation, whatever the routing is)."""
    T, H, I, E, k = 30, 64, 96, 6, 3
    x, lg, gu, dn = _rand_layer(T, H, I, 1, 0, seed=13)
    gu = np.repeat(gu, E, axis=0)
    dn = np.repeat(dn, E, axis=0)
    lg = wl.normal_f32(T * E, 99).reshape(T, E)
    out = oracle.moe_layer(x, lg, gu, dn, k).out
    _, y = _torch_ffn(_t64(x), _t64(gu[0]), _t64(dn[0]))
    np.testing.assert_allclose(out, y.numpy(), rtol=3e-5, atol=3e-6)


def test_only_one_expert_nonzero_marks_its_tokens():
    T, H, I, E, k = 64, 32, 32, 8, 2
    x, lg, gu, dn = _rand_layer(T, H, I, E, 0, seed=55)
    keep = 5
    dn2 = np.zeros_like(dn)
    dn2[keep] = dn[keep]
    res = oracle.moe_layer(x, lg, gu, dn2, k)
    routed = (res.routing.idx == keep).any(axis=1)
    nz = np.abs(res.out).max(axis=1) > 0
    np.testing.assert_array_equal(nz, routed)
    assert routed.any() and (~routed).any()


@pytest.mark.parametrize("S", [0, 2])
def test_brute_force_per_token_equals_pipeline_bit_for_bit(S):
    T, H, I, E, k = 37, 64, 128, 8, 2
    x, lg, gu, dn = _rand_layer(T, H, I, E, S, seed=71)
    full = oracle.moe_layer(x, lg, gu, dn, k, S).out
    toks = np.arange(T, dtype=np.int32)[::-1].copy()      # any order, any subset
    some = oracle.moe_tokens(x, lg, gu, dn, k, toks, S)
    np.testing.assert_array_equal(some, full[toks])


def test_tiny_config_full_layer_runs_and_is_sane():
    """Config 1 (T=256,H=512,I=1024,E=8,k=2) in full: finite, O(1) magnitudes, and a
    sampled token recomputed with library matmuls."""
    cfg = wl.CONFIGS["c1_tiny"]
    inp = wl.make_inputs(cfg)
    res = oracle.moe_layer(inp.x, inp.logits, inp.gate_up, inp.down, cfg.k)
    assert np.isfinite(res.out).all()
    assert 1e-3 < np.abs(res.out).mean() < 10
    t = 123
    ref = torch.zeros(cfg.H, dtype=torch.float64)
    for j in range(cfg.k):
        e = int(res.routing.idx[t, j])
        _, y = _torch_ffn(_t64(inp.x[t:t + 1]), _t64(inp.gate_up[e]), _t64(inp.down[e]))
        ref += float(res.routing.gates[t, j]) * y[0]
    np.testing.assert_allclose(res.out[t], ref.numpy(), rtol=5e-5, atol=1e-6)
