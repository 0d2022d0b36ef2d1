"""The synthetic-input generator: reproducible, order-independent, correctly distributed,
and shaped like the paper's Table 1 rows where a config claims one."""
import os

import numpy as np

import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_model_shapes.txt")


def _table1():
    rows = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, E, k, H, I = line.split()
        rows[name] = tuple(int(v) for v in (E, k, H, I))
    return rows


def test_configs_that_claim_a_table1_shape_have_it():
    t1 = _table1()
    for cfg_name, row in [("c3_qwen3_30b", "Qwen3-30B"), ("c4_dsv2lite_T64", "DSv2-Lite")]:
        c = wl.CONFIGS[cfg_name]
        assert (c.E, c.k, c.H, c.I) == t1[row]
    # every Table 1 shape is tileable by this build's 128-wide tiles
    for E, k, H, I in t1.values():
        assert H % 128 == 0 and I % 128 == 0 and k <= E


def test_streams_are_reproducible_and_counter_based():
    a = wl.normal_f32(1001, seed=42)
    b = wl.normal_f32(1001, seed=42)
    np.testing.assert_array_equal(a, b)
    # a prefix of a longer stream equals the shorter stream (element i depends on (seed,i) only)
    np.testing.assert_array_equal(wl.normal_f32(500, seed=42), a[:500])
    assert not np.array_equal(a, wl.normal_f32(1001, seed=43))
    # bf16 stream = RNE rounding of the fp32 stream
    np.testing.assert_array_equal(wl.normal_bf16(1001, seed=42), wl.f32_to_bf16_bits(a))


def test_distribution_moments():
    z = wl.normal_f32(1 << 20, seed=7, mean=0.0, std=1.0).astype(np.float64)
    assert abs(z.mean()) < 5e-3 and abs(z.std() - 1.0) < 5e-3
    assert abs((z ** 3).mean()) < 2e-2 and abs((z ** 4).mean() - 3.0) < 5e-2
    w = wl.bf16_bits_to_f32(wl.normal_bf16(1 << 18, seed=8, mean=0.0, std=0.02)).astype(np.float64)
    assert abs(w.std() - 0.02) < 3e-4


def test_config1_matches_the_stated_recipe():
    cfg = wl.CONFIGS["c1_tiny"]
    inp = wl.make_inputs(cfg)
    assert inp.x.shape == (256, 512) and inp.logits.shape == (256, 8)
    assert inp.gate_up.shape == (8, 2048, 512) and inp.down.shape == (8, 512, 1024)
    assert abs(wl.bf16_bits_to_f32(inp.gate_up).std() - 0.02) < 1e-3
    assert abs(wl.bf16_bits_to_f32(inp.x).std() - 1.0) < 2e-2


def test_skew_is_per_layer_and_within_range():
    cfg = wl.CONFIGS["c5_qwen3_235b"]
    s = [wl.layer_skew(cfg, l) for l in range(cfg.layers)]
    assert all(0.8 <= v <= 1.6 for v in s) and len(set(s)) == cfg.layers
    p0, p1 = (wl.expert_permutation(cfg.E, wl.tensor_seed(cfg, l, 5)) for l in (0, 1))
    assert sorted(p0) == list(range(cfg.E)) and not np.array_equal(p0, p1)


def test_token_sample_is_stratified():
    s = wl.stratified_token_sample(4096, 64, seed=1)
    assert s[0] == 0 and s[-1] == 4095 and len(set(s)) == len(s) and len(s) >= 60
    assert np.diff(s).max() < 3 * 4096 // 62


def test_expert_weights_equal_the_slices_of_the_full_tensors():
    cfg = wl.MoEConfig("slice", 77, T=8, H=128, I=256, E=5, k=2, S=1)
    gu, dn = wl.make_weights(cfg)
    for e in (0, 3, 5):
        g, d = wl.expert_weights(cfg, e)
        np.testing.assert_array_equal(g, gu[e])
        np.testing.assert_array_equal(d, dn[e])


def test_table1_bench_configs_cover_every_row_and_sequence_length():
    t1 = _table1()
    names = {"DSv3": "dsv3", "Phi-3.5-MoE": "phi35", "Qwen3-30B": "qwen3_30b", "Qwen3.5-35B": "qwen35_35b",
             "DSv2-Lite": "dsv2lite", "DSv2": "dsv2"}
    for row, short in names.items():
        for T in (2048, 4096, 8192, 16384):      # 16k: the longest sequence of the ablation (Section 5.6)
            c = wl.CONFIGS[f"t1_{short}_T{T}"]
            assert (c.E, c.k, c.H, c.I) == t1[row] and c.T == T
