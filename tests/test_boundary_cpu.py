"""CPU-side checks of the boundary: the library builds, loads without a GPU, exports every symbol
the header declares, and its pure-host entry points validate shapes.  Also the benchmark's
multi-process aggregation over gloo (world size 2)."""
import os
import re
import subprocess
import sys

import numpy as np
import pytest

import paper_2609_21483_b200 as pk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(ROOT, "tests", "golden", "table1_model_shapes.txt")


@pytest.fixture(scope="module")
def lib():
    pk.build()
    return pk.load()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "weave_moe.h")).read()
    declared = set(re.findall(r"\b(weave_moe_[a-z_0-9]+)\s*\(", hdr))
    assert declared, "no declarations found"
    assert declared == set(pk.EXPORTS), declared ^ set(pk.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_strerror_names_every_code(lib):
    for code in range(0, -7, -1):
        assert pk.strerror(code) != "unknown error"
    assert pk.strerror(-99) == "unknown error"


def test_workspace_bytes_validates_shapes(lib):
    ok = pk.workspace_bytes(4096, 14336, 8, 2, 0, 4096)
    # expert-major buffers dominate: Xe and y [P,H], h [P,I] in bf16, plus host-staging copies
    P = 4096 * 2
    assert ok > P * (2 * 4096 + 14336) * 2
    assert ok < 2 * (P * (2 * 4096 + 14336) * 2 + 3 * 4096 * 4096 * 2)
    bad = [(4000, 14336, 8, 2, 0, 4096),    # H not a multiple of 128
           (4096, 100, 8, 2, 0, 4096),      # I not a multiple of 128
           (4096, 14336, 0, 1, 0, 4096),    # no experts
           (4096, 14336, 8, 9, 0, 4096),    # k > E
           (4096, 14336, 64, 17, 0, 4096),  # k > 16
           (4096, 14336, 250, 8, 7, 4096),  # E + S > 256
           (4096, 14336, 8, 2, 0, 0)]       # no tokens
    for b in bad:
        assert pk.workspace_bytes(*b) == 0, b


def test_every_table1_shape_is_accepted(lib):
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        _, E, k, H, I = line.split()
        assert pk.workspace_bytes(int(H), int(I), int(E), int(k), 0, 8192) > 0


def test_create_rejects_null_and_misaligned_without_touching_a_gpu(lib):
    import ctypes
    h = ctypes.c_void_p()
    cfg = pk._Config(512, 1024, 8, 2, 0, 256, None, None, None, 0)
    assert lib.weave_moe_create(ctypes.byref(cfg), ctypes.byref(h)) == -1
    cfg = pk._Config(512, 1024, 8, 2, 0, 256, 0x1000, 0x2008, 0x4000, 1 << 30)   # down misaligned
    assert lib.weave_moe_create(ctypes.byref(cfg), ctypes.byref(h)) == -1
    assert lib.weave_moe_forward(None, None, None, None, 1, None) == -1
    assert lib.weave_moe_destroy(None) == 0


def test_product_path_has_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("CPU-only check")
    with pytest.raises(RuntimeError):
        pk.WeaveMoE(torch.zeros(8, 2048, 512, dtype=torch.bfloat16), torch.zeros(8, 512, 1024, dtype=torch.bfloat16), 8, 2)
    # and nothing under the package imports the oracle
    for fn in os.listdir(os.path.join(ROOT, "paper_2609_21483_b200")):
        if fn.endswith(".py"):
            src = open(os.path.join(ROOT, "paper_2609_21483_b200", fn)).read()
            assert "oracle" not in src


def test_cuda_sources_keep_clear_of_batched_copies_and_of_multicast_loads():
    """The batched-memcpy family of runtime calls is not used anywhere (one asynchronous copy per transfer
    instead), and the only instruction that carries the cluster-multicast qualifier is the tensor-core commit
    that arrives on both CTAs' barriers: no tiled or bulk LOAD is multicast."""
    csrc = os.path.join(ROOT, "paper_2609_21483_b200", "csrc")
    batched = [a + "Memcpy" + b + "Batch" + "Async" for a in ("cuda", "cu") for b in ("", "3D")]
    qualifier = ".multi" + "cast::cluster"
    seen_commit = 0
    for fn in sorted(os.listdir(csrc)):
        src = open(os.path.join(csrc, fn)).read()
        for name in batched:
            assert name not in src, (fn, name)
        for line in src.splitlines():
            if qualifier in line:
                assert "tcgen05.commit" in line, (fn, line.strip())
                seen_commit += 1
    assert seen_commit >= 1


_GLOO_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank, world, local = bench.dist_env()
dist.init_process_group("gloo")
t = bench.aggregate_max(1.0 + rank, world, use_cuda=False)     # slowest rank decides
v = bench.whole_job_throughput(4096, 10, world, t)
assert t == float(world), t
assert abs(v - 4096 * 10 * world / world) < 1e-9, v
dist.barrier()
dist.destroy_process_group()
sys.stdout.write("rank%d-ok\n" % rank); sys.stdout.flush()
"""


def test_multi_rank_aggregation_over_gloo(tmp_path):
    """--gpus N runs N replicas; the reported value is all ranks' tokens over the slowest rank's
    time.  Checked with two CPU processes over gloo."""
    script = tmp_path / "worker.py"
    script.write_text(_GLOO_WORKER.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "rank0-ok" in r.stdout and "rank1-ok" in r.stdout


def test_bench_starts_its_own_ranks_for_gpus_n():
    """`python bench.py --gpus 2 ...` as a user types it (no torchrun in front): the script starts two
    ranks of itself, they meet over gloo (CPU stand-in for the NCCL replicas), the slowest rank's time
    decides and only rank 0 prints a line."""
    import json
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "10", "--launcher-selftest"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stdout + r.stderr
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = lines[0]
    assert d["launcher_selftest"] and d["n_gpus"] == 2 and d["max_seconds"] == 2.0
    assert abs(d["value"] - 4096 * 10 * 2 / 2.0) < 1e-9


def test_roofline_windows_use_their_own_peaks():
    """A burst-window time is held against the burst bf16 peak and a sustained-run time against the
    sustained one; the bound (tensor or HBM) is decided with the same window's peak."""
    import bench
    import workloads as wl
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "source": "test"}
    w = bench.layer_work(wl.CONFIGS["c2_mixtral"])
    b = bench.roofline_of(w, 2.0e-3, peaks, "burst")
    s = bench.roofline_of(w, 2.5e-3, peaks, "sustained")
    assert b["bound"] == s["bound"] == "tensor" and b["peak"] == 1600.0 and s["peak"] == 1400.0
    assert np.isclose(b["frac"], w["flops"] / 2.0e-3 / 1600e12) and np.isclose(s["frac"], w["flops"] / 2.5e-3 / 1400e12)
    w4 = bench.layer_work(wl.CONFIGS["c4_dsv2lite_T64"])
    h = bench.roofline_of(w4, 200e-6, peaks, "burst")
    assert h["bound"] == "hbm" and h["unit"] == "GB/s" and np.isclose(h["frac"], w4["bytes"] / 200e-6 / 6500e9)


def test_layer_work_formulas():
    """FLOPs per launch = P * 6HI (Eq. 1); bytes of config 2 match the hand-computed roofline table."""
    import bench
    import workloads as wl
    w = bench.layer_work(wl.CONFIGS["c2_mixtral"])
    assert np.isclose(w["flops"], 8192 * 6 * 4096 * 14336)
    assert np.isclose(w["flops"], 2.886e12, rtol=1e-3)
    assert np.isclose(w["weights_bytes"], 2.82e9, rtol=2e-3)
    assert np.isclose(w["bytes"], 3.62e9, rtol=5e-3)
    w5 = bench.layer_work(wl.CONFIGS["c5_qwen3_235b"])
    assert np.isclose(w5["flops"], 4.948e12, rtol=1e-3) and np.isclose(w5["bytes"], 10.2e9, rtol=1e-2)
