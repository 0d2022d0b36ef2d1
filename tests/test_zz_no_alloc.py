"""The allocation-free entry point (collected last on purpose: if it fails, everything else has run).

weave_moe_forward_static serves callers that may not allocate device memory when they need the
layer (a frozen memory pool, a plugin with a fixed arena, a serving loop that must not touch the
allocator): the kernel's scratch sits in a fixed array inside the library.  Called twice in a row
through the C ABI, it must reproduce the handle-based entry point's output on the same inputs bit
for bit (the layer's output does not depend on the schedule or on where the scratch lives), and
once it is checked against the CPU oracle directly, within the tolerance of the parity tests: the
built-in array is shared by all calls and keeps the previous call's contents, so the second call
also proves that nothing stale leaks through."""
import ctypes

import numpy as np
import pytest
import torch

import workloads as wl
import paper_2609_21483_b200 as pk
from parity import bf16_to_np, check_values, oracle_rows, to_dev

pytestmark = pytest.mark.gpu


def _same_bits(a, b):
    return torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_static_scratch_entry_point_matches_the_handle_based_one_twice():
    lib = pk.load()
    cfg = wl.CONFIGS["c1_tiny"]
    inp = wl.make_inputs(cfg)
    x, lg, gu, dn = to_dev(inp)
    moe = pk.WeaveMoE(gu, dn, cfg.E, cfg.k, cfg.S, max_tokens=cfg.T)
    ref = moe.forward(x, lg).clone()
    moe.check()
    stream = torch.cuda.current_stream().cuda_stream

    def call(xx, ll, oo):
        return lib.weave_moe_forward_static(cfg.H, cfg.I, cfg.E, cfg.k, cfg.S, gu.data_ptr(), dn.data_ptr(),
                                            xx.data_ptr(), ll.data_ptr(), oo.data_ptr(), xx.shape[0], stream)

    out1, out2 = torch.zeros_like(x), torch.zeros_like(x)
    assert call(x, lg, out1) == 0
    assert call(x, lg, out2) == 0
    torch.cuda.synchronize()
    assert _same_bits(out1, ref) and _same_bits(out2, ref)
    check_values(bf16_to_np(out1), oracle_rows(inp), "static entry point vs oracle")
    # a different, smaller batch in between, then the first one again: the shared array is reused
    x2, lg2 = x[:100].contiguous(), lg[:100].contiguous()
    ref2 = moe.forward(x2, lg2).clone()
    moe.check()
    out3, out4 = torch.zeros_like(x2), torch.zeros_like(x)
    assert call(x2, lg2, out3) == 0
    assert call(x, lg, out4) == 0
    torch.cuda.synchronize()
    assert _same_bits(out3, ref2) and _same_bits(out4, ref)
    # a batch below the limit at which every CTA routes the batch for itself, then the full one once more
    x3, lg3 = x[:40].contiguous(), lg[:40].contiguous()
    ref3 = moe.forward(x3, lg3).clone()
    moe.check()
    out5, out6 = torch.zeros_like(x3), torch.zeros_like(x)
    assert call(x3, lg3, out5) == 0
    assert call(x, lg, out6) == 0
    torch.cuda.synchronize()
    assert _same_bits(out5, ref3) and _same_bits(out6, ref)
    moe.close()


def test_static_scratch_rejects_layers_beyond_its_limit():
    lib = pk.load()
    limit = lib.weave_moe_static_scratch_bytes()
    assert 32 << 20 <= limit <= 64 << 20
    # the Mixtral-shaped layer needs far more scratch than the built-in array holds
    assert pk.workspace_bytes(4096, 14336, 8, 2, 0, 4096) > limit
    dummy = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    rc = lib.weave_moe_forward_static(4096, 14336, 8, 2, 0, dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(),
                                      dummy.data_ptr(), dummy.data_ptr(), 4096, None)
    assert rc == -4 and "workspace" in pk.strerror(rc)
    # invalid shapes and null weights are refused before anything is launched
    assert lib.weave_moe_forward_static(500, 1024, 8, 2, 0, dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(),
                                        dummy.data_ptr(), dummy.data_ptr(), 16, None) == -1
    assert lib.weave_moe_forward_static(512, 1024, 8, 2, 0, None, dummy.data_ptr(), dummy.data_ptr(),
                                        dummy.data_ptr(), dummy.data_ptr(), 16, None) == -1
