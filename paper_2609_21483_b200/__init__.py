"""Python binding of the weave_moe C ABI (include/weave_moe.h).

Argument marshalling only: every step of the layer runs inside the CUDA library.  PyTorch is
used for device memory and streams.  There is no CPU or eager fallback: if the shared library
is missing or the device is not an sm_100 GPU, calls fail loudly.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC_DIR = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libweave_moe.so")
_SOURCES = ["weave_moe.cu", "weave_kernel.cuh", "weave_ptx.cuh"]

WEAVE_OK = 0
WEAVE_ERR_INVALID_ARG = -1
SCHED_AUTO, SCHED_FIXED, SCHED_SERIAL = 0, 1, 2
PLAN_SPLIT, PLAN_DISPATCH_ALL, PLAN_PHASED, PLAN_REJOIN = 0, 1, 2, 3
ERR_NONFINITE_LOGITS, ERR_TIMEOUT = -5, -6

_lib = None


class WeaveError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


def build(force: bool = False, verbose: bool = False) -> str:
    """nvcc -gencode arch=compute_100a,code=sm_100a -> libweave_moe.so next to this file."""
    srcs = [os.path.join(_SRC_DIR, s) for s in _SOURCES]
    hdr = os.path.join(os.path.dirname(_HERE), "include", "weave_moe.h")
    newest = max(os.path.getmtime(p) for p in srcs + [hdr])
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= newest:
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", LIB_PATH, srcs[0], "-lcudart"]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    return LIB_PATH


class _Config(ctypes.Structure):
    _fields_ = [("hidden", ctypes.c_int), ("ffn", ctypes.c_int), ("num_experts", ctypes.c_int),
                ("top_k", ctypes.c_int), ("num_shared", ctypes.c_int), ("max_tokens", ctypes.c_int),
                ("gate_up", ctypes.c_void_p), ("down", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


EXPORTS = [
    "weave_moe_workspace_bytes", "weave_moe_create", "weave_moe_forward", "weave_moe_forward_host",
    "weave_moe_destroy", "weave_moe_set_schedule", "weave_moe_set_cost_tables", "weave_moe_get_plan",
    "weave_moe_get_geometry", "weave_moe_get_routing", "weave_moe_get_intermediates",
    "weave_moe_status", "weave_moe_set_timeout_ms", "weave_moe_debug_withhold_flag",
    "weave_moe_last_cuda_error", "weave_moe_strerror", "weave_moe_set_trace",
    "weave_moe_forward_static", "weave_moe_static_scratch_bytes", "weave_moe_set_sm_count",
    "weave_moe_set_expert_parallel", "weave_moe_get_ep_descriptors",
    "weave_moe_forward_host_pipelined", "weave_moe_host_wait", "weave_moe_debug_gemm_queue",
    "weave_moe_get_plan_kind", "weave_moe_set_model_options", "weave_moe_last_timeout_where",
    "weave_moe_debug_wait_log",
]


def load():
    """dlopen the library and declare the prototypes.  Fails if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: run __graft_entry__.build() (there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cip, cfp = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_float)
    vpp = ctypes.POINTER(ctypes.c_void_p)
    lib.weave_moe_workspace_bytes.restype = ctypes.c_size_t
    lib.weave_moe_workspace_bytes.argtypes = [ctypes.POINTER(_Config)]
    lib.weave_moe_create.restype = ci
    lib.weave_moe_create.argtypes = [ctypes.POINTER(_Config), vpp]
    lib.weave_moe_forward.restype = ci
    lib.weave_moe_forward.argtypes = [vp, vp, vp, vp, ci, vp]
    lib.weave_moe_forward_host.restype = ci
    lib.weave_moe_forward_host.argtypes = [vp, vp, vp, vp, ci, vp]
    lib.weave_moe_forward_host_pipelined.restype = ci
    lib.weave_moe_forward_host_pipelined.argtypes = [vp, vp, vp, vp, ci, vp]
    lib.weave_moe_host_wait.restype = ci
    lib.weave_moe_host_wait.argtypes = [vp]
    lib.weave_moe_destroy.restype = ci
    lib.weave_moe_destroy.argtypes = [vp]
    lib.weave_moe_set_schedule.restype = ci
    lib.weave_moe_set_schedule.argtypes = [vp, ci, ci, ci, ci]
    lib.weave_moe_set_cost_tables.restype = ci
    lib.weave_moe_set_cost_tables.argtypes = [vp, vp, vp, vp, ctypes.c_float, ci, ci, ci]
    lib.weave_moe_get_plan.restype = ci
    lib.weave_moe_get_plan.argtypes = [vp, cip, cip, cip, cfp]
    lib.weave_moe_get_plan_kind.restype = ci
    lib.weave_moe_get_plan_kind.argtypes = [vp, cip]
    lib.weave_moe_set_model_options.restype = ci
    lib.weave_moe_set_model_options.argtypes = [vp, ci, ci]
    lib.weave_moe_last_timeout_where.restype = ci
    lib.weave_moe_last_timeout_where.argtypes = [vp]
    lib.weave_moe_debug_wait_log.restype = ci
    lib.weave_moe_debug_wait_log.argtypes = [vp, vp, ci]
    lib.weave_moe_get_geometry.restype = ci
    lib.weave_moe_get_geometry.argtypes = [vp, cip, cip, cip, cip, cip, cip, cip]
    lib.weave_moe_get_routing.restype = ci
    lib.weave_moe_get_routing.argtypes = [vp, vpp, vpp, vpp, vpp, vpp, vpp]
    lib.weave_moe_get_intermediates.restype = ci
    lib.weave_moe_get_intermediates.argtypes = [vp, vpp, vpp, vpp]
    lib.weave_moe_status.restype = ci
    lib.weave_moe_status.argtypes = [vp]
    lib.weave_moe_set_timeout_ms.restype = ci
    lib.weave_moe_set_timeout_ms.argtypes = [vp, ci]
    lib.weave_moe_debug_withhold_flag.restype = ci
    lib.weave_moe_debug_withhold_flag.argtypes = [vp, ci]
    lib.weave_moe_set_expert_parallel.restype = ci
    lib.weave_moe_set_expert_parallel.argtypes = [vp, ci, ci]
    lib.weave_moe_get_ep_descriptors.restype = ci
    lib.weave_moe_get_ep_descriptors.argtypes = [vp] + [ctypes.POINTER(ctypes.c_longlong)] * 3
    lib.weave_moe_set_sm_count.restype = ci
    lib.weave_moe_set_sm_count.argtypes = [vp, ci]
    lib.weave_moe_set_trace.restype = ci
    lib.weave_moe_set_trace.argtypes = [vp, vp, ci]
    lib.weave_moe_forward_static.restype = ci
    lib.weave_moe_forward_static.argtypes = [ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, ci, vp]
    lib.weave_moe_static_scratch_bytes.restype = ctypes.c_size_t
    lib.weave_moe_static_scratch_bytes.argtypes = []
    lib.weave_moe_last_cuda_error.restype = ci
    lib.weave_moe_last_cuda_error.argtypes = [vp]
    lib.weave_moe_debug_gemm_queue.restype = ci
    lib.weave_moe_debug_gemm_queue.argtypes = [vp, ci, ci, ci, ci, vp, ci]
    lib.weave_moe_strerror.restype = ctypes.c_char_p
    lib.weave_moe_strerror.argtypes = [ci]
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().weave_moe_strerror(code).decode()


def gemm_queue(rows, nt0: int, nt1: int):
    """Host-only: the GEMM tile queue for rows[chunk][expert] -> int32 array [n_tiles, 6] of
    (type, leader m-block, peer m-block or -1, n-tile, chunk, leader rows); no GPU involved."""
    import numpy as np
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    if rows.ndim == 1:
        rows = rows[None, :]
    K, EE = rows.shape
    n = load().weave_moe_debug_gemm_queue(rows.ctypes.data, EE, K, nt0, nt1, None, 0)
    if n < 0:
        raise WeaveError(n, "weave_moe_debug_gemm_queue")
    out = np.zeros((n, 6), np.int32)
    if n:
        _check(0 if load().weave_moe_debug_gemm_queue(rows.ctypes.data, EE, K, nt0, nt1, out.ctypes.data, n) == n
               else WEAVE_ERR_INVALID_ARG, "weave_moe_debug_gemm_queue")
    return out


def workspace_bytes(hidden, ffn, num_experts, top_k, num_shared, max_tokens) -> int:
    cfg = _Config(hidden, ffn, num_experts, top_k, num_shared, max_tokens, None, None, None, 0)
    return int(load().weave_moe_workspace_bytes(ctypes.byref(cfg)))


def _check(rc: int, what: str):
    if rc != WEAVE_OK:
        raise WeaveError(rc, what)


def forward_static(x, logits, gate_up, down, num_experts: int, top_k: int, num_shared: int = 0, out=None,
                   stream: Optional[int] = None):
    """The layer for callers that must not allocate device memory: no handle, no workspace; the
    kernel's scratch is a fixed array inside the library (see weave_moe_forward_static in the
    header for the size limit and the sharing rules).  `out` must be passed by such callers; it is
    created here only as a convenience when omitted."""
    import torch
    lib = load()
    EE, twoI, H = gate_up.shape
    T = x.shape[0]
    assert x.is_cuda and logits.is_cuda and gate_up.is_cuda and down.is_cuda
    assert x.dtype == torch.bfloat16 and logits.dtype == torch.float32
    assert x.is_contiguous() and logits.is_contiguous() and gate_up.is_contiguous() and down.is_contiguous()
    if out is None:
        out = torch.empty_like(x)
    if stream is None:
        stream = torch.cuda.current_stream(x.device).cuda_stream
    with torch.cuda.device(x.device):
        _check(lib.weave_moe_forward_static(H, twoI // 2, num_experts, top_k, num_shared, gate_up.data_ptr(),
                                            down.data_ptr(), x.data_ptr(), logits.data_ptr(), out.data_ptr(), T,
                                            stream), "weave_moe_forward_static")
    return out


class WeaveMoE:
    """One MoE layer: weights [E+S,2I,H] / [E+S,H,I] bf16 on the GPU, a workspace, a handle."""

    def __init__(self, gate_up, down, num_experts: int, top_k: int, num_shared: int = 0,
                 max_tokens: int = 4096):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("WeaveMoE needs a CUDA device (sm_100); there is no CPU path")
        self._torch = torch
        self._lib = load()
        assert gate_up.is_cuda and down.is_cuda and gate_up.dtype == torch.bfloat16 and down.dtype == torch.bfloat16
        assert gate_up.is_contiguous() and down.is_contiguous()
        EE, twoI, H = gate_up.shape
        I = twoI // 2
        assert EE == num_experts + num_shared and tuple(down.shape) == (EE, H, I)
        self.H, self.I, self.E, self.k, self.S, self.max_tokens = H, I, num_experts, top_k, num_shared, max_tokens
        self.gate_up, self.down = gate_up, down
        nbytes = workspace_bytes(H, I, num_experts, top_k, num_shared, max_tokens)
        if nbytes == 0:
            raise WeaveError(-1, "weave_moe_workspace_bytes")
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=gate_up.device)
        base = self.workspace.data_ptr()
        self._ws_off = (-base) % 1024
        cfg = _Config(H, I, num_experts, top_k, num_shared, max_tokens, gate_up.data_ptr(), down.data_ptr(),
                      base + self._ws_off, nbytes)
        self._h = ctypes.c_void_p()
        with torch.cuda.device(gate_up.device):
            _check(self._lib.weave_moe_create(ctypes.byref(cfg), ctypes.byref(self._h)), "weave_moe_create")
        self.last_T = 0

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self._torch.cuda.synchronize()
            self._lib.weave_moe_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the layer
    def forward(self, x, logits, out=None, stream: Optional[int] = None):
        torch = self._torch
        T = x.shape[0]
        assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.shape[1] == self.H
        assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
        assert tuple(logits.shape) == (T, self.E)
        if out is None:
            out = torch.empty_like(x)
        if stream is None:
            stream = torch.cuda.current_stream(x.device).cuda_stream
        _check(self._lib.weave_moe_forward(self._h, x.data_ptr(), logits.data_ptr(), out.data_ptr(), T, stream),
               "weave_moe_forward")
        self.last_T = T
        return out

    def forward_host(self, x_host, logits_host, out_host, stream: Optional[int] = None):
        """x_host/out_host: CPU bf16 [T,H]; logits_host: CPU fp32 [T,E] (pinned for async copies)."""
        torch = self._torch
        T = x_host.shape[0]
        assert not x_host.is_cuda and not logits_host.is_cuda and not out_host.is_cuda
        assert x_host.dtype == torch.bfloat16 and logits_host.dtype == torch.float32 and out_host.dtype == torch.bfloat16
        assert x_host.is_contiguous() and logits_host.is_contiguous() and out_host.is_contiguous()
        if stream is None:
            stream = torch.cuda.current_stream(self.gate_up.device).cuda_stream
        _check(self._lib.weave_moe_forward_host(self._h, x_host.data_ptr(), logits_host.data_ptr(),
                                                out_host.data_ptr(), T, stream), "weave_moe_forward_host")
        self.last_T = T
        return out_host

    def forward_host_pipelined(self, x_host, logits_host, out_host, stream: Optional[int] = None):
        """Like forward_host, but copies overlap the neighbouring calls' kernels; call host_wait()
        before reading out_host."""
        torch = self._torch
        T = x_host.shape[0]
        assert x_host.is_pinned() and logits_host.is_pinned() and out_host.is_pinned()
        assert x_host.dtype == torch.bfloat16 and logits_host.dtype == torch.float32 and out_host.dtype == torch.bfloat16
        assert x_host.is_contiguous() and logits_host.is_contiguous() and out_host.is_contiguous()
        if stream is None:
            stream = torch.cuda.current_stream(self.gate_up.device).cuda_stream
        _check(self._lib.weave_moe_forward_host_pipelined(self._h, x_host.data_ptr(), logits_host.data_ptr(),
                                                          out_host.data_ptr(), T, stream),
               "weave_moe_forward_host_pipelined")
        self.last_T = T
        return out_host

    def host_wait(self):
        _check(self._lib.weave_moe_host_wait(self._h), "weave_moe_host_wait")

    # ---- scheduling
    def set_schedule(self, mode: int, c: int = 0, K: int = 1, steal: int = 0):
        _check(self._lib.weave_moe_set_schedule(self._h, mode, c, K, steal), "weave_moe_set_schedule")

    def set_cost_tables(self, bw, tflops, eff_chunk, alpha: float, c_min: int = 2, c_max: int = 74, c_step: int = 2):
        import numpy as np
        bw = np.ascontiguousarray(bw, dtype=np.float32)
        tf = np.ascontiguousarray(tflops, dtype=np.float32)
        eff = np.ascontiguousarray(eff_chunk, dtype=np.float32)
        n_sm = self.geometry()["n_sm"]
        assert bw.shape == (n_sm + 1,) and tf.shape == (n_sm + 1,) and eff.shape == (4,)
        _check(self._lib.weave_moe_set_cost_tables(self._h, bw.ctypes.data, tf.ctypes.data, eff.ctypes.data,
                                                   alpha, c_min, c_max, c_step), "weave_moe_set_cost_tables")

    def plan(self):
        c, K, s, t = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_float()
        _check(self._lib.weave_moe_get_plan(self._h, ctypes.byref(c), ctypes.byref(K), ctypes.byref(s),
                                            ctypes.byref(t)), "weave_moe_get_plan")
        kind = ctypes.c_int()
        _check(self._lib.weave_moe_get_plan_kind(self._h, ctypes.byref(kind)), "weave_moe_get_plan_kind")
        return {"c": c.value, "K": K.value, "n_steal": s.value, "t_total_us": t.value, "kind": kind.value}

    def set_model_options(self, kinds_mask: int = 7, elastic: int = -1):
        """Plan kinds AUTO may choose (bit 0 the paper's split, bit 1 dispatch-all, bit 2 phased, bit 3 rejoin) and
        the elastic-stealing switch (-1 = on under AUTO only)."""
        _check(self._lib.weave_moe_set_model_options(self._h, kinds_mask, elastic), "weave_moe_set_model_options")

    def last_timeout_where(self) -> int:
        return int(self._lib.weave_moe_last_timeout_where(self._h))

    def wait_log(self):
        """Records {cta, warp, wait id, object, wanted, how} of the waits that failed in the launch whose
        failure the last status() reported."""
        n = int(self._lib.weave_moe_debug_wait_log(self._h, None, 0))
        buf = (ctypes.c_int32 * (6 * max(n, 1)))()
        n = min(n, int(self._lib.weave_moe_debug_wait_log(self._h, buf, n)))
        return [tuple(buf[6 * i:6 * i + 6]) for i in range(n)]

    def geometry(self):
        v = [ctypes.c_int() for _ in range(7)]
        _check(self._lib.weave_moe_get_geometry(self._h, *[ctypes.byref(a) for a in v]), "weave_moe_get_geometry")
        names = ["n_sm", "block_m", "tile_n0", "tile_n1", "route_block", "combine_tile", "gemm_tile_m"]
        return {n: a.value for n, a in zip(names, v)}

    # ---- verification surface
    def _view(self, ptr: int, count: int, dtype):
        torch = self._torch
        off = ptr - self.workspace.data_ptr()
        nbytes = count * torch.empty((), dtype=dtype).element_size()
        assert 0 <= off and off + nbytes <= self.workspace.numel()
        return self.workspace[off:off + nbytes].view(dtype)

    def routing(self, T: Optional[int] = None):
        """Views into the workspace (valid until the next forward)."""
        torch = self._torch
        T = self.last_T if T is None else T
        p = [ctypes.c_void_p() for _ in range(6)]
        _check(self._lib.weave_moe_get_routing(self._h, *[ctypes.byref(a) for a in p]), "weave_moe_get_routing")
        EE, P = self.E + self.S, T * (self.k + self.S)
        return {
            "topk_idx": self._view(p[0].value, T * self.k, torch.int32).view(T, self.k),
            "gates": self._view(p[1].value, T * self.k, torch.float32).view(T, self.k),
            "counts": self._view(p[2].value, EE, torch.int32),
            "offsets": self._view(p[3].value, EE + 1, torch.int32),
            "row_of": self._view(p[4].value, T * self.k, torch.int32).view(T, self.k),
            "token_of": self._view(p[5].value, P, torch.int32),
        }

    def intermediates(self, T: Optional[int] = None):
        torch = self._torch
        T = self.last_T if T is None else T
        P = T * (self.k + self.S)
        p = [ctypes.c_void_p() for _ in range(3)]
        _check(self._lib.weave_moe_get_intermediates(self._h, *[ctypes.byref(a) for a in p]),
               "weave_moe_get_intermediates")
        return {
            "xe": self._view(p[0].value, P * self.H, torch.bfloat16).view(P, self.H),
            "h": self._view(p[1].value, P * self.I, torch.bfloat16).view(P, self.I),
            "y": self._view(p[2].value, P * self.H, torch.bfloat16).view(P, self.H),
        }

    def status(self) -> int:
        """Synchronises; returns 0, ERR_NONFINITE_LOGITS or ERR_TIMEOUT and clears it."""
        return int(self._lib.weave_moe_status(self._h))

    def check(self):
        st = self.status()
        if st != WEAVE_OK:
            raise WeaveError(st, f"device status (wait id {self._lib.weave_moe_last_timeout_where(self._h)})")

    def set_expert_parallel(self, ep_rank: int, ep_size: int):
        """Act as rank ep_rank of ep_size (see weave_moe_set_expert_parallel); ep_size = 1 = off."""
        _check(self._lib.weave_moe_set_expert_parallel(self._h, ep_rank, ep_size), "weave_moe_set_expert_parallel")

    def ep_descriptors(self):
        v = [ctypes.c_longlong() for _ in range(3)]
        _check(self._lib.weave_moe_get_ep_descriptors(self._h, *[ctypes.byref(a) for a in v]),
               "weave_moe_get_ep_descriptors")
        return {"x_local": v[0].value, "x_in": v[1].value, "x_in_uniq": v[2].value}

    def set_sm_count(self, n_sm: int):
        _check(self._lib.weave_moe_set_sm_count(self._h, n_sm), "weave_moe_set_sm_count")

    def set_timeout_ms(self, ms: int):
        _check(self._lib.weave_moe_set_timeout_ms(self._h, ms), "weave_moe_set_timeout_ms")

    def debug_withhold_flag(self, m_block: int):
        _check(self._lib.weave_moe_debug_withhold_flag(self._h, m_block), "weave_moe_debug_withhold_flag")

    # ---- timeline
    def enable_trace(self, events_per_cta: int = 2048):
        """Allocates the event buffer and switches the in-kernel timeline on (0 = off)."""
        torch = self._torch
        if events_per_cta <= 0:
            _check(self._lib.weave_moe_set_trace(self._h, None, 0), "weave_moe_set_trace")
            self._trace = None
            return
        n_sm = self.geometry()["n_sm"]
        self._trace = torch.zeros(n_sm, events_per_cta, 4, dtype=torch.int32, device=self.gate_up.device)
        _check(self._lib.weave_moe_set_trace(self._h, self._trace.data_ptr(), events_per_cta), "weave_moe_set_trace")

    def read_trace(self):
        """Events of the last forward: list (one per CTA) of arrays [n,4] = start, end, kind<<24|id, extra."""
        import numpy as np
        self._torch.cuda.synchronize()
        raw = self._trace.cpu().numpy().view(np.uint32)
        return [raw[c, :int(raw[c, -1, 0])] for c in range(raw.shape[0])]
