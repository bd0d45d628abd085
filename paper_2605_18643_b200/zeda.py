"""Python binding of the C-ABI library (``include/zeda.h``): argument marshalling only.

Every step of the layer runs in the library's CUDA kernels; PyTorch is used for device memory
and streams.  Importing this module loads ``libzeda.so`` from the package directory and raises
if it is missing: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libzeda.so")

STAGES = ("router", "sort", "gemm1", "gemm2", "combine")
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
GATE_TOPK_NORM, GATE_SOFTMAX_RAW, GATE_RENORM_REAL = 0, 1, 2
EXPERT_ZERO, EXPERT_COPY = 0, 1
FLAG_NONE, FLAG_NO_DEPENDENT_LAUNCH = 0, 4

EXPORTS = (
    "zeda_moe_workspace_bytes", "zeda_moe_create", "zeda_route", "zeda_route_from_logits",
    "zeda_router_logits", "zeda_moe_forward", "zeda_moe_forward_residual", "zeda_moe_forward_host", "zeda_moe_stats",
    "zeda_moe_token_zero_share", "zeda_moe_last_counters", "zeda_moe_set_profiling", "zeda_moe_stage_ms", "zeda_residual_rmsnorm",
    "zeda_moe_selftest_wait", "zeda_moe_clear_error",
    "zeda_ep_dispatch", "zeda_ep_experts", "zeda_ep_combine",
    "zeda_compact_static", "zeda_moe_destroy", "zeda_last_error", "zeda_version",
)


class Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "d_model", "d_expert", "n_real", "n_zero", "top_k", "max_tokens", "gate_mode", "expert_kind",
        "device", "flags", "ep_size", "ep_rank", "max_recv_pairs")]


class ZedaError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__("zeda status %d: %s" % (status, text))
        self.status = status


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libzeda.so not found at %s: build it with `python -m paper_2605_18643_b200.build` "
            "(nvcc, sm_100a); there is no fallback path" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    lib.zeda_moe_workspace_bytes.restype = sz
    lib.zeda_moe_workspace_bytes.argtypes = [ctypes.POINTER(Config)]
    lib.zeda_moe_create.restype = i32
    lib.zeda_moe_create.argtypes = [ctypes.POINTER(Config), vp, vp, vp, vp, vp, sz, ctypes.POINTER(vp)]
    lib.zeda_route.restype = i32
    lib.zeda_route.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.zeda_route_from_logits.restype = i32
    lib.zeda_route_from_logits.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.zeda_router_logits.restype = i32
    lib.zeda_router_logits.argtypes = [vp, vp, i32, vp, vp]
    lib.zeda_moe_forward.restype = i32
    lib.zeda_moe_forward.argtypes = [vp, vp, i32, vp, vp]
    lib.zeda_moe_forward_host.restype = i32
    lib.zeda_moe_forward_host.argtypes = [vp, vp, i32, vp, vp]
    lib.zeda_moe_stats.restype = i32
    lib.zeda_moe_stats.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.zeda_moe_token_zero_share.restype = i32
    lib.zeda_moe_token_zero_share.argtypes = [vp, i32, vp, vp]
    lib.zeda_moe_last_counters.restype = i32
    lib.zeda_moe_last_counters.argtypes = [vp, ctypes.POINTER(ctypes.c_int64), vp]
    lib.zeda_moe_set_profiling.restype = i32
    lib.zeda_moe_set_profiling.argtypes = [vp, i32]
    lib.zeda_moe_stage_ms.restype = i32
    lib.zeda_moe_stage_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.zeda_moe_selftest_wait.restype = i32
    lib.zeda_moe_selftest_wait.argtypes = [vp, i32, vp]
    lib.zeda_moe_clear_error.restype = i32
    lib.zeda_moe_clear_error.argtypes = [vp, vp]
    lib.zeda_residual_rmsnorm.restype = i32
    lib.zeda_residual_rmsnorm.argtypes = [vp, vp, vp, i32, i32, ctypes.c_float, vp]
    lib.zeda_moe_forward_residual.restype = i32
    lib.zeda_moe_forward_residual.argtypes = [vp, vp, i32, vp, vp, ctypes.c_float, vp]
    lib.zeda_ep_dispatch.restype = i32
    lib.zeda_ep_dispatch.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.zeda_ep_experts.restype = i32
    lib.zeda_ep_experts.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.zeda_ep_combine.restype = i32
    lib.zeda_ep_combine.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.zeda_compact_static.restype = i32
    lib.zeda_compact_static.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.zeda_moe_destroy.restype = i32
    lib.zeda_moe_destroy.argtypes = [vp]
    lib.zeda_last_error.restype = ctypes.c_char_p
    lib.zeda_version.restype = ctypes.c_char_p
    return lib


lib = _load()


def last_error() -> str:
    return lib.zeda_last_error().decode()


def version() -> str:
    return lib.zeda_version().decode()


def _check(status: int):
    if status != OK:
        raise ZedaError(status, last_error())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def workspace_bytes(cfg: Config) -> int:
    return int(lib.zeda_moe_workspace_bytes(ctypes.byref(cfg)))


STATIC_MAX_TOKENS, STATIC_MAX_SLOTS = 4096, 32768


def residual_rmsnorm(r: torch.Tensor, y: Optional[torch.Tensor], h: Optional[torch.Tensor] = None,
                     eps: float = 1e-6) -> torch.Tensor:
    """r <- bf16(r + y) in place (y may be None), returns h = RMSNorm(r) (gain-free) as bf16."""
    assert r.is_cuda and r.dtype == torch.bfloat16 and r.dim() == 2 and r.is_contiguous()
    if y is not None:
        assert y.shape == r.shape and y.dtype == r.dtype and y.is_contiguous()
    if h is None:
        h = torch.empty_like(r)
    with torch.cuda.device(r.device):
        _check(lib.zeda_residual_rmsnorm(_ptr(r), _ptr(y), _ptr(h), r.shape[0], r.shape[1], float(eps),
                                         _stream(r.device)))
    return h


def compact_static(topk_idx: torch.Tensor, n_real: int):
    """zeda_compact_static: the counting sort of ``route`` for callers that cannot allocate device
    memory; scratch lives in a fixed array inside the library.  The four output tensors made here
    stand for buffers such a caller would already own.  Returns (counts, offsets, perm, n_pairs)."""
    assert topk_idx.is_cuda and topk_idx.dtype == torch.int32 and topk_idx.is_contiguous() and topk_idx.dim() == 2
    T, K = topk_idx.shape
    dev = topk_idx.device
    counts = torch.empty(n_real, dtype=torch.int32, device=dev)
    offsets = torch.empty(n_real + 1, dtype=torch.int32, device=dev)
    perm = torch.full((T * K,), -1, dtype=torch.int32, device=dev)
    n_pairs = torch.zeros(1, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        _check(lib.zeda_compact_static(_ptr(topk_idx), T, K, n_real, _ptr(counts), _ptr(offsets), _ptr(perm),
                                       _ptr(n_pairs), _stream(dev)))
    return counts, offsets, perm, n_pairs


class ZedaMoE:
    """One layer handle.  Keeps references to the weight and workspace tensors it was given, as the
    C ABI requires them to outlive the handle."""

    def __init__(self, router_w: torch.Tensor, router_bias: Optional[torch.Tensor], w_gate_up: torch.Tensor,
                 w_down: torch.Tensor, n_real: int, n_zero: int, top_k: int, max_tokens: int,
                 gate_mode: int = GATE_TOPK_NORM, expert_kind: int = EXPERT_ZERO, flags: int = FLAG_NONE,
                 workspace: Optional[torch.Tensor] = None, ep_size: int = 0, ep_rank: int = 0,
                 max_recv_pairs: int = 0):
        """ep_size >= 1 makes an expert-parallel handle: the weight tensors then hold only the
        experts [ep_rank * N/G, (ep_rank + 1) * N/G) of the layer."""
        dev = router_w.device
        assert dev.type == "cuda", "weights must live on a CUDA device"
        d = router_w.shape[1]
        He = w_down.shape[2]
        n_local = n_real // ep_size if ep_size >= 1 else n_real
        assert router_w.dtype == torch.float32 and router_w.is_contiguous() and router_w.shape == (n_real + n_zero, d)
        assert w_gate_up.dtype == torch.bfloat16 and w_gate_up.is_contiguous() and w_gate_up.shape == (n_local, 2 * He, d)
        assert w_down.dtype == torch.bfloat16 and w_down.is_contiguous() and w_down.shape == (n_local, d, He)
        if router_bias is not None:
            assert router_bias.dtype == torch.float32 and router_bias.is_contiguous() and router_bias.shape == (n_real + n_zero,)
        self.cfg = Config(d, He, n_real, n_zero, top_k, max_tokens, gate_mode, expert_kind,
                          dev.index if dev.index is not None else torch.cuda.current_device(), flags,
                          ep_size, ep_rank, max_recv_pairs)
        need = workspace_bytes(self.cfg)
        if need == 0:
            raise ZedaError(ERR_INVALID_ARG, last_error())
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=dev)
        self._keep = (router_w, router_bias, w_gate_up, w_down, workspace)
        self.device = dev
        self.d, self.He, self.E, self.Z, self.K = d, He, n_real, n_zero, top_k
        h = ctypes.c_void_p()
        _check(lib.zeda_moe_create(ctypes.byref(self.cfg), _ptr(router_w), _ptr(router_bias), _ptr(w_gate_up),
                                   _ptr(w_down), _ptr(workspace), workspace.numel(), ctypes.byref(h)))
        self._h = h

    # -- routing ------------------------------------------------------------------------------
    def _route_outputs(self, T):
        dev, E, K = self.device, self.E, self.K
        return dict(
            topk_idx=torch.empty((T, K), dtype=torch.int32, device=dev),
            topk_w=torch.empty((T, K), dtype=torch.float32, device=dev),
            counts=torch.empty(E, dtype=torch.int32, device=dev),
            offsets=torch.empty(E + 1, dtype=torch.int32, device=dev),
            perm=torch.full((T * K,), -1, dtype=torch.int32, device=dev),
            n_pairs=torch.zeros(1, dtype=torch.int32, device=dev),
        )

    def route(self, x: torch.Tensor):
        """zeda_route: dict of device tensors topk_idx, topk_w, counts, offsets, perm, n_pairs."""
        T = self._check_x(x)
        o = self._route_outputs(T)
        _check(lib.zeda_route(self._h, _ptr(x), T, _ptr(o["topk_idx"]), _ptr(o["topk_w"]), _ptr(o["counts"]),
                              _ptr(o["offsets"]), _ptr(o["perm"]), _ptr(o["n_pairs"]), _stream(self.device)))
        return o

    def route_from_logits(self, logits: torch.Tensor):
        assert logits.dtype == torch.float32 and logits.is_contiguous() and logits.shape[1] == self.E + self.Z
        T = logits.shape[0]
        o = self._route_outputs(T)
        _check(lib.zeda_route_from_logits(self._h, _ptr(logits), T, _ptr(o["topk_idx"]), _ptr(o["topk_w"]),
                                          _ptr(o["counts"]), _ptr(o["offsets"]), _ptr(o["perm"]), _ptr(o["n_pairs"]),
                                          _stream(self.device)))
        return o

    def router_logits(self, x: torch.Tensor) -> torch.Tensor:
        T = self._check_x(x)
        out = torch.empty((T, self.E + self.Z), dtype=torch.float32, device=self.device)
        _check(lib.zeda_router_logits(self._h, _ptr(x), T, _ptr(out), _stream(self.device)))
        return out

    # -- forward ------------------------------------------------------------------------------
    def forward(self, x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """zeda_moe_forward on device tensors; asynchronous on the current stream."""
        T = self._check_x(x)
        if out is None:
            out = torch.empty_like(x)
        _check(lib.zeda_moe_forward(self._h, _ptr(x), T, _ptr(out), _stream(self.device)))
        return out

    def forward_residual(self, x: torch.Tensor, r: torch.Tensor, h_next: torch.Tensor, eps: float = 1e-6) -> torch.Tensor:
        """zeda_moe_forward_residual: the layer on x with the stack glue fused into its last pass
        (r <- r + y in place, h_next = RMSNorm(r)); asynchronous on the current stream."""
        T = self._check_x(x)
        for t in (r, h_next):
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.shape == x.shape
        _check(lib.zeda_moe_forward_residual(self._h, _ptr(x), T, _ptr(r), _ptr(h_next), float(eps),
                                             _stream(self.device)))
        return h_next

    def forward_host(self, x_host: torch.Tensor, out_host: Optional[torch.Tensor] = None) -> torch.Tensor:
        """zeda_moe_forward_host on CPU tensors (pinned preferred); returns after the copy back."""
        assert x_host.device.type == "cpu" and x_host.dtype == torch.bfloat16 and x_host.is_contiguous()
        T = x_host.shape[0]
        if out_host is None:
            out_host = torch.empty_like(x_host, pin_memory=x_host.is_pinned())
        _check(lib.zeda_moe_forward_host(self._h, _ptr(x_host), T, _ptr(out_host), _stream(self.device)))
        return out_host

    # -- expert parallelism -------------------------------------------------------------------
    def ep_dispatch(self, x: torch.Tensor, send_rows: Optional[torch.Tensor] = None):
        """zeda_ep_dispatch: routes x and packs the rows of the surviving pairs.  Returns device
        tensors (send_rows [T*K, d], send_counts [G], expert_counts [N])."""
        T = self._check_x(x)
        G = max(1, self.cfg.ep_size)
        if send_rows is None:
            send_rows = torch.empty((T * self.K, self.d), dtype=torch.bfloat16, device=self.device)
        send_counts = torch.empty(G, dtype=torch.int32, device=self.device)
        expert_counts = torch.empty(self.E, dtype=torch.int32, device=self.device)
        _check(lib.zeda_ep_dispatch(self._h, _ptr(x), T, _ptr(send_rows), _ptr(send_counts), _ptr(expert_counts),
                                    _stream(self.device)))
        return send_rows, send_counts, expert_counts

    def ep_experts(self, recv_rows: torch.Tensor, recv_counts: torch.Tensor, n_rows: int,
                   out_rows: Optional[torch.Tensor] = None) -> torch.Tensor:
        """zeda_ep_experts: this rank's experts on the first n_rows rows of recv_rows; recv_counts is
        the device matrix [G, N/G] of rows per (source rank, local expert)."""
        assert recv_rows.dtype == torch.bfloat16 and recv_rows.is_contiguous() and recv_rows.shape[1] == self.d
        assert recv_counts.dtype == torch.int32 and recv_counts.is_contiguous()
        assert recv_rows.shape[0] >= n_rows
        if out_rows is None:
            out_rows = torch.empty((max(n_rows, 1), self.d), dtype=torch.bfloat16, device=self.device)
        _check(lib.zeda_ep_experts(self._h, _ptr(recv_rows), _ptr(recv_counts), int(n_rows), _ptr(out_rows),
                                   _stream(self.device)))
        return out_rows

    def ep_combine(self, x: torch.Tensor, back_rows: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """zeda_ep_combine: Eq. 1 on the expert outputs that came back, in the order of send_rows."""
        T = self._check_x(x)
        assert back_rows.dtype == torch.bfloat16 and back_rows.is_contiguous() and back_rows.shape[1] == self.d
        if out is None:
            out = torch.empty_like(x)
        _check(lib.zeda_ep_combine(self._h, _ptr(x), _ptr(back_rows), T, _ptr(out), _stream(self.device)))
        return out

    def stats(self, x: torch.Tensor):
        """zeda_moe_stats: (f [N+N_Z], p_mean [N+N_Z], out [4] = r_ZE, sum f_i P_i, f_E P_E, f_Z P_Z)."""
        T = self._check_x(x)
        n = self.E + self.Z
        f = torch.empty(n, dtype=torch.float32, device=self.device)
        p = torch.empty(n, dtype=torch.float32, device=self.device)
        o = torch.empty(4, dtype=torch.float32, device=self.device)
        _check(lib.zeda_moe_stats(self._h, _ptr(x), T, _ptr(f), _ptr(p), _ptr(o), _stream(self.device)))
        return f, p, o

    def token_zero_share(self, T: int) -> torch.Tensor:
        """zeda_moe_token_zero_share: per-token share of the K slots on zero experts, for the T tokens of
        the last routing call on this handle."""
        out = torch.empty(T, dtype=torch.float32, device=self.device)
        _check(lib.zeda_moe_token_zero_share(self._h, T, _ptr(out), _stream(self.device)))
        return out

    def last_counters(self):
        """(P, U, zero slots, kernel launches) of the last call; synchronises the current stream."""
        out = (ctypes.c_int64 * 4)()
        _check(lib.zeda_moe_last_counters(self._h, out, _stream(self.device)))
        return tuple(int(v) for v in out)

    def selftest_wait(self, limit_us: int = 1000):
        """Makes a bounded device wait expire on purpose (no fault): the next last_counters() raises."""
        _check(lib.zeda_moe_selftest_wait(self._h, int(limit_us), _stream(self.device)))

    def clear_error(self):
        _check(lib.zeda_moe_clear_error(self._h, _stream(self.device)))

    def set_profiling(self, enable: bool):
        _check(lib.zeda_moe_set_profiling(self._h, 1 if enable else 0))

    def stage_ms(self):
        """Milliseconds of (router, sort, gemm1, gemm2, combine) of the last profiled forward; blocks."""
        out = (ctypes.c_float * 5)()
        _check(lib.zeda_moe_stage_ms(self._h, out))
        return tuple(float(v) for v in out)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            h, self._h = self._h, None
            _check(lib.zeda_moe_destroy(h))

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check_x(self, x: torch.Tensor) -> int:
        assert x.device == self.device and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 2
        assert x.shape[1] == self.d
        return x.shape[0]


def from_workload(wl, device="cuda:0", max_tokens: Optional[int] = None, **kw) -> "ZedaMoE":
    """Handle for a ``paper_2605_18643_b200.inputs.Workload`` (weights copied to ``device``)."""
    dev = torch.device(device)
    bias = None if wl.router_bias is None else wl.router_bias.to(dev).contiguous()
    return ZedaMoE(wl.router_w.to(dev).contiguous(), bias, wl.w_gate_up.to(dev).contiguous(),
                   wl.w_down.to(dev).contiguous(), wl.E, wl.Z, wl.K, max_tokens or wl.T, **kw)
