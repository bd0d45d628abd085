"""Seeded synthetic workloads for the zero-expert MoE layer.

This module only *makes inputs*: tensors with the shapes of a Qwen3-30B-A3B MoE
layer (Appendix D, table of architectural parameters: H=2048, H_e=768, N=128,
N_Z=64, K=8), a router whose zero-expert rows are drawn from the same Gaussian
as the normal rows (the initialisation rule of Section 2.1), and a router bias
that steers the share of top-K slots landing on zero experts to a target
(about one half, the equilibrium N_Z w / (N + N_Z w) of Section 2.2 for
N=128, N_Z=64, w=2).  It holds no part of the layer's forward arithmetic and
is imported by neither the CUDA library nor the CPU oracle; the tests and the
benchmark hand its tensors to both.

The only arithmetic here is input conditioning: a float64 matrix product and a
sort to (a) find the bias offset that gives the requested zero-slot fraction and
(b) redraw token rows whose top-(K+1) logits are closer than the tie margin, so
that a top-K decision never hangs on the last bits of a logit.
"""
from __future__ import annotations

import dataclasses
import functools
import math
from typing import Optional

import numpy as np
import torch

TIE_MARGIN = 1.0e-3
_MARGIN_SLACK = 1.1  # generate with 10 % head-room over the stated margin

# tensor ids for derived seeds: seed * 1000 + id
_ID_X, _ID_ROUTER, _ID_GATE_UP, _ID_DOWN, _ID_PERM, _ID_SHIFT, _ID_REDRAW = 1, 2, 3, 4, 5, 6, 7


@dataclasses.dataclass
class Workload:
    name: str
    T: int
    d: int
    He: int
    E: int
    Z: int
    K: int
    x: torch.Tensor                      # [T, d] bf16
    router_w: torch.Tensor               # [E+Z, d] fp32, rows 0..E-1 normal, E.. zero experts
    router_bias: Optional[torch.Tensor]  # [E+Z] fp32 or None
    w_gate_up: torch.Tensor              # [E, 2*He, d] bf16, gate rows first
    w_down: torch.Tensor                 # [E, d, He] bf16
    zero_bias: float = 0.0               # offset added to every zero-expert bias entry
    zero_fraction: float = 0.0           # measured share of top-K slots on zero experts
    redrawn_tokens: int = 0

    @property
    def n_cand(self) -> int:
        return self.E + self.Z


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> uint16 numpy array holding the same bit patterns."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def _gen(seed: int, tensor_id: int, extra: int = 0) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 1000 + tensor_id + 7919 * extra)
    return g


def _normal(shape, std, seed, tensor_id, dtype, extra=0):
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=dtype)
    g = _gen(seed, tensor_id, extra)
    step = 1 << 24
    for s in range(0, n, step):  # chunked: fp32 scratch stays small
        m = min(step, n - s)
        out[s:s + m] = (torch.randn(m, generator=g, dtype=torch.float32) * std).to(dtype)
    return out.view(*shape)


@functools.lru_cache(maxsize=2)
def expert_weights(E: int, He: int, d: int, seed: int = 0):
    """Expert weights ~ N(0, 0.02^2) in bf16: ([E, 2He, d], [E, d, He])."""
    w_gate_up = _normal((E, 2 * He, d), 0.02, seed, _ID_GATE_UP, torch.bfloat16)
    w_down = _normal((E, d, He), 0.02, seed, _ID_DOWN, torch.bfloat16)
    return w_gate_up, w_down


def _topk_gaps(logits32: torch.Tensor, K: int) -> torch.Tensor:
    """Smallest gap between neighbours among the K+1 largest logits of each row."""
    kk = min(K + 1, logits32.shape[1])
    top = torch.topk(logits32, kk, dim=1, sorted=True).values
    if kk < 2:
        return torch.full((logits32.shape[0],), float("inf"))
    return (top[:, :-1] - top[:, 1:]).min(dim=1).values


def _zero_fraction(logits32: torch.Tensor, E: int, K: int) -> float:
    idx = torch.topk(logits32, K, dim=1).indices
    return float((idx >= E).float().mean())


def _logits32(x: torch.Tensor, router_w: torch.Tensor, bias: Optional[torch.Tensor]) -> torch.Tensor:
    l = x.double() @ router_w.double().t()
    if bias is not None:
        l = l + bias.double()
    return l.float()


def make_layer(name: str, T: int, d: int, He: int, E: int, Z: int, K: int, seed: int = 0,
               zero_fraction: Optional[float] = 0.5, zipf_s: float = 0.0,
               token_shift: float = 0.0, weight_seed: Optional[int] = None,
               x: Optional[torch.Tensor] = None, with_experts: bool = True) -> Workload:
    """One layer's worth of seeded inputs.

    zero_fraction: target mean share of top-K slots on zero experts (ignored when Z == 0;
        None leaves the zero rows unbiased).
    zipf_s: > 0 puts a log-Zipf(s) popularity prior on the normal experts' bias
        (b_e = log p_pi(e), p_k ~ k^-s, pi a seeded permutation).
    token_shift: a > 0 adds a * u (u a seeded unit vector) to every zero-expert router row, so
        each token's zero logits move together by a * <x_t, u> ~ N(0, a^2) and the per-token
        zero share spreads from 0 to 100 %.
    x: optional caller-supplied activations (used by the layer stack); rows are never redrawn then.
    with_experts: False leaves w_gate_up / w_down as None (the layer stack draws them on the device
        with device_expert_weights: 58 GB of them do not pass through host memory).
    """
    assert K <= E + Z
    ws = seed if weight_seed is None else weight_seed
    w_gate_up, w_down = expert_weights(E, He, d, ws) if with_experts else (None, None)
    router_w = _normal((E + Z, d), 0.02, seed, _ID_ROUTER, torch.float32)
    own_x = x is None
    if own_x:
        x = _normal((T, d), 1.0, seed, _ID_X, torch.bfloat16)
    else:
        assert x.shape == (T, d) and x.dtype == torch.bfloat16
        x = x.detach().cpu().clone()

    if Z > 0 and token_shift > 0.0:
        u = torch.randn(d, generator=_gen(seed, _ID_SHIFT), dtype=torch.float32)
        u = u / u.norm()
        router_w[E:] += token_shift * u

    bias = torch.zeros(E + Z, dtype=torch.float32)
    use_bias = False
    if zipf_s > 0.0:
        ranks = torch.arange(1, E + 1, dtype=torch.float64)
        p = ranks.pow(-zipf_s)
        p = p / p.sum()
        pi = torch.randperm(E, generator=_gen(seed, _ID_PERM))
        bias[:E] = p[pi].log().float()
        use_bias = True

    c = 0.0
    if Z > 0 and zero_fraction is not None:
        use_bias = True
        base = _logits32(x, router_w, bias)
        lo, hi = -40.0, 40.0
        for _ in range(40):
            c = 0.5 * (lo + hi)
            trial = base.clone()
            trial[:, E:] += c
            if _zero_fraction(trial, E, K) < zero_fraction:
                lo = c
            else:
                hi = c
        c = float(np.float32(0.5 * (lo + hi)))
        bias[E:] += c

    bias_or_none = bias if use_bias else None

    redrawn = 0
    if own_x:
        margin = TIE_MARGIN * _MARGIN_SLACK
        for attempt in range(1, 64):
            gaps = _topk_gaps(_logits32(x, router_w, bias_or_none), K)
            bad = torch.nonzero(gaps < margin).flatten()
            if bad.numel() == 0:
                break
            redrawn += int(bad.numel())
            g = _gen(seed, _ID_REDRAW, attempt)
            fresh = torch.randn(bad.numel(), d, generator=g, dtype=torch.float32).to(torch.bfloat16)
            x[bad] = fresh
        else:
            raise RuntimeError("could not reach the top-K tie margin")

    l32 = _logits32(x, router_w, bias_or_none)
    zf = _zero_fraction(l32, E, K) if Z > 0 else 0.0
    return Workload(name=name, T=T, d=d, He=He, E=E, Z=Z, K=K, x=x, router_w=router_w,
                    router_bias=bias_or_none, w_gate_up=w_gate_up, w_down=w_down,
                    zero_bias=c, zero_fraction=zf, redrawn_tokens=redrawn)


QWEN = dict(d=2048, He=768, E=128, Z=64, K=8)


def tiny(seed: int = 0, **over) -> Workload:
    """Tiny layer: T=64, d=256, 8 normal + 4 zero experts of width 128, top-2, ~50 % zero slots."""
    kw = dict(T=64, d=256, He=128, E=8, Z=4, K=2, zero_fraction=0.5)
    kw.update(over)
    return make_layer("tiny", seed=seed, **kw)


def decode(seed: int = 0, T: int = 64, **over) -> Workload:
    """Decode batch on the Qwen3-30B-A3B-shaped layer; per-token zero share spans 0..100 %."""
    kw = dict(QWEN, T=T, zero_fraction=0.5, token_shift=2.5)
    kw.update(over)
    return make_layer("decode", seed=seed, **kw)


def prefill(seed: int = 0, T: int = 8192, **over) -> Workload:
    """Prefill batch with Zipf(1.1)-skewed normal-expert load and ~50 % zero slots."""
    kw = dict(QWEN, T=T, zero_fraction=0.5, zipf_s=1.1)
    kw.update(over)
    return make_layer("prefill", seed=seed, **kw)


def sweep_point(zero_fraction: float, seed: int = 0, T: int = 2048, **over) -> Workload:
    """One point of the zero-fraction sweep; 0.0 means Z=0, the static top-K layer."""
    kw = dict(QWEN, T=T)
    if zero_fraction <= 0.0:
        kw.update(Z=0, zero_fraction=None)
    else:
        kw.update(zero_fraction=zero_fraction)
    kw.update(over)
    return make_layer("sweep_f%02d" % round(100 * zero_fraction), seed=seed, **kw)


def static_reference(wl: Workload) -> Workload:
    """The same layer with the zero experts removed (Z=0): same x, expert weights, normal router
    rows and normal-expert bias.  This is the static top-K layer the paper starts from."""
    bias = None if wl.router_bias is None else wl.router_bias[:wl.E].clone()
    return dataclasses.replace(wl, name=wl.name + "_static", Z=0, router_w=wl.router_w[:wl.E].clone(),
                               router_bias=bias, zero_bias=0.0, zero_fraction=0.0)


def device_expert_weights(E: int, He: int, d: int, seed: int, device):
    """Expert weights ~ N(0, 0.02^2) in bf16 drawn on `device` from a seeded generator of that
    device (same shapes as expert_weights; a different, device-side random stream)."""
    g = torch.Generator(device=device)
    g.manual_seed(seed * 1000 + _ID_GATE_UP)
    w_gate_up = torch.empty(E, 2 * He, d, dtype=torch.bfloat16, device=device)
    w_down = torch.empty(E, d, He, dtype=torch.bfloat16, device=device)
    for w in (w_gate_up, w_down):
        for e in range(E):  # per expert: the fp32 scratch stays small
            w[e] = (torch.randn(w[e].shape, generator=g, dtype=torch.float32, device=device) * 0.02).to(torch.bfloat16)
    return w_gate_up, w_down


def stack_layers(n_layers: int = 48, T: int = 4096, seed: int = 0, **over):
    """Router-side inputs of a stack of Qwen3-30B-A3B-shaped MoE blocks (48 in the paper's models,
    Section 4.2): per layer its own router rows and a zero-expert bias calibrated, on a proxy batch of
    RMS-normalised N(0,1) tokens, to that layer's zero-slot target ~ U[0.3, 0.7].  Expert weights are
    left out (see device_expert_weights).  Returns (list of Workloads, residual stream r0 [T, d])."""
    kw = dict(QWEN)
    kw.update(over)
    fr = stack_layer_fractions(n_layers, seed)
    proxy = rmsnorm_bf16(_normal((T, kw["d"]), 1.0, seed, _ID_X, torch.bfloat16, extra=77))
    layers = [make_layer("stack_l%d" % l, T=T, seed=seed * 100 + l + 1, zero_fraction=fr[l], x=proxy,
                         with_experts=False, **kw) for l in range(n_layers)]
    r0 = _normal((T, kw["d"]), 1.0, seed, _ID_X, torch.bfloat16, extra=78)
    return layers, r0


def stack_layer_fractions(n_layers: int = 48, seed: int = 0):
    """Per-layer zero-slot targets ~ U[0.3, 0.7] for the layer stack."""
    g = _gen(seed, 99)
    return (0.3 + 0.4 * torch.rand(n_layers, generator=g, dtype=torch.float64)).tolist()


def rmsnorm_bf16(r: torch.Tensor, eps: float = 1e-6) -> torch.Tensor:
    """Gain-free RMS normalisation of a bf16 residual stream (glue between stacked layers; not part
    of the paper's method): fp32 math, bf16 result."""
    rf = r.float()
    return (rf * torch.rsqrt(rf.pow(2).mean(dim=-1, keepdim=True) + eps)).to(torch.bfloat16)


def replica_tokens(wl: Workload, rank: int) -> torch.Tensor:
    """A fresh token batch for data-parallel replica `rank` of the same layer: x ~ N(0,1) from a
    rank-derived seed, rows redrawn until the layer's router sees the top-K tie margin."""
    x = _normal((wl.T, wl.d), 1.0, 5000 + rank, _ID_X, torch.bfloat16)
    margin = TIE_MARGIN * _MARGIN_SLACK
    for attempt in range(1, 64):
        gaps = _topk_gaps(_logits32(x, wl.router_w, wl.router_bias), wl.K)
        bad = torch.nonzero(gaps < margin).flatten()
        if bad.numel() == 0:
            return x
        g = _gen(5000 + rank, _ID_REDRAW, attempt)
        x[bad] = torch.randn(bad.numel(), wl.d, generator=g, dtype=torch.float32).to(torch.bfloat16)
    raise RuntimeError("could not reach the top-K tie margin")
