"""ctypes access to the CPU oracle (``zeda_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the CUDA library or its Python binding.
Arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zeda_oracle.c")
_LIB = os.path.join(_HERE, "libzeda_oracle.so")

GATE_TOPK_NORM, GATE_SOFTMAX_RAW, GATE_RENORM_REAL = 0, 1, 2
EXPERT_ZERO, EXPERT_COPY = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over tokens only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.zeda_oracle_num_threads.restype = ctypes.c_int
        _lib.zeda_oracle_compact.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 tensors are passed as uint16 bit patterns"
    return a


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def num_threads() -> int:
    return int(_load().zeda_oracle_num_threads())


def logits(x_bits, router_w, router_bias=None):
    """fp32 router logits [T, N+N_Z] (fp64 accumulation, one rounding)."""
    x_bits = _u16(x_bits)
    router_w = _f32(router_w)
    router_bias = _f32(router_bias)
    T, d = x_bits.shape
    n = router_w.shape[0]
    assert router_w.shape[1] == d
    out = np.empty((T, n), dtype=np.float32)
    _load().zeda_oracle_logits(_p(x_bits), _p(router_w), _p(router_bias),
                               ctypes.c_int(T), ctypes.c_int(d), ctypes.c_int(n), _p(out))
    return out


def route(logits_f32, n_real, n_zero, K, gate_mode=GATE_TOPK_NORM):
    """Top-K indices [T,K] int32 and routing weights [T,K] fp64."""
    l = _f32(logits_f32)
    T, n = l.shape
    assert n == n_real + n_zero and 1 <= K <= n
    idx = np.empty((T, K), dtype=np.int32)
    w = np.empty((T, K), dtype=np.float64)
    _load().zeda_oracle_route(_p(l), ctypes.c_int(T), ctypes.c_int(n_real), ctypes.c_int(n_zero),
                              ctypes.c_int(K), ctypes.c_int(gate_mode), _p(idx), _p(w))
    return idx, w


def compact(topk_idx, n_real):
    """counts [E], offsets [E+1], perm [P] (source slot t*K+k), P."""
    idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    T, K = idx.shape
    counts = np.empty(n_real, dtype=np.int32)
    offsets = np.empty(n_real + 1, dtype=np.int32)
    perm = np.empty(T * K, dtype=np.int32)
    P = _load().zeda_oracle_compact(_p(idx), ctypes.c_int(T), ctypes.c_int(n_real), ctypes.c_int(K),
                                    _p(counts), _p(offsets), _p(perm))
    return counts, offsets, perm[:P].copy(), int(P)


def expert(x_row_bits, w_gate_up_e_bits, w_down_e_bits):
    """One expert on one token: fp64 vector [d]."""
    x_row_bits = _u16(x_row_bits)
    wgu = _u16(w_gate_up_e_bits)
    wd = _u16(w_down_e_bits)
    d = x_row_bits.shape[0]
    He = wgu.shape[0] // 2
    assert wgu.shape == (2 * He, d) and wd.shape == (d, He)
    o = np.empty(d, dtype=np.float64)
    _load().zeda_oracle_expert(_p(x_row_bits), _p(wgu), _p(wd), ctypes.c_int(d), ctypes.c_int(He), _p(o))
    return o


def forward(x_bits, router_w, router_bias, w_gate_up_bits, w_down_bits, n_real, n_zero, K,
            gate_mode=GATE_TOPK_NORM, expert_kind=EXPERT_ZERO, token_ids=None, want_y=True):
    """Layer forward for all tokens or for ``token_ids``.

    Returns (y fp64 [n,d] or None, idx int32 [n,K], w fp64 [n,K]).
    """
    x_bits = _u16(x_bits)
    router_w = _f32(router_w)
    router_bias = _f32(router_bias)
    wgu = _u16(w_gate_up_bits)
    wd = _u16(w_down_bits)
    T, d = x_bits.shape
    He = wd.shape[2] if n_real > 0 else 0
    if n_real > 0:
        assert wgu.shape == (n_real, 2 * He, d) and wd.shape == (n_real, d, He)
    assert router_w.shape == (n_real + n_zero, d)
    if token_ids is None:
        ids, n = None, T
    else:
        ids = np.ascontiguousarray(token_ids, dtype=np.int32)
        n = ids.shape[0]
        assert n == 0 or (ids.min() >= 0 and ids.max() < T)
    y = np.empty((n, d), dtype=np.float64) if want_y else None
    idx = np.empty((n, K), dtype=np.int32)
    w = np.empty((n, K), dtype=np.float64)
    _load().zeda_oracle_forward(_p(x_bits), ctypes.c_int(d), ctypes.c_int(He), ctypes.c_int(n_real),
                                ctypes.c_int(n_zero), ctypes.c_int(K), ctypes.c_int(gate_mode),
                                ctypes.c_int(expert_kind), _p(router_w), _p(router_bias), _p(wgu), _p(wd),
                                _p(ids), ctypes.c_int(n), _p(y), _p(idx), _p(w))
    return y, idx, w


def stats(logits_f32, topk_idx, n_real, n_zero, alpha=1.0, group_w=1.0):
    """Eq. 4-6 forward values: dict with f, P, r_ze, L_A, L_GA."""
    l = _f32(logits_f32)
    idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    T, K = idx.shape
    n = n_real + n_zero
    f = np.empty(n, dtype=np.float64)
    pm = np.empty(n, dtype=np.float64)
    out = np.empty(3, dtype=np.float64)
    _load().zeda_oracle_stats(_p(l), _p(idx), ctypes.c_int(T), ctypes.c_int(n_real), ctypes.c_int(n_zero),
                              ctypes.c_int(K), ctypes.c_double(alpha), ctypes.c_double(group_w),
                              _p(f), _p(pm), _p(out))
    return {"f": f, "P": pm, "r_ze": float(out[0]), "L_A": float(out[1]), "L_GA": float(out[2])}


def token_zero_share(topk_idx, n_real):
    """Per-token share of the K slots on zero experts, fp64 [T]."""
    idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    T, K = idx.shape
    out = np.empty(T, dtype=np.float64)
    _load().zeda_oracle_token_zero_share(_p(idx), ctypes.c_int(T), ctypes.c_int(n_real), ctypes.c_int(K), _p(out))
    return out


def _bf16_to_f64(bits):
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _f64_to_bf16_bits(v):
    """Round-to-nearest-even of float64 values to bf16 bit patterns (via the exact float32 when the
    value is one, else through the integer significand; inputs here are sums of two bf16 values,
    which float64 holds exactly)."""
    v = np.asarray(v, dtype=np.float64)
    f = v.astype(np.float32)  # exact or correctly rounded once; see the callers' note
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) >> 16
    return r.astype(np.uint16)


def residual_rmsnorm(r_bits, y_bits=None, eps=1e-6):
    """Glue between stacked MoE blocks (a device of the layer-stack workload, not part of the
    paper's layer): r' = bf16(r + y) element by element (y may be None: r' = r), then the gain-free
    RMS normalisation h = r' / sqrt(mean(r'^2) + eps) per row, in fp64.

    Returns (r' as uint16 bit patterns, h as float64).  The sum of two bf16 values is exact in
    float32 whenever their exponents differ by at most 16, and rounds back to the larger operand
    otherwise, so rounding it through float32 and then to bf16 equals rounding the exact sum."""
    r = _bf16_to_f64(r_bits)
    if y_bits is not None:
        r_new_bits = _f64_to_bf16_bits(r + _bf16_to_f64(y_bits))
    else:
        r_new_bits = np.ascontiguousarray(r_bits, dtype=np.uint16).copy()
    rn = _bf16_to_f64(r_new_bits)
    ms = np.mean(rn * rn, axis=-1, keepdims=True)
    return r_new_bits, rn / np.sqrt(ms + eps)
