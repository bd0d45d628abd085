"""FLOP model of the MoE branch (Appendix D) and the roofline bounds built on it.

Host-side bookkeeping only; nothing here touches a GPU.
"""
from __future__ import annotations


def moe_flops_orig(n, H, He, N, K):
    """Static layer: F = 6 K n H He + 2 N n H (Appendix D, shared MoE cost decomposition)."""
    return 6 * K * n * H * He + 2 * N * n * H


def moe_flops_zeda(n, H, He, N, NZ, K, r_ze):
    """Zero-expert layer: F = 6 (1 - r_ZE) K n H He + 2 (N + N_Z) n H (Appendix D)."""
    return 6 * (1.0 - r_ze) * K * n * H * He + 2 * (N + NZ) * n * H


def expert_flops_pairs(P, H, He):
    """Expert FLOPs for P surviving (token, normal expert) pairs: three [H x He] products each."""
    return 6 * P * H * He


def router_flops(T, H, n_cand):
    return 2 * n_cand * T * H


def prefill_ratio(l, H, Hattn, gkv, He, N, NZ, K, r_ze):
    """F_ZEDA / F_orig for prefill of l tokens (boxed prefill ratio, Appendix D)."""
    attn = 2 * l * Hattn + 2 * (1 + gkv) * H * Hattn
    return (attn + 3 * (1 - r_ze) * K * H * He + (N + NZ) * H) / (attn + 3 * K * H * He + N * H)


def decode_ratio(l, H, Hattn, gkv, He, N, NZ, K, r_ze):
    """F_ZEDA / F_orig for decoding l tokens with a KV cache (boxed decode ratio, Appendix D)."""
    attn = (l - 1) * Hattn + 2 * (1 + gkv) * H * Hattn
    return (attn + 3 * (1 - r_ze) * K * H * He + (N + NZ) * H) / (attn + 3 * K * H * He + N * H)


def target_zero_ratio(N, NZ, w):
    """Equilibrium zero-expert activation ratio of the group loss: N_Z w / (N + N_Z w) (Section 2.2)."""
    return NZ * w / (N + NZ * w)


def layer_algorithmic_bytes(T, d, He, n_cand, U):
    """Bytes the method itself must move for one layer call: the bf16 weights of the U distinct
    active experts, x read, y written (bf16) and the fp32 router rows."""
    return U * 3 * d * He * 2 + 2 * T * d * 2 + n_cand * d * 4


def layer_roofline_seconds(T, d, He, n_cand, P, U, peak_flops, peak_bytes_per_s):
    """Slower of active-expert FLOPs at the tensor peak and algorithmic bytes at the HBM peak."""
    t_flop = expert_flops_pairs(P, d, He) / peak_flops
    t_mem = layer_algorithmic_bytes(T, d, He, n_cand, U) / peak_bytes_per_s
    return max(t_flop, t_mem), t_flop, t_mem
