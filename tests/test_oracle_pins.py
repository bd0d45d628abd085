"""Pins for the CPU oracle: each test checks it against something fixed by the paper or by plain
mathematics (brute force, closed forms, invariants, library routines on special cases), never
against the CUDA path."""
import itertools
import os

import numpy as np
import pytest
import torch
from scipy.special import expit, softmax

import oracle
from paper_2605_18643_b200 import flops, inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(a: np.ndarray) -> np.ndarray:
    return inputs.bits(torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def small_layer(seed, T=10, d=16, He=12, E=5, Z=3, K=3, bias=True):
    rng = np.random.default_rng(seed)
    x = bf16_bits(rng.standard_normal((T, d)))
    rw = rng.standard_normal((E + Z, d)).astype(np.float32) * 0.5
    rb = (rng.standard_normal(E + Z).astype(np.float32) * 0.3) if bias else None
    wgu = bf16_bits(rng.standard_normal((E, 2 * He, d)) * 0.3)
    wd = bf16_bits(rng.standard_normal((E, d, He)) * 0.3)
    return x, rw, rb, wgu, wd, dict(n_real=E, n_zero=Z, K=K)


def dense_layer(x, rw, rb, wgu, wd, n_real, n_zero, K, idx, w):
    """Second, structurally different formulation: every normal expert applied to every token
    with library matrix products, then a 0/1 selection mask times the weights (Eq. 1)."""
    X = bits_to_f64(x)
    E = n_real
    He = wd.shape[2]
    Wg = bits_to_f64(wgu)[:, :He, :]
    Wu = bits_to_f64(wgu)[:, He:, :]
    Wd = bits_to_f64(wd)
    A = np.einsum("tc,ejc->tej", X, Wg)
    U = np.einsum("tc,ejc->tej", X, Wu)
    Hm = A * expit(A) * U
    O = np.einsum("tej,ecj->tec", Hm, Wd)                   # [T, E, d]
    G = np.zeros((X.shape[0], E + n_zero))
    np.put_along_axis(G, idx.astype(np.int64), w, axis=1)    # gate of each selected candidate
    return np.einsum("te,tec->tc", G[:, :E], O)


# ---------------------------------------------------------------- logits

def test_logits_match_library_matmul():
    x, rw, rb, *_ = small_layer(1, T=7, d=33)
    got = oracle.logits(x, rw, rb)
    want = (bits_to_f64(x) @ rw.astype(np.float64).T + rb.astype(np.float64)).astype(np.float32)
    assert got.dtype == np.float32
    # one fp32 rounding of an fp64 sum: at most one ulp apart from the library product
    assert np.all(np.abs(got.astype(np.float64) - want) <= np.spacing(np.abs(want)).astype(np.float64))
    got_nb = oracle.logits(x, rw, None)
    assert np.allclose(got_nb, bits_to_f64(x) @ rw.astype(np.float64).T, rtol=1e-6, atol=1e-7)


def test_logits_hand_example():
    # x = [1, 2, -0.5], rows [1,0,2] and [0.5,0.5,0.5], bias [0.25,-1]: exact in binary
    x = bf16_bits(np.array([[1.0, 2.0, -0.5]]))
    rw = np.array([[1.0, 0.0, 2.0], [0.5, 0.5, 0.5]], dtype=np.float32)
    rb = np.array([0.25, -1.0], dtype=np.float32)
    assert oracle.logits(x, rw, rb).tolist() == [[0.25, 0.25]]


# ---------------------------------------------------------------- top-K

@pytest.mark.parametrize("n_real,n_zero,K", [(3, 1, 1), (4, 2, 2), (5, 3, 3), (8, 4, 3), (6, 0, 2)])
def test_topk_brute_force(n_real, n_zero, K):
    rng = np.random.default_rng(100 + n_real * 10 + K)
    n = n_real + n_zero
    l = rng.standard_normal((40, n)).astype(np.float32)
    idx, _ = oracle.route(l, n_real, n_zero, K)
    for t in range(l.shape[0]):
        best = max(itertools.combinations(range(n), K), key=lambda s: float(np.sum(l[t, list(s)].astype(np.float64))))
        assert set(idx[t].tolist()) == set(best)
        assert len(set(idx[t].tolist())) == K
        sel = l[t, idx[t]]
        assert np.all(sel[:-1] >= sel[1:])                   # slot order: descending logit
        rest = np.delete(l[t], idx[t])
        assert rest.size == 0 or rest.max() <= sel.min()


def test_topk_ties_go_to_lower_index():
    l = np.array([[0.5, 2.0, 2.0, 0.5, 2.0, -1.0]], dtype=np.float32)
    idx, _ = oracle.route(l, 4, 2, 4)
    assert idx.tolist() == [[1, 2, 4, 0]]
    idx, _ = oracle.route(np.zeros((1, 5), dtype=np.float32), 3, 2, 3)
    assert idx.tolist() == [[0, 1, 2]]


# ---------------------------------------------------------------- routing weights

def test_gate_weight_invariants():
    rng = np.random.default_rng(7)
    n_real, n_zero, K = 6, 4, 4
    l = (rng.standard_normal((50, 10)) * 2).astype(np.float32)
    idx, w0 = oracle.route(l, n_real, n_zero, K, oracle.GATE_TOPK_NORM)
    idx1, w1 = oracle.route(l, n_real, n_zero, K, oracle.GATE_SOFTMAX_RAW)
    idx2, w2 = oracle.route(l, n_real, n_zero, K, oracle.GATE_RENORM_REAL)
    assert np.array_equal(idx, idx1) and np.array_equal(idx, idx2)   # selection ignores the mode
    p = softmax(l.astype(np.float64), axis=1)
    psel = np.take_along_axis(p, idx.astype(np.int64), axis=1)
    real = idx < n_real
    # mode 1: the full-softmax entries themselves
    assert np.allclose(w1, psel, rtol=1e-13, atol=0)
    assert np.all(w1.sum(1) <= 1 + 1e-12)
    # mode 0: normalised over the K selected slots, zero slots included in the sum
    assert np.allclose(w0.sum(1), 1.0, rtol=1e-13)
    assert np.allclose(w0, psel / psel.sum(1, keepdims=True), rtol=1e-13)
    zero_mass = np.where(real, 0.0, w0).sum(1)
    assert np.allclose(np.where(real, w0, 0.0).sum(1), 1.0 - zero_mass, rtol=1e-12)
    assert np.any(zero_mass > 0.05)                         # surviving weights are NOT rescaled
    # both modes keep the ratio exp(l_a - l_b)
    la = np.take_along_axis(l.astype(np.float64), idx.astype(np.int64), axis=1)
    for wm in (w0, w1):
        assert np.allclose(wm[:, 0] / wm[:, -1], np.exp(la[:, 0] - la[:, -1]), rtol=1e-12)
    # mode 2 (Eq. 7): sums to one over the selected normal experts, zero slots carry nothing
    has_real = real.any(1)
    assert np.allclose(np.where(real, w2, 0.0).sum(1)[has_real], 1.0, rtol=1e-13)
    assert np.all(w2[~real] == 0.0)
    assert np.allclose(w2[real], (w0 / np.where(real, w0, 0.0).sum(1, keepdims=True))[real], rtol=1e-12)


def test_softmax_is_shift_invariant_and_stable():
    l = np.array([[1000.0, 999.0, 998.0, -1000.0]], dtype=np.float32)
    _, w = oracle.route(l, 3, 1, 2, oracle.GATE_SOFTMAX_RAW)
    want = softmax(np.array([0.0, -1.0, -2.0, -2000.0]))[:2]
    assert np.allclose(w[0], want, rtol=1e-13)


# ---------------------------------------------------------------- compaction / counting sort

def test_compact_matches_library_stable_sort():
    rng = np.random.default_rng(3)
    T, K, n_real, n_zero = 37, 3, 6, 5
    l = rng.standard_normal((T, n_real + n_zero)).astype(np.float32)
    idx, _ = oracle.route(l, n_real, n_zero, K)
    counts, offsets, perm, P = oracle.compact(idx, n_real)
    flat = idx.reshape(-1)
    real_slots = np.nonzero(flat < n_real)[0]
    want = real_slots[np.argsort(flat[real_slots], kind="stable")]
    assert P == real_slots.size == T * K - int((flat >= n_real).sum())
    assert np.array_equal(perm, want)
    assert np.array_equal(counts, np.bincount(flat[real_slots], minlength=n_real))
    assert offsets[0] == 0 and np.array_equal(np.diff(offsets), counts) and offsets[-1] == P
    e_sorted = flat[perm]
    assert np.all(np.diff(e_sorted) >= 0)
    for e in range(n_real):
        seg = perm[offsets[e]:offsets[e + 1]]
        assert np.all(np.diff(seg) > 0) and np.all(flat[seg] == e)


def test_compact_degenerate_cases():
    # every slot on a zero expert: nothing survives
    idx = np.full((5, 2), 4, dtype=np.int32)
    counts, offsets, perm, P = oracle.compact(idx, 3)
    assert P == 0 and perm.size == 0 and counts.tolist() == [0, 0, 0] and offsets.tolist() == [0, 0, 0, 0]
    # every token on one expert
    idx = np.tile(np.array([[1, 3]], dtype=np.int32), (4, 1))
    counts, offsets, perm, P = oracle.compact(idx, 3)
    assert P == 4 and counts.tolist() == [0, 4, 0] and perm.tolist() == [0, 2, 4, 6]


# ---------------------------------------------------------------- expert math

def test_single_expert_is_a_plain_swiglu_mlp():
    # K=1, Z=0, N=1: the layer is one SwiGLU MLP with routing weight exactly 1
    x, rw, rb, wgu, wd, _ = small_layer(11, T=6, d=24, He=20, E=1, Z=0, K=1)
    y, idx, w = oracle.forward(x, rw, rb, wgu, wd, 1, 0, 1)
    assert np.all(idx == 0) and np.all(w == 1.0)
    X = bits_to_f64(x)
    He = 20
    Wg, Wu, Wd = bits_to_f64(wgu)[0, :He], bits_to_f64(wgu)[0, He:], bits_to_f64(wd)[0]
    a = X @ Wg.T
    want = ((a * expit(a)) * (X @ Wu.T)) @ Wd.T
    assert np.allclose(y, want, rtol=1e-12, atol=1e-14)
    o = oracle.expert(x[2], wgu[0], wd[0])
    assert np.allclose(o, want[2], rtol=1e-12, atol=1e-14)


def test_expert_hand_example():
    # d=2, He=1: gate row [1,0], up row [0,1], down column [2,-1]; x=[0,3] -> silu(0)=0 -> 0;
    # x=[ln-free case] x=[1,3]: a=1, u=3, h=3/(1+e^-1), o=[2h,-h]
    wgu = bf16_bits(np.array([[[1.0, 0.0], [0.0, 1.0]]]))
    wd = bf16_bits(np.array([[[2.0], [-1.0]]]))
    assert oracle.expert(bf16_bits(np.array([0.0, 3.0])), wgu[0], wd[0]).tolist() == [0.0, 0.0]
    h = 3.0 / (1.0 + np.exp(-1.0))
    o = oracle.expert(bf16_bits(np.array([1.0, 3.0])), wgu[0], wd[0])
    assert np.allclose(o, [2 * h, -h], rtol=1e-15)


@pytest.mark.parametrize("mode", [oracle.GATE_TOPK_NORM, oracle.GATE_SOFTMAX_RAW, oracle.GATE_RENORM_REAL])
def test_dense_mask_formulation(mode):
    x, rw, rb, wgu, wd, cfg = small_layer(5)
    y, idx, w = oracle.forward(x, rw, rb, wgu, wd, gate_mode=mode, **cfg)
    want = dense_layer(x, rw, rb, wgu, wd, idx=idx, w=w, **cfg)
    assert np.allclose(y, want, rtol=1e-12, atol=1e-13)
    # and the routing inside forward() is the routing of the stand-alone calls
    idx_s, w_s = oracle.route(oracle.logits(x, rw, rb), cfg["n_real"], cfg["n_zero"], cfg["K"], mode)
    assert np.array_equal(idx, idx_s) and np.array_equal(w, w_s)


def test_token_subset_equals_full_run():
    x, rw, rb, wgu, wd, cfg = small_layer(6)
    y, idx, w = oracle.forward(x, rw, rb, wgu, wd, **cfg)
    ids = np.array([7, 0, 3], dtype=np.int32)
    ys, idxs, ws = oracle.forward(x, rw, rb, wgu, wd, token_ids=ids, **cfg)
    assert np.array_equal(ys, y[ids]) and np.array_equal(idxs, idx[ids]) and np.array_equal(ws, w[ids])


# ---------------------------------------------------------------- zero-expert semantics (Section 2.1)

def static_topk_moe(x, rw, rb, wgu, wd, K):
    """Independent static top-K MoE, y = sum_{i in S(h)} g_i(h) E_i(h), written with numpy only."""
    X = bits_to_f64(x)
    l = (X @ rw.astype(np.float64).T + (0 if rb is None else rb.astype(np.float64))).astype(np.float32)
    order = np.argsort(-l.astype(np.float64), axis=1, kind="stable")[:, :K]
    p = softmax(l.astype(np.float64), axis=1)
    He = wd.shape[2]
    y = np.zeros((X.shape[0], X.shape[1]))
    for t in range(X.shape[0]):
        g = p[t, order[t]] / p[t, order[t]].sum()
        for k, e in enumerate(order[t]):
            a = bits_to_f64(wgu[e, :He]) @ X[t]
            u = bits_to_f64(wgu[e, He:]) @ X[t]
            y[t] += g[k] * (bits_to_f64(wd[e]) @ (a * expit(a) * u))
    return y, order


def test_z0_reduces_to_static_moe():
    x, rw, rb, wgu, wd, cfg = small_layer(8, Z=0)
    y, idx, w = oracle.forward(x, rw, rb, wgu, wd, **cfg)
    want, order = static_topk_moe(x, rw, rb, wgu, wd, cfg["K"])
    assert np.array_equal(idx, order.astype(np.int32))
    assert np.allclose(y, want, rtol=1e-12, atol=1e-14)


def test_never_selected_zero_experts_change_nothing():
    x, rw, rb, wgu, wd, cfg = small_layer(9, Z=0)
    y0, idx0, w0 = oracle.forward(x, rw, rb, wgu, wd, **cfg)
    rng = np.random.default_rng(0)
    rw2 = np.concatenate([rw, rng.standard_normal((4, rw.shape[1])).astype(np.float32)])
    rb2 = np.concatenate([rb, np.full(4, -1e30, dtype=np.float32)])
    y1, idx1, w1 = oracle.forward(x, rw2, rb2, wgu, wd, n_real=cfg["n_real"], n_zero=4, K=cfg["K"])
    assert np.array_equal(idx0, idx1) and np.array_equal(w0, w1) and np.array_equal(y0, y1)


def test_all_zero_token_outputs_exact_zero():
    x, rw, rb, wgu, wd, cfg = small_layer(10)
    rb = rb.copy()
    rb[cfg["n_real"]:] += 100.0          # zero experts win every slot
    y, idx, w = oracle.forward(x, rw, rb, wgu, wd, **cfg)
    assert np.all(idx >= cfg["n_real"])
    assert np.all(y == 0.0) and not np.any(np.signbit(y))
    counts, offsets, perm, P = oracle.compact(idx, cfg["n_real"])
    assert P == 0


def test_zero_slots_remove_exactly_their_expert_terms():
    # Eq. 1 against the same token routed without zero experts: with zero slots the output is the
    # static sum restricted to the surviving experts, weights untouched.
    x, rw, rb, wgu, wd, cfg = small_layer(12)
    y, idx, w = oracle.forward(x, rw, rb, wgu, wd, gate_mode=oracle.GATE_SOFTMAX_RAW, **cfg)
    E = cfg["n_real"]
    for t in range(x.shape[0]):
        acc = np.zeros(x.shape[1])
        for k in range(cfg["K"]):
            if idx[t, k] < E:
                acc += w[t, k] * oracle.expert(x[t], wgu[idx[t, k]], wd[idx[t, k]])
        assert np.allclose(y[t], acc, rtol=1e-13, atol=1e-15)


def test_renorm_identity_eq7():
    x, rw, rb, wgu, wd, cfg = small_layer(13)
    y, idx, w = oracle.forward(x, rw, rb, wgu, wd, gate_mode=oracle.GATE_TOPK_NORM, **cfg)
    yr, idxr, wr = oracle.forward(x, rw, rb, wgu, wd, gate_mode=oracle.GATE_RENORM_REAL, **cfg)
    s = np.where(idx < cfg["n_real"], w, 0.0).sum(1, keepdims=True)
    assert np.any((s > 0) & (s < 0.99))
    assert np.allclose(yr * s, y, rtol=1e-12, atol=1e-15)


def test_copy_expert_identity_appendix_b():
    x, rw, rb, wgu, wd, cfg = small_layer(14)
    y, idx, w = oracle.forward(x, rw, rb, wgu, wd, **cfg)
    yc, _, _ = oracle.forward(x, rw, rb, wgu, wd, expert_kind=oracle.EXPERT_COPY, **cfg)
    zero_mass = np.where(idx >= cfg["n_real"], w, 0.0).sum(1, keepdims=True)
    assert np.any(zero_mass > 0)
    assert np.allclose(yc - y, zero_mass * bits_to_f64(x), rtol=1e-10, atol=1e-13)


# ---------------------------------------------------------------- statistics (Eq. 4-6)

def test_stats_closed_forms():
    rng = np.random.default_rng(21)
    n_real, n_zero, K, T = 6, 3, 3, 200
    l = rng.standard_normal((T, n_real + n_zero)).astype(np.float32)
    idx, _ = oracle.route(l, n_real, n_zero, K)
    s = oracle.stats(l, idx, n_real, n_zero, alpha=0.1, group_w=2.0)
    p = softmax(l.astype(np.float64), axis=1)
    f = np.array([(idx == i).any(1).mean() for i in range(n_real + n_zero)])
    assert np.allclose(s["f"], f) and np.allclose(s["P"], p.mean(0), rtol=1e-12)
    assert np.isclose(s["f"].sum(), K) and np.isclose(s["P"].sum(), 1.0)
    assert np.isclose(s["r_ze"], (idx >= n_real).mean())
    assert np.isclose(s["L_A"], 0.1 * (n_real + n_zero) / K * np.sum(f * p.mean(0)))
    fE, fZ, pE, pZ = f[:n_real].sum(), f[n_real:].sum(), p.mean(0)[:n_real].sum(), p.mean(0)[n_real:].sum()
    assert np.isclose(s["L_GA"], 0.1 * (n_real + n_zero * 2.0) / K * (fE * pE / n_real + fZ * pZ / (n_zero * 2.0)))
    # perfectly uniform routing probabilities and loads: L_A = alpha (Switch/GShard fixed point)
    lu = np.zeros((9, 9), dtype=np.float32)
    idxu = np.array([[(t + k) % 9 for k in range(3)] for t in range(9)], dtype=np.int32)
    su = oracle.stats(lu, idxu, 6, 3, alpha=0.25, group_w=1.0)
    assert np.isclose(su["L_A"], 0.25) and np.isclose(su["L_GA"], 0.25)


# ---------------------------------------------------------------- FLOP model (Appendix D)

def test_flop_model_reproduces_printed_speedups():
    q = dict(H=2048, Hattn=4096, gkv=1 / 8, He=768, N=128, NZ=64, K=8, r_ze=0.5)
    rows = [r.split() for r in open(os.path.join(GOLDEN, "flop_speedup_table.txt")) if not r.startswith("#")]
    assert len(rows) == 8
    for l, pre, dec in rows:
        assert abs(1 / flops.prefill_ratio(int(l), **q) - float(pre)) < 6e-4
        assert abs(1 / flops.decode_ratio(int(l), **q) - float(dec)) < 6e-4


def test_flop_closed_forms():
    assert flops.expert_flops_pairs(1, 2048, 768) == 9_437_184
    assert flops.moe_flops_orig(1, 2048, 768, 128, 8) == 76_021_760
    assert flops.moe_flops_zeda(1, 2048, 768, 128, 64, 8, 0.5) == 38_535_168
    assert flops.moe_flops_zeda(5, 2048, 768, 128, 0, 8, 0.0) == flops.moe_flops_orig(5, 2048, 768, 128, 8)
    assert flops.router_flops(8192, 2048, 192) == 2 * 192 * 8192 * 2048
    assert flops.target_zero_ratio(128, 64, 2.0) == 0.5


def test_pair_count_matches_flop_model():
    wl = inputs.tiny()
    l = oracle.logits(inputs.bits(wl.x), wl.router_w.numpy(), wl.router_bias.numpy())
    idx, _ = oracle.route(l, wl.E, wl.Z, wl.K)
    _, _, _, P = oracle.compact(idx, wl.E)
    r = oracle.stats(l, idx, wl.E, wl.Z)["r_ze"]
    assert P == round(wl.T * wl.K * (1 - r))
    want = flops.moe_flops_zeda(wl.T, wl.d, wl.He, wl.E, wl.Z, wl.K, r)
    assert np.isclose(flops.expert_flops_pairs(P, wl.d, wl.He) + flops.router_flops(wl.T, wl.d, wl.E + wl.Z), want)


# ---------------------------------------------------------------------------------- layer-stack glue

def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def test_residual_rmsnorm_closed_forms():
    # a constant row c normalises to c / sqrt(c^2 + eps); the mean square of h is ms / (ms + eps)
    import torch as _t
    for c in (0.5, -2.0, 0.0):
        r = _t.full((3, 128), c, dtype=_t.bfloat16)
        nb, h = oracle.residual_rmsnorm(_bits(r), None, eps=1e-6)
        assert np.array_equal(nb, _bits(r))
        assert np.allclose(h, c / np.sqrt(c * c + 1e-6), rtol=0, atol=1e-15)
    g = _t.Generator().manual_seed(3)
    r = (_t.randn(7, 192, generator=g) * 4).to(_t.bfloat16)
    _, h = oracle.residual_rmsnorm(_bits(r), None, eps=1e-6)
    rd = r.double().numpy()
    ms = (rd * rd).mean(axis=1)
    assert np.allclose((h * h).mean(axis=1), ms / (ms + 1e-6), rtol=1e-13)
    # scale invariance up to eps: normalising 8 r gives the same direction (power-of-two scale keeps bf16 exact)
    _, h8 = oracle.residual_rmsnorm(_bits((r.float() * 8).to(_t.bfloat16)), None, eps=0.0)
    _, h1 = oracle.residual_rmsnorm(_bits(r), None, eps=0.0)
    assert np.allclose(h8, h1, rtol=1e-13)


def test_residual_add_is_the_correctly_rounded_sum():
    # brute force over bf16 operands against exact rational arithmetic: the stored residual is the
    # bf16 nearest to r + y (ties to even), including pairs whose exponents are far apart
    import fractions
    import torch as _t
    vals = _t.tensor([1.0, 1.0078125, -1.0078125, 3.0e-5, 255.0, 0.00390625, -0.0078125, 1.5, 6.1e-5, 128.5, 2.0 ** -20, 1.00390625],
                     dtype=_t.float32).to(_t.bfloat16)
    a = vals.repeat_interleave(len(vals)).view(1, -1)
    b = vals.repeat(len(vals)).view(1, -1)
    pad = 64 - a.shape[1] % 64
    a = _t.cat([a, _t.zeros(1, pad, dtype=_t.bfloat16)], 1)
    b = _t.cat([b, _t.zeros(1, pad, dtype=_t.bfloat16)], 1)
    nb, _ = oracle.residual_rmsnorm(_bits(a), _bits(b))
    got = (nb.astype(np.uint32) << 16).view(np.float32).astype(np.float64)[0]
    for i in range(len(vals) ** 2):
        exact = fractions.Fraction(float(a[0, i])) + fractions.Fraction(float(b[0, i]))
        g = fractions.Fraction(float(got[i]))
        if exact == 0:
            assert g == 0
            continue
        # g is a bf16 value within half a bf16 ulp of the exact sum
        e = np.floor(np.log2(abs(float(exact))))
        ulp = fractions.Fraction(2) ** int(e - 7)
        assert abs(g - exact) <= ulp / 2, (float(a[0, i]), float(b[0, i]), float(g))


def test_token_zero_share_counts_slots_and_averages_to_r_ze():
    # Section 2.2 / 4.1: per token, the share of its K slots on zero experts; its batch mean is r_ZE
    rng = np.random.default_rng(3)
    E, Z, K, T = 6, 5, 4, 300
    l = rng.standard_normal((T, E + Z)).astype(np.float32)
    l[0, E:] += 100.0          # token 0: every slot on a zero expert
    l[1, :E] += 100.0          # token 1: none
    idx, _ = oracle.route(l, E, Z, K)
    r = oracle.token_zero_share(idx, E)
    assert r[0] == 1.0 and r[1] == 0.0
    assert set(np.unique(r * K)).issubset(set(range(K + 1)))             # multiples of 1/K
    brute = np.array([sum(1 for i in row if i >= E) / K for row in idx])
    assert np.array_equal(r, brute)
    s = oracle.stats(l, idx, E, Z)
    assert abs(r.mean() - s["r_ze"]) < 1e-15
    assert np.array_equal(oracle.token_zero_share(np.zeros((3, 2), dtype=np.int32), 1), np.zeros(3))   # Z = 0 layer
