"""The synthetic-workload recipe: determinism, tie margin, zero-slot fraction, load skew."""
import numpy as np
import torch

import oracle
from paper_2605_18643_b200 import inputs


def _route(wl):
    b = None if wl.router_bias is None else wl.router_bias.numpy()
    l = oracle.logits(inputs.bits(wl.x), wl.router_w.numpy(), b)
    idx, w = oracle.route(l, wl.E, wl.Z, wl.K)
    return l, idx, w


def test_tiny_is_deterministic_and_calibrated():
    a, b = inputs.tiny(), inputs.tiny()
    assert torch.equal(a.x, b.x) and torch.equal(a.router_w, b.router_w) and torch.equal(a.w_down, b.w_down)
    assert a.x.dtype == torch.bfloat16 and a.router_w.dtype == torch.float32
    assert (a.T, a.d, a.He, a.E, a.Z, a.K) == (64, 256, 128, 8, 4, 2)
    l, idx, _ = _route(a)
    assert abs(float((idx >= a.E).mean()) - 0.5) < 0.05
    assert abs(float(a.w_gate_up.float().std()) - 0.02) < 0.002


def test_tie_margin_on_oracle_logits():
    for wl in (inputs.tiny(), inputs.tiny(seed=3), inputs.make_layer("m", 256, 128, 32, 16, 8, 4, seed=5)):
        l, idx, _ = _route(wl)
        top = -np.sort(-l.astype(np.float64), axis=1)[:, :wl.K + 1]
        assert np.min(top[:, :-1] - top[:, 1:]) >= inputs.TIE_MARGIN


def test_token_shift_spreads_per_token_zero_share():
    wl = inputs.make_layer("d", 256, 256, 32, 32, 16, 8, seed=1, zero_fraction=0.5, token_shift=2.5)
    _, idx, _ = _route(wl)
    share = (idx >= wl.E).mean(1)
    assert abs(share.mean() - 0.5) < 0.03
    assert share.min() == 0.0 and share.max() == 1.0


def test_zipf_prior_skews_expert_load():
    wl = inputs.make_layer("p", 2048, 128, 32, 32, 16, 4, seed=2, zero_fraction=0.5, zipf_s=1.1)
    _, idx, _ = _route(wl)
    counts, _, _, P = oracle.compact(idx, wl.E)
    assert abs(P / (wl.T * wl.K) - 0.5) < 0.02
    assert counts.max() > 6 * max(1, counts.min())


def test_static_reference_drops_zero_rows():
    wl = inputs.tiny()
    st = inputs.static_reference(wl)
    assert st.Z == 0 and st.router_w.shape[0] == wl.E and torch.equal(st.x, wl.x)
    assert torch.equal(st.router_w, wl.router_w[:wl.E])
