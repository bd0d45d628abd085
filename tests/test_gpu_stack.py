"""GPU parity of the layer-stack glue (residual update + RMS normalisation) and of a small stack of
zero-expert MoE blocks.  Per layer the oracle is fed the GPU's own layer input: once two inputs
differ in their last bit a routing decision may differ, so an end-to-end comparison at depth would
test the inputs, not the layer."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_18643_b200 import inputs

pytestmark = pytest.mark.gpu

REL_L2, MAX_ABS_RMS = 1e-2, 5e-2


@pytest.fixture(scope="module")
def zeda():
    from paper_2605_18643_b200 import zeda as z
    return z


def _bits(t):
    return inputs.bits(t.cpu())


def _ulp_bf16(v):
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(v), 1e-30))) - 7)


@pytest.mark.parametrize("T,d", [(1, 64), (37, 256), (300, 2048), (5, 8192)])
def test_residual_rmsnorm_matches_the_oracle(zeda, T, d):
    g = torch.Generator().manual_seed(11)
    r = (torch.randn(T, d, generator=g) * 3).to(torch.bfloat16)
    y = torch.randn(T, d, generator=g).to(torch.bfloat16)
    y[0, : d // 2] = (r[0, : d // 2].float() * 2.0 ** -12).to(torch.bfloat16)  # operands far apart in exponent
    dev = torch.device("cuda:0")
    for with_y in (True, False):
        rg = r.to(dev).clone()
        h = zeda.residual_rmsnorm(rg, y.to(dev) if with_y else None)
        torch.cuda.synchronize()
        r_ref, h_ref = oracle.residual_rmsnorm(_bits(r), _bits(y) if with_y else None)
        assert np.array_equal(_bits(rg), r_ref)                      # the stored residual: bit-exact
        hg = h.float().cpu().numpy().astype(np.float64)
        assert np.all(np.abs(hg - h_ref) <= 1.01 * _ulp_bf16(h_ref))  # fp32 math, one bf16 rounding
        assert np.mean(np.abs(hg - h_ref) > 0.51 * _ulp_bf16(h_ref)) < 2e-3


def test_residual_rmsnorm_argument_errors(zeda):
    dev = torch.device("cuda:0")
    r = torch.zeros(4, 96, dtype=torch.bfloat16, device=dev)  # 96 is not a multiple of 64
    with pytest.raises(zeda.ZedaError) as e:
        zeda.residual_rmsnorm(r, None)
    assert e.value.status == -2
    zeda.residual_rmsnorm(torch.zeros(0, 64, dtype=torch.bfloat16, device=dev), None)  # empty: nothing happens


def test_three_layer_stack_per_layer_parity(zeda):
    T, d, He, E, Z, K = 300, 256, 128, 8, 4, 2
    dev = torch.device("cuda:0")
    layers = [inputs.make_layer("stack%d" % l, T=T, d=d, He=He, E=E, Z=Z, K=K, seed=40 + l, zero_fraction=f)
              for l, f in enumerate((0.3, 0.5, 0.7))]
    mods = [zeda.from_workload(wl, dev) for wl in layers]
    r = inputs.make_layer("stack_in", T=T, d=d, He=He, E=E, Z=Z, K=K, seed=39).x.to(dev).clone()
    y = None
    checked = 0
    for wl, m in zip(layers, mods):
        r_before = r.clone()
        h = zeda.residual_rmsnorm(r, y)
        y = m.forward(h)
        torch.cuda.synchronize()
        # glue against the oracle on the GPU's own residual and previous output
        r_ref, h_ref = oracle.residual_rmsnorm(_bits(r_before), None if checked == 0 else _bits(y_prev))
        assert np.array_equal(_bits(r), r_ref)
        # layer against the oracle on the GPU's own h, on tokens whose top-(K+1) logits are a margin apart
        bias = None if wl.router_bias is None else wl.router_bias.numpy()
        lg = oracle.logits(_bits(h), wl.router_w.numpy(), bias)
        top = -np.sort(-lg.astype(np.float64), axis=1)[:, : K + 1]
        ok = np.nonzero(np.min(top[:, :-1] - top[:, 1:], axis=1) >= 1e-3)[0].astype(np.int32)
        assert ok.size > T // 2
        ids = ok[:: max(1, ok.size // 40)]
        y_ref, idx_ref, _ = oracle.forward(_bits(h), wl.router_w.numpy(), bias, inputs.bits(wl.w_gate_up),
                                           inputs.bits(wl.w_down), E, Z, K, token_ids=ids)
        yg = y[torch.as_tensor(ids, device=dev, dtype=torch.long)].float().cpu().numpy().astype(np.float64)
        den = np.linalg.norm(y_ref)
        assert den > 0 and np.linalg.norm(yg - y_ref) / den <= REL_L2
        assert np.max(np.abs(yg - y_ref)) <= MAX_ABS_RMS * np.sqrt(np.mean(y_ref ** 2))
        routed = m.route(h)["topk_idx"].cpu().numpy()
        assert np.array_equal(routed[ids], idx_ref)
        y_prev = y.clone()
        checked += 1
    for m in mods:
        m.close()
    assert checked == 3
