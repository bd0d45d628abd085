"""Parity of the CUDA library (through its C ABI) with the CPU oracle on the same seeded inputs.

Bars: routing indices, per-expert counts, offsets, permutation and P bit-exact; routing weights
within fp32 rounding (rel 1e-5); layer output rel-L2 <= 1e-2 and max-abs <= 5e-2 * RMS(y).
"""
import copy

import numpy as np
import pytest
import torch

import oracle
from paper_2605_18643_b200 import inputs

pytestmark = pytest.mark.gpu

REL_L2 = 1e-2
MAX_ABS_RMS = 5e-2
W_RTOL = 1e-5


@pytest.fixture(scope="module")
def zeda():
    from paper_2605_18643_b200 import zeda as z
    return z


def np_bias(wl):
    return None if wl.router_bias is None else wl.router_bias.numpy()


def oracle_route(wl, gate_mode=0):
    l = oracle.logits(inputs.bits(wl.x), wl.router_w.numpy(), np_bias(wl))
    idx, w = oracle.route(l, wl.E, wl.Z, wl.K, gate_mode)
    counts, offsets, perm, P = oracle.compact(idx, wl.E)
    return l, idx, w, counts, offsets, perm, P


def oracle_forward(wl, token_ids=None, gate_mode=0, expert_kind=0):
    return oracle.forward(inputs.bits(wl.x), wl.router_w.numpy(), np_bias(wl), inputs.bits(wl.w_gate_up),
                          inputs.bits(wl.w_down), wl.E, wl.Z, wl.K, gate_mode=gate_mode,
                          expert_kind=expert_kind, token_ids=token_ids)


def check_route(o, idx, w, counts, offsets, perm, P):
    assert np.array_equal(o["topk_idx"].cpu().numpy(), idx)
    assert int(o["n_pairs"].item()) == P
    assert np.array_equal(o["counts"].cpu().numpy(), counts)
    assert np.array_equal(o["offsets"].cpu().numpy(), offsets)
    got_perm = o["perm"].cpu().numpy()
    assert np.array_equal(got_perm[:P], perm)
    assert np.all(got_perm[P:] == -1)                       # the tail is left untouched
    gw = o["topk_w"].cpu().numpy().astype(np.float64)
    assert np.allclose(gw, w, rtol=W_RTOL, atol=1e-30)


def check_y(y_gpu, y_ref):
    y_gpu = y_gpu.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(y_gpu))
    num = np.linalg.norm(y_gpu - y_ref)
    den = np.linalg.norm(y_ref)
    rms = np.sqrt(np.mean(y_ref ** 2))
    if den == 0.0:
        assert num == 0.0
        return 0.0
    assert num / den <= REL_L2, "rel L2 %.3e" % (num / den)
    assert np.max(np.abs(y_gpu - y_ref)) <= MAX_ABS_RMS * rms
    return num / den


def sample_tokens(T, n, seed):
    return np.sort(np.random.default_rng(seed).choice(T, size=n, replace=False)).astype(np.int32)


def run_layer(zeda, wl, token_ids=None, gate_mode=0, expert_kind=0, flags=0, check_routing=True):
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev, gate_mode=gate_mode, expert_kind=expert_kind, flags=flags)
    x = wl.x.to(dev)
    if check_routing:
        l, idx, w, counts, offsets, perm, P = oracle_route(wl, gate_mode)
        gl = m.router_logits(x).cpu().numpy()
        # fp32 accumulation over d products: the bar grows with d beyond the spec width
        assert np.max(np.abs(gl.astype(np.float64) - l.astype(np.float64))) < 2e-5 * max(1.0, wl.d / 2048)
        check_route(m.route(x), idx, w, counts, offsets, perm, P)
    y = m.forward(x)
    torch.cuda.synchronize()
    y_ref, idx_ref, _ = oracle_forward(wl, token_ids, gate_mode, expert_kind)
    ysel = y if token_ids is None else y[torch.as_tensor(token_ids, device=dev, dtype=torch.long)]
    err = check_y(ysel, y_ref)
    # tokens without a surviving slot: every element is +0 (bit pattern 0)
    if expert_kind == 0:
        dead = np.nonzero((idx_ref >= wl.E).all(axis=1))[0]
        if dead.size:
            rows = ysel[torch.as_tensor(dead, device=dev, dtype=torch.long)].view(torch.int16)
            assert int(rows.abs().max().item()) == 0
    P_dev, U_dev, zero_slots, launches = m.last_counters()
    assert launches > 0
    m.close()
    return err, (P_dev, U_dev, zero_slots)


# ---------------------------------------------------------------------------------- tiny layer

def test_tiny_routing_and_forward(zeda):
    wl = inputs.tiny()
    err, (P, U, zs) = run_layer(zeda, wl)
    assert P + zs == wl.T * wl.K and 0 < P < wl.T * wl.K


@pytest.mark.parametrize("gate_mode", [0, 1, 2])
@pytest.mark.parametrize("expert_kind", [0, 1])
def test_tiny_gate_modes_and_copy_experts(zeda, gate_mode, expert_kind):
    run_layer(zeda, inputs.tiny(seed=1), gate_mode=gate_mode, expert_kind=expert_kind)


@pytest.mark.parametrize("gate_mode,expert_kind", [(1, 0), (2, 0), (0, 1), (2, 1)])
def test_gate_modes_and_copy_experts_on_the_large_batch_kernels(zeda, gate_mode, expert_kind):
    # T > 128: separate top-K kernel, tensor-core router, multi-CTA counting sort
    wl = inputs.tiny(seed=3, T=300)
    run_layer(zeda, wl, token_ids=sample_tokens(300, 40, 2), gate_mode=gate_mode, expert_kind=expert_kind)


def test_tiny_static_layer_z0(zeda):
    wl = inputs.tiny(seed=2, Z=0, zero_fraction=None)
    err, (P, U, zs) = run_layer(zeda, wl)
    assert zs == 0 and P == wl.T * wl.K


def test_route_from_logits_is_bit_exact_with_ties(zeda):
    wl = inputs.tiny()
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev, max_tokens=300)
    rng = np.random.default_rng(0)
    l = rng.standard_normal((300, wl.E + wl.Z)).astype(np.float32)
    l[:50] = np.round(l[:50] * 2) / 2          # many exact ties
    l[50] = 0.0
    # zeros of both signs are equal logits: the lower id wins whatever its sign bit
    l[51] = np.where(np.arange(wl.E + wl.Z) % 2 == 0, -0.0, 0.0)
    l[52] = np.where(np.arange(wl.E + wl.Z) % 3 == 0, 0.0, -0.0)
    l[53] = -1.0
    l[53, [5, 2, 9]] = [-0.0, 0.0, -0.0]
    l[54] = np.where(rng.random(wl.E + wl.Z) < 0.5, -0.0, 0.0)
    assert np.signbit(l[51, 0]) and not np.signbit(l[51, 1])
    idx, w = oracle.route(l, wl.E, wl.Z, wl.K)
    assert list(idx[51]) == [0, 1] and list(idx[53]) == [2, 5]
    counts, offsets, perm, P = oracle.compact(idx, wl.E)
    o = m.route_from_logits(torch.from_numpy(l).to(dev))
    torch.cuda.synchronize()
    check_route(o, idx, w, counts, offsets, perm, P)
    m.close()


def test_forward_is_deterministic(zeda):
    wl = inputs.tiny(seed=4)
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    x = wl.x.to(dev)
    a = m.forward(x).clone()
    b = m.forward(x).clone()
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    m.close()


# ---------------------------------------------------------------------------------- edge cases

@pytest.mark.parametrize("T", [1, 7, 129, 257])
def test_ragged_token_counts(zeda, T):
    run_layer(zeda, inputs.tiny(seed=5, T=T))


def test_empty_batch_touches_nothing(zeda):
    wl = inputs.tiny()
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    x = torch.empty((0, wl.d), dtype=torch.bfloat16, device=dev)
    y = m.forward(x)
    assert y.shape == (0, wl.d)
    m.close()


def test_every_slot_on_a_zero_expert(zeda):
    wl = inputs.tiny(seed=6)
    wl.router_bias[wl.E:] += 50.0
    err, (P, U, zs) = run_layer(zeda, wl)
    assert P == 0 and U == 0 and zs == wl.T * wl.K


def test_all_tokens_on_one_expert(zeda):
    wl = inputs.tiny(seed=7, T=200)
    wl.router_bias[:wl.E] -= 50.0
    wl.router_bias[3] += 100.0
    err, (P, U, zs) = run_layer(zeda, wl)
    o = oracle_route(wl)
    assert o[3][3] == wl.T and (np.delete(o[3], 3) == 0).all() and U == 1   # expert 3 has every token


def test_argument_errors(zeda):
    wl = inputs.tiny()
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    x = wl.x.to(dev)
    with pytest.raises(zeda.ZedaError) as e:
        m.forward(torch.cat([x, x]))                        # T > max_tokens
    assert e.value.status == zeda.ERR_INVALID_ARG
    st = zeda.lib.zeda_moe_forward(m._h, x.data_ptr() + 2, wl.T - 1, x.data_ptr(), None)
    assert st == zeda.ERR_INVALID_ARG                       # misaligned
    st = zeda.lib.zeda_moe_forward(m._h, x.data_ptr(), wl.T, x.data_ptr(), None)
    assert st == zeda.ERR_INVALID_ARG                       # x and y overlap
    y = m.forward(x)                                        # the handle still works afterwards
    torch.cuda.synchronize()
    assert torch.isfinite(y.float()).all()
    m.close()


def test_host_buffer_entry_point(zeda):
    wl = inputs.tiny(seed=8)
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    y_dev = m.forward(wl.x.to(dev)).cpu()
    y_host = m.forward_host(wl.x.pin_memory())
    assert torch.equal(y_dev.view(torch.int16), y_host.view(torch.int16))
    y_pageable = m.forward_host(wl.x.clone())
    assert torch.equal(y_dev.view(torch.int16), y_pageable.view(torch.int16))
    m.close()


def test_host_buffer_entry_point_in_two_chunks(zeda):
    # from 4096 tokens on the host-buffer call copies and computes in two chunks on three streams: the
    # result is, bit for bit, that of the two chunks passed through zeda_moe_forward one after the other
    # (also for a ragged split and on a second call), and the whole-batch result up to the last bits of
    # the routing weights (the router slices its reduction axis by batch size)
    for T in (4096, 5000):
        wl = inputs.tiny(seed=17, T=T)
        dev = torch.device("cuda:0")
        m = zeda.from_workload(wl, dev)
        x = wl.x.to(dev)
        T0 = (T // 2 + 255) // 256 * 256
        y_whole = m.forward(x).float().cpu()
        y_chunks = torch.cat([m.forward(x[:T0].contiguous()), m.forward(x[T0:].contiguous())]).cpu()
        x_pin = wl.x.pin_memory()
        for _ in range(2):
            y_host = m.forward_host(x_pin)
            assert torch.equal(y_chunks.view(torch.int16), y_host.view(torch.int16))
        assert m.last_counters()[3] > 0
        diff = (y_host.float() - y_whole).norm() / y_whole.norm()
        assert float(diff) < 1e-3
        m.close()


def test_routing_statistics(zeda):
    wl = inputs.tiny(seed=9, T=200)
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    f, p, o = m.stats(wl.x.to(dev))
    l, idx, *_ = oracle_route(wl)
    s = oracle.stats(l, idx, wl.E, wl.Z, alpha=1.0, group_w=1.0)
    assert np.allclose(f.cpu().numpy(), s["f"], rtol=1e-5, atol=1e-7)
    assert np.allclose(p.cpu().numpy(), s["P"], rtol=1e-4, atol=1e-7)
    o = o.cpu().numpy().astype(np.float64)
    assert np.isclose(o[0], s["r_ze"], rtol=1e-5)
    n = wl.E + wl.Z
    assert np.isclose(o[1] * n / wl.K, s["L_A"], rtol=1e-4)
    assert np.isclose((wl.E + wl.Z) / wl.K * (o[2] / wl.E + o[3] / wl.Z), s["L_GA"], rtol=1e-4)
    m.close()


def test_per_token_zero_share(zeda):
    # the decode recipe spreads the per-token zero share over 0..100 %
    wl = inputs.decode()
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    x = wl.x.to(dev)
    m.forward(x)
    r = m.token_zero_share(wl.T).cpu().numpy()
    _, idx, *_ = oracle_route(wl)
    want = oracle.token_zero_share(idx, wl.E)
    assert np.array_equal(r, want.astype(np.float32))
    assert r.min() == 0.0 and r.max() == 1.0 and abs(r.mean() - wl.zero_fraction) < 1e-6
    with pytest.raises(zeda.ZedaError):
        m.token_zero_share(wl.T - 1)               # not the size of the last routing call
    m.close()


def test_tensor_core_router_path(zeda):
    # T >= 256 sends the router GEMM to the tensor cores (three-way bf16 split of the fp32 rows)
    for T in (256, 1000):
        wl = inputs.tiny(seed=10, T=T)
        run_layer(zeda, wl, token_ids=sample_tokens(T, 48, 1))


@pytest.mark.parametrize("T,max_tokens", [(300, 300), (2500, 2500), (2500, 9000), (5000, 5000), (300, 20000)])
def test_router_with_sliced_reduction_axis(zeda, T, max_tokens):
    # mid-sized batches cut the router's reduction axis into 2 or 4 slices (as many as keep the grid
    # within the SMs and the slices within the workspace); the top-K kernel adds them.  Routing from
    # x must equal both the oracle's and the routing from the complete logits.
    wl = inputs.tiny(seed=12, T=T, d=512, E=96, Z=40, K=4)
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev, max_tokens=max_tokens)
    x = wl.x.to(dev)
    l, idx, w, counts, offsets, perm, P = oracle_route(wl)
    a = m.route(x)
    check_route(a, idx, w, counts, offsets, perm, P)
    b = m.route_from_logits(m.router_logits(x))
    assert torch.equal(a["topk_idx"], b["topk_idx"]) and torch.equal(a["perm"], b["perm"])
    # the statistics read complete logits, whichever way the routing before them got its own
    f, p, _ = m.stats(x)
    s = oracle.stats(l, idx, wl.E, wl.Z, alpha=1.0, group_w=1.0)
    assert np.allclose(f.cpu().numpy(), s["f"], rtol=1e-5, atol=1e-7)
    assert np.allclose(p.cpu().numpy(), s["P"], rtol=1e-4, atol=1e-7)
    m.close()


# ---------------------------------------------------------------------------------- full-size configs

def test_decode_config_full_parity(zeda):
    wl = inputs.decode()
    err, (P, U, zs) = run_layer(zeda, wl)
    assert abs(zs / (wl.T * wl.K) - 0.5) < 0.03


def test_decode_config_static_reference(zeda):
    wl = inputs.decode(Z=0, zero_fraction=None, token_shift=0.0)
    run_layer(zeda, wl)


def test_prefill_config_routing_exact_and_sampled_outputs(zeda):
    wl = inputs.prefill()
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    x = wl.x.to(dev)
    # routing of all 8192 tokens, bit-exact (oracle routing only: no expert math)
    _, idx, w = oracle.forward(inputs.bits(wl.x), wl.router_w.numpy(), np_bias(wl), inputs.bits(wl.w_gate_up),
                               inputs.bits(wl.w_down), wl.E, wl.Z, wl.K, want_y=False)
    counts, offsets, perm, P = oracle.compact(idx, wl.E)
    check_route(m.route(x), idx, w, counts, offsets, perm, P)
    assert np.sort(counts)[-1] > 10 * max(1, np.sort(counts)[len(counts) // 2])   # the Zipf skew is there
    ids_l = sample_tokens(wl.T, 64, 5)
    l_ref = oracle.logits(inputs.bits(wl.x)[ids_l], wl.router_w.numpy(), np_bias(wl))
    l_gpu = m.router_logits(x).cpu().numpy()[ids_l]
    assert np.max(np.abs(l_gpu.astype(np.float64) - l_ref.astype(np.float64))) < 2e-5
    # outputs on a token sample (each token's output depends on its own row only)
    ids = sample_tokens(wl.T, 192, 0)
    y = m.forward(x)
    torch.cuda.synchronize()
    y_ref, _, _ = oracle_forward(wl, ids)
    check_y(y[torch.as_tensor(ids, device=dev, dtype=torch.long)], y_ref)
    # every element of the full batch is the same bits on a second run: work items are handed out at
    # run time, but no sum depends on who computes it
    y2 = m.forward(x)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    m.close()


@pytest.mark.parametrize("f", [0.0, 0.25, 0.5, 0.75])
def test_sweep_config_sampled(zeda, f):
    wl = inputs.sweep_point(f)
    ids = sample_tokens(wl.T, 64, int(f * 100))
    # routing of all 2048 tokens is compared bit for bit: at this size the router runs on the tensor
    # cores with its reduction axis in slices
    err, (P, U, zs) = run_layer(zeda, wl, token_ids=ids)
    assert abs(zs / (wl.T * wl.K) - f) < 0.02


# ---------------------------------------------------------------------------------- kernel-path coverage

def test_dependent_launch_flag_gives_identical_bits(zeda):
    # the same kernels launched fully stream-ordered (flag 4) and with programmatic dependent launch
    wl = inputs.tiny(seed=5, T=700)
    dev = torch.device("cuda:0")
    x = wl.x.to(dev)
    outs = []
    for flags in (0, 4):
        m = zeda.from_workload(wl, dev, flags=flags)
        for _ in range(3):  # back-to-back calls overlap the tail of one with the head of the next
            y = m.forward(x)
        torch.cuda.synchronize()
        outs.append(y.view(torch.int16).clone())
        m.close()
    assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("d,He", [(320, 192), (64, 64), (576, 448)])
def test_ragged_weight_row_blocks(zeda, d, He):
    # d not a multiple of 256 and H_e not a multiple of 128: the last weight-row block of both
    # expert GEMMs is partly (or, for one CTA of the pair, wholly) out of range
    wl = inputs.tiny(seed=6, T=200, d=d, He=He)
    run_layer(zeda, wl, token_ids=sample_tokens(200, 40, 3))


def test_experts_with_many_tiles(zeda):
    # few experts, many tokens: every expert spans several 256-row tiles plus a ragged one
    wl = inputs.tiny(seed=7, T=3000, E=4, Z=2)
    err, (P, U, zs) = run_layer(zeda, wl, token_ids=sample_tokens(3000, 48, 4))
    assert U == 4 and P > 4 * 256


@pytest.mark.parametrize("T", [2400, 1400])
def test_narrow_tiles_that_take_two_weight_row_blocks_per_item(zeda, T):
    # Skewed load on the large-batch kernels.  T = 2400: experts with 0, 1, 2, 9 ... 53 pairs (tiles of
    # at most 64 rows: two weight-row blocks per work item in both expert GEMMs), 97, 201, 533 (two
    # full tiles and a narrow one) and 1449.  T = 1400 (175 slots per candidate) takes the first GEMM's
    # form for mid-sized batches, where tiles of up to 128 rows (here 127) run as such items too.
    # H_e = 320 and d = 768 give both GEMMs three weight-row blocks: a pair and an odd one.  Every
    # token is checked.
    wl = inputs.tiny(seed=11, T=T, E=12, Z=4, K=2, d=768, He=320, zipf_s=0.8)
    _, idx, _, counts, _, _, P = oracle_route(wl)
    c = np.sort(counts)
    assert c[0] == 0 and np.any((c > 0) & (c <= 32)) and np.any((c > 32) & (c <= 64))
    assert np.any((c > 64) & (c <= 128)) and np.any((c > 128) & (c <= 512)) and np.any(c > 512)
    assert any(0 < int(v) % 256 <= 64 for v in c if v > 256)  # a narrow tile behind full ones
    err, (P_dev, U, zs) = run_layer(zeda, wl)
    assert P_dev == P


def test_routing_with_many_sort_blocks(zeda):
    # more than 256 blocks of 128 tokens: the counting sort takes its three-launch path
    wl = inputs.tiny(seed=8, T=33000, d=64, He=64)
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    l, idx, w, counts, offsets, perm, P = oracle_route(wl)
    x = wl.x.to(dev)
    check_route(m.route(x), idx, w, counts, offsets, perm, P)
    ids = sample_tokens(wl.T, 48, 9)
    y = m.forward(x)
    torch.cuda.synchronize()
    y_ref, _, _ = oracle_forward(wl, ids)
    check_y(y[torch.as_tensor(ids, device=dev, dtype=torch.long)], y_ref)
    m.close()


@pytest.mark.parametrize("T", [40, 600])
def test_maximum_candidates_and_top_k(zeda, T):
    # the limits of the interface: N + N_Z = 512 candidates (16 logits per lane in the top-K warp,
    # four candidate tiles in the tensor-core router) and K = 16 slots per token
    wl = inputs.tiny(seed=13, T=T, d=256, He=128, E=384, Z=128, K=16)
    err, (P, U, zs) = run_layer(zeda, wl, token_ids=sample_tokens(T, 24, 6))
    assert P + zs == T * 16 and zs > 0 and U > 100


def test_one_handle_many_batch_sizes(zeda):
    # one handle (workspace sized for the largest batch) serves calls of very different sizes in a
    # row: nothing of an earlier call (work lists, counters, histograms) may leak into the next
    base = inputs.tiny(seed=14, T=900)
    dev = torch.device("cuda:0")
    m = zeda.from_workload(base, dev, max_tokens=900)
    for T in (900, 5, 300, 64, 1, 257, 900):
        wl = copy.copy(base)                      # the same layer on the first T tokens
        wl.x, wl.T = base.x[:T].contiguous(), T
        x = wl.x.to(dev)
        l, idx, w, counts, offsets, perm, P = oracle_route(wl)
        check_route(m.route(x), idx, w, counts, offsets, perm, P)
        y = m.forward(x)
        torch.cuda.synchronize()
        ids = sample_tokens(T, min(T, 32), T)
        y_ref, _, _ = oracle_forward(wl, ids)
        check_y(y[torch.as_tensor(ids, device=dev, dtype=torch.long)], y_ref)
    m.close()


@pytest.mark.parametrize("E,Z,K", [(1, 1, 2), (1, 0, 1), (8, 4, 1), (2, 30, 8)])
def test_degenerate_expert_sets(zeda, E, Z, K):
    # one normal expert; no zero expert at all with K = 1; a single slot per token; far more zero
    # experts than normal ones
    for T in (33, 300):
        wl = inputs.tiny(seed=15, T=T, E=E, Z=Z, K=K, zero_fraction=None)
        run_layer(zeda, wl, token_ids=sample_tokens(T, 24, 7))


def test_wide_model_and_expert_dimensions(zeda):
    # many k-steps per work item in both GEMMs (d = 4096: 64 k-steps in GEMM1; H_e = 2048: 32 in
    # GEMM2) and many weight-row blocks
    wl = inputs.tiny(seed=16, T=320, d=4096, He=2048, E=4, Z=2, K=2)
    run_layer(zeda, wl, token_ids=sample_tokens(320, 16, 8))


# ---------------------------------------------------------------------------------- second model shape

def test_glm_shaped_layer_and_net_point(zeda):
    # Table of adapted models (Section 3.1): the second model has N=64, K=4, N_Z=32; its hidden
    # sizes are not in the paper, so d and H_e are free parameters here.  NET (the paper's iso-FLOP
    # static baseline) is the same layer with no zero experts and K/2 slots.
    shape = dict(T=512, d=1024, He=512, E=64, Z=32, K=4)
    wl = inputs.make_layer("glm_shaped", seed=12, zero_fraction=0.5, **shape)
    err, (P, U, zs) = run_layer(zeda, wl, token_ids=sample_tokens(512, 40, 5))
    assert abs(zs / (wl.T * wl.K) - 0.5) < 0.03
    net = inputs.make_layer("glm_net", seed=12, zero_fraction=None, **dict(shape, Z=0, K=2))
    err, (Pn, Un, zsn) = run_layer(zeda, net, token_ids=sample_tokens(512, 40, 6))
    assert zsn == 0 and Pn == net.T * net.K
    # NET spends K/2 expert evaluations per token; the zero-expert layer about K (1 - r_ZE) = K/2 on average
    assert abs(P / Pn - 1.0) < 0.06


def test_expired_device_wait_is_reported_and_the_handle_stays_usable(zeda):
    # failure detection without a fault: a wait with a 1 ms limit on a barrier that nothing signals
    wl = inputs.tiny(seed=9)
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    x = wl.x.to(dev)
    y0 = m.forward(x).view(torch.int16).clone()
    m.last_counters()                       # no error pending
    m.selftest_wait(limit_us=1000)
    with pytest.raises(zeda.ZedaError) as e:
        m.last_counters()
    assert e.value.status == -5 and "wait expired" in str(e.value)
    with pytest.raises(zeda.ZedaError):     # sticky until cleared
        m.last_counters()
    m.clear_error()
    y1 = m.forward(x).view(torch.int16)
    torch.cuda.synchronize()
    assert torch.equal(y0, y1)
    m.last_counters()
    m.close()


def test_forward_can_be_captured_in_a_cuda_graph(zeda):
    # the call enqueues kernels only (no allocation, no host synchronisation): it can be captured once
    # and replayed on new contents of the same buffers
    wl = inputs.tiny(seed=13, T=300)
    dev = torch.device("cuda:0")
    m = zeda.from_workload(wl, dev)
    x = wl.x.to(dev)
    y = torch.empty_like(x)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(2):
            m.forward(x, y)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            m.forward(x, y)
    torch.cuda.synchronize()
    x2 = inputs.tiny(seed=14, T=300).x.to(dev)
    for src in (x2, wl.x.to(dev)):
        x.copy_(src)
        graph.replay()
        torch.cuda.synchronize()
        got = y.view(torch.int16).clone()
        want = m.forward(src.clone()).view(torch.int16)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
    del graph
    m.close()
