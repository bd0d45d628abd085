"""Expert-parallel forward on one GPU: a whole group of ranks stepped in one process (each rank its
own handle with its share of the experts; device copies stand in for the all-to-all), every rank's
output compared with the CPU oracle's forward of that rank's tokens with ALL experts."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_18643_b200 import ep, inputs

pytestmark = pytest.mark.gpu

REL_L2, MAX_ABS_RMS = 1e-2, 5e-2


@pytest.fixture(scope="module")
def zeda():
    from paper_2605_18643_b200 import zeda as z
    return z


def make_group(zeda, layer, G, max_tokens, dev, gate_mode=0, expert_kind=0):
    E, n_local = layer.E, layer.E // G
    rw, rb = layer.router_w.to(dev), layer.router_bias.to(dev)
    ranks = []
    for r in range(G):
        wgu = layer.w_gate_up[r * n_local:(r + 1) * n_local].contiguous().to(dev)
        wd = layer.w_down[r * n_local:(r + 1) * n_local].contiguous().to(dev)
        m = zeda.ZedaMoE(rw, rb, wgu, wd, E, layer.Z, layer.K, max_tokens, gate_mode=gate_mode, expert_kind=expert_kind,
                         ep_size=G, ep_rank=r, max_recv_pairs=G * max_tokens * layer.K)
        ranks.append(ep.ExpertParallelMoE(m, None))
    return ranks


def check_rank_output(layer, x_cpu, y_gpu, ids=None, gate_mode=0, expert_kind=0):
    y_ref, idx, _ = oracle.forward(inputs.bits(x_cpu), layer.router_w.numpy(), layer.router_bias.numpy(),
                                   inputs.bits(layer.w_gate_up), inputs.bits(layer.w_down), layer.E, layer.Z, layer.K,
                                   gate_mode=gate_mode, expert_kind=expert_kind, token_ids=ids)
    yg = y_gpu.float().cpu().numpy().astype(np.float64)
    if ids is not None:
        yg = yg[ids]
    den = np.linalg.norm(y_ref)
    if den == 0.0:
        assert np.linalg.norm(yg) == 0.0
        return idx
    assert np.linalg.norm(yg - y_ref) / den <= REL_L2
    assert np.max(np.abs(yg - y_ref)) <= MAX_ABS_RMS * np.sqrt(np.mean(y_ref ** 2))
    if expert_kind == 0:
        dead = np.nonzero((idx >= layer.E).all(axis=1))[0]
        if dead.size:
            assert not yg[dead].any() and not np.signbit(yg[dead]).any()      # exact +0 for tokens with no real slot
    return idx


@pytest.mark.parametrize("G", [1, 2, 4])
def test_group_in_one_process_matches_the_oracle(zeda, G):
    dev = torch.device("cuda:0")
    layer = inputs.tiny(seed=31, T=64, E=8, Z=4, K=3)
    Ts = [300, 7, 129, 0][:G] if G > 1 else [300]
    ranks = make_group(zeda, layer, G, 300, dev)
    xs_cpu = [inputs.replica_tokens(inputs.tiny(seed=31, T=max(T, 1), E=8, Z=4, K=3), 10 + r)[:T] for r, T in enumerate(Ts)]
    xs = [x.to(dev) for x in xs_cpu]
    ys = ep.forward_group_in_one_process(ranks, xs)
    torch.cuda.synchronize()
    for r in range(G):
        assert ys[r].shape == xs[r].shape
        if Ts[r]:
            check_rank_output(layer, xs_cpu[r], ys[r])
        ranks[r].moe.last_counters()          # no device-side failure recorded
    # zero-expert slots never enter the exchange: the rows a rank packs are its surviving pairs only
    send_rows, send_counts, expert_counts = ranks[0].moe.ep_dispatch(xs[0])
    torch.cuda.synchronize()
    idx = oracle.forward(inputs.bits(xs_cpu[0]), layer.router_w.numpy(), layer.router_bias.numpy(), inputs.bits(layer.w_gate_up),
                         inputs.bits(layer.w_down), layer.E, layer.Z, layer.K, want_y=False)[1]
    counts, offsets, perm, P = oracle.compact(idx, layer.E)
    assert int(send_counts.sum().item()) == P < Ts[0] * layer.K
    assert np.array_equal(expert_counts.cpu().numpy(), counts)
    assert send_counts.tolist() == ep.send_counts_from_offsets(torch.from_numpy(offsets), layer.E, G)
    want_rows = xs_cpu[0][torch.from_numpy(perm // layer.K).long()]
    assert torch.equal(send_rows[:P].cpu().view(torch.int16), want_rows.view(torch.int16))
    for r in ranks:
        r.moe.close()


def test_one_rank_group_equals_the_plain_layer_bit_for_bit(zeda):
    dev = torch.device("cuda:0")
    layer = inputs.tiny(seed=32, T=400)
    plain = zeda.from_workload(layer, dev)
    x = layer.x.to(dev)
    y0 = plain.forward(x)
    ranks = make_group(zeda, layer, 1, layer.T, dev)
    y1 = ep.forward_group_in_one_process(ranks, [x])[0]
    torch.cuda.synchronize()
    assert torch.equal(y0.view(torch.int16), y1.view(torch.int16))
    with pytest.raises(zeda.ZedaError):
        ranks[0].moe.forward(x)               # an expert-parallel handle runs the layer through the three calls
    plain.close()
    ranks[0].moe.close()


@pytest.mark.parametrize("gate_mode,expert_kind", [(2, 0), (0, 1)])
def test_group_with_gate_modes_and_copy_experts(zeda, gate_mode, expert_kind):
    dev = torch.device("cuda:0")
    layer = inputs.tiny(seed=33, T=200, E=8, Z=4, K=2)
    ranks = make_group(zeda, layer, 2, 200, dev, gate_mode, expert_kind)
    xs_cpu = [layer.x, inputs.replica_tokens(layer, 3)[:150]]
    ys = ep.forward_group_in_one_process(ranks, [x.to(dev) for x in xs_cpu])
    torch.cuda.synchronize()
    for r in range(2):
        check_rank_output(layer, xs_cpu[r], ys[r], gate_mode=gate_mode, expert_kind=expert_kind)
        ranks[r].moe.close()


def test_qwen_shaped_group_of_four(zeda):
    # the spec layer shape, experts over four ranks, 512 tokens per rank
    dev = torch.device("cuda:0")
    layer = inputs.prefill(T=512)
    ranks = make_group(zeda, layer, 4, 512, dev)
    xs_cpu = [layer.x] + [inputs.replica_tokens(layer, 20 + r) for r in range(1, 4)]
    ys = ep.forward_group_in_one_process(ranks, [x.to(dev) for x in xs_cpu])
    torch.cuda.synchronize()
    for r in range(4):
        ids = np.sort(np.random.default_rng(r).choice(512, 24, replace=False)).astype(np.int32)
        check_rank_output(layer, xs_cpu[r], ys[r], ids=ids)
        ranks[r].moe.last_counters()
        ranks[r].moe.close()


def test_row_count_that_contradicts_the_count_matrix_is_reported(zeda):
    dev = torch.device("cuda:0")
    layer = inputs.tiny(seed=34, T=100)
    ranks = make_group(zeda, layer, 1, 100, dev)
    m = ranks[0].moe
    x = layer.x.to(dev)
    send_rows, send_counts, expert_counts = m.ep_dispatch(x)
    P = int(send_counts.sum().item())
    m.ep_experts(send_rows, expert_counts.view(1, -1).contiguous(), P - 1)     # one row short of the matrix's sum
    with pytest.raises(zeda.ZedaError) as e:
        m.last_counters()
    assert e.value.status == zeda.ERR_TIMEOUT and "21" in str(e.value)
    m.clear_error()
    out = m.ep_experts(send_rows, expert_counts.view(1, -1).contiguous(), P)     # the handle still works
    y = m.ep_combine(x, out)
    torch.cuda.synchronize()
    check_rank_output(layer, layer.x, y)
    st = zeda.lib.zeda_ep_experts(m._h, send_rows.data_ptr(), expert_counts.data_ptr(), 10 ** 6, out.data_ptr(), None)
    assert st == zeda.ERR_INVALID_ARG and "max_recv_pairs" in zeda.last_error()    # refused on the host, nothing launched
    m.close()
