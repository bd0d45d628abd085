"""Expert-parallel dispatch plan and exchange on CPU: two gloo ranks on 127.0.0.1.

Each rank routes its own tokens with the oracle, builds the send plan with the product's host-side
plan functions (paper_2605_18643_b200.ep), exchanges counts and rows through the product's exchange
class over gloo, applies the oracle's expert to every received row, sends the results back and
combines.  Checked: zero-expert slots never enter a send list; the rows a rank receives are exactly
the pairs of its experts; the round trip restores every rank's (expert, token) order; and the
combined output equals the oracle's forward of that rank's tokens with all experts."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import json, os, sys
sys.path.insert(0, %(root)r)
import numpy as np
import torch
import torch.distributed as dist
import oracle
from paper_2605_18643_b200 import ep, inputs

rank = int(os.environ["RANK"]); G = int(os.environ["WORLD_SIZE"])
dist.init_process_group(backend="gloo")
wl = inputs.tiny(seed=21, T=90 + 40 * rank, E=8, Z=4, K=3)
if rank == 1:   # same layer on every rank (rank 0's), this rank's own tokens
    base = inputs.tiny(seed=21, T=90, E=8, Z=4, K=3)
    wl.router_w, wl.router_bias, wl.w_gate_up, wl.w_down = base.router_w, base.router_bias, base.w_gate_up, base.w_down
E, Z, K, d = wl.E, wl.Z, wl.K, wl.d
n_local = E // G
xb = inputs.bits(wl.x)
bias = wl.router_bias.numpy()
_, idx, w = oracle.forward(xb, wl.router_w.numpy(), bias, inputs.bits(wl.w_gate_up), inputs.bits(wl.w_down), E, Z, K, want_y=False)
counts, offsets, perm, P = oracle.compact(idx, E)

# ---- plan: what goes where
send_splits = ep.send_counts_from_offsets(torch.from_numpy(offsets), E, G)
assert sum(send_splits) == P == int((idx < E).sum())            # zero slots are not in any send list
slot_expert = idx.reshape(-1)[perm]
assert (slot_expert < E).all()
for r in range(G):                                               # block r holds exactly the pairs of rank r's experts
    lo = sum(send_splits[:r]); blk = slot_expert[lo:lo + send_splits[r]]
    assert all(ep.owner_of_expert(int(e), E, G) == r for e in blk)
send_rows = wl.x[torch.from_numpy(perm // K).long()]            # x rows of the surviving pairs, (expert, token) order

xchg = ep.TorchDistExchange()
recv_counts = xchg.counts(torch.from_numpy(counts))
recv_splits, n_rows = ep.recv_layout(recv_counts)
recv_rows = xchg.rows(send_rows, send_splits, recv_splits)
tot = torch.tensor([P, n_rows], dtype=torch.int64); dist.all_reduce(tot)
assert int(tot[0]) == int(tot[1])                                # every sent row is received once

# ---- this rank's experts on what it received (oracle arithmetic), in received order
out = torch.empty((max(n_rows, 1), d), dtype=torch.float64)
row = 0
wgu, wd = inputs.bits(wl.w_gate_up), inputs.bits(wl.w_down)
for s in range(G):
    for j in range(n_local):
        e = rank * n_local + j
        for _ in range(int(recv_counts[s, j])):
            out[row] = torch.from_numpy(oracle.expert(inputs.bits(recv_rows[row:row + 1])[0], wgu[e], wd[e]))
            row += 1
assert row == n_rows
back = xchg.rows(out, recv_splits, send_splits)                  # results return in the order of send_rows

# ---- combine (Eq. 1) and compare with the oracle's forward of this rank's tokens
y = np.zeros((wl.T, d))
inv = np.full(wl.T * K, -1); inv[perm] = np.arange(P)
for t in range(wl.T):
    for k in range(K):
        p = inv[t * K + k]
        if p >= 0:
            y[t] += w[t, k] * back[p].numpy()
y_ref, _, _ = oracle.forward(xb, wl.router_w.numpy(), bias, wgu, wd, E, Z, K)
err = float(np.max(np.abs(y - y_ref)))
dist.barrier()
print(json.dumps({"rank": rank, "P": int(P), "slots": int(wl.T * K), "recv": int(n_rows), "err": err,
                  "send": send_splits, "recv_splits": recv_splits}))
dist.destroy_process_group()
'''


def _env(rank, world, port):
    e = dict(os.environ)
    e.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
             MASTER_PORT=str(port), OMP_NUM_THREADS="2")
    return e


def test_two_gloo_ranks_dispatch_compute_and_return():
    port = 33500 + os.getpid() % 2000
    procs = [subprocess.Popen([sys.executable, "-c", WORKER % {"root": ROOT}], env=_env(r, 2, port),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=600) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = [json.loads(o[0].strip().splitlines()[-1]) for o in outs]
    for r in res:
        assert 0 < r["P"] < r["slots"]            # some slots fell on zero experts and were dropped
        assert r["err"] < 1e-12                   # same fp64 arithmetic, other grouping only
    # what rank a sends to rank b is what b receives from a
    for a in range(2):
        for b in range(2):
            assert res[a]["send"][b] == res[b]["recv_splits"][a]


def test_plan_functions_on_small_cases():
    import torch
    sys.path.insert(0, ROOT)
    from paper_2605_18643_b200 import ep
    offsets = torch.tensor([0, 3, 3, 10, 11, 11, 11, 20, 26])          # 8 experts
    assert ep.send_counts_from_offsets(offsets, 8, 1) == [26]
    assert ep.send_counts_from_offsets(offsets, 8, 2) == [11, 15]
    assert ep.send_counts_from_offsets(offsets, 8, 4) == [3, 8, 0, 15]
    assert [ep.owner_of_expert(e, 8, 4) for e in range(8)] == [0, 0, 1, 1, 2, 2, 3, 3]
    per, total = ep.recv_layout(torch.tensor([[1, 2], [0, 0], [5, 1]]))
    assert per == [3, 0, 6] and total == 9
