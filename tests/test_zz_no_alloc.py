"""zeda_compact_static: the allocation-free counting sort, for callers that are handed device
buffers but may not call the CUDA allocator themselves (plug-ins inside a host framework, code in
a region where allocation is forbidden, fixed-budget processes).  Its scratch is a fixed array in
the library, so the checks are: same results as the workspace-based entry point and as the CPU
oracle, bit for bit, on calls in a row with different inputs (the array keeps the previous call's
contents), at the stated maximum sizes, with padding ids, and a clear refusal beyond the maximum.
Collected last so that a failure here cannot hide the other GPU tests."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_18643_b200 import inputs

pytestmark = pytest.mark.gpu


def check_against_oracle(zeda, idx_np, n_real):
    dev = torch.device("cuda:0")
    idx = torch.from_numpy(idx_np).to(dev)
    counts, offsets, perm, n_pairs = zeda.compact_static(idx, n_real)
    torch.cuda.synchronize()
    # a dropped slot is a dropped slot: the oracle sees padding ids as a zero-expert id
    ref_in = np.where(idx_np < 0, n_real, idx_np).astype(np.int32)
    c_ref, o_ref, p_ref, P = oracle.compact(ref_in, n_real)
    assert int(n_pairs.item()) == P
    assert np.array_equal(counts.cpu().numpy(), c_ref)
    assert np.array_equal(offsets.cpu().numpy(), o_ref)
    got = perm.cpu().numpy()
    assert np.array_equal(got[:P], p_ref)
    assert np.all(got[P:] == -1)                       # the tail is left untouched
    return P


def test_static_compaction_matches_workspace_entry_point_twice():
    from paper_2605_18643_b200 import zeda
    dev = torch.device("cuda:0")
    # two different batches, the larger first so that stale scratch would show in the second
    for seed, T in ((11, 1000), (12, 130)):
        wl = inputs.tiny(seed=seed, T=T)
        m = zeda.from_workload(wl, dev)
        ref = m.route(wl.x.to(dev))
        torch.cuda.synchronize()
        counts, offsets, perm, n_pairs = zeda.compact_static(ref["topk_idx"], wl.E)
        torch.cuda.synchronize()
        P = int(ref["n_pairs"].item())
        assert int(n_pairs.item()) == P and 0 < P < T * wl.K
        assert torch.equal(counts, ref["counts"])
        assert torch.equal(offsets, ref["offsets"])
        assert torch.equal(perm, ref["perm"])          # first P entries equal, the tail untouched (-1)
        assert check_against_oracle(zeda, ref["topk_idx"].cpu().numpy(), wl.E) == P
        m.close()


def test_static_compaction_at_its_maximum_sizes_then_a_small_call():
    # the largest call the fixed array admits (32 sort blocks, 512 experts, 32768 slots, zero-expert
    # ids mixed in), then a small one right after it: nothing of the large call may leak
    from paper_2605_18643_b200 import zeda
    rng = np.random.default_rng(5)
    T, K, n_real = zeda.STATIC_MAX_TOKENS, 8, 512
    assert T * K == zeda.STATIC_MAX_SLOTS
    idx = np.stack([rng.permutation(n_real + 200)[:K] for _ in range(T)]).astype(np.int32)
    P = check_against_oracle(zeda, idx, n_real)
    assert 0 < P < T * K
    small = np.stack([rng.permutation(12)[:2] for _ in range(77)]).astype(np.int32)
    check_against_oracle(zeda, small, 8)
    one_expert = np.zeros((300, 1), dtype=np.int32)     # a single expert holding every slot
    assert check_against_oracle(zeda, one_expert, 1) == 300


def test_static_compaction_drops_padding_ids():
    # ids < 0 (padding slots) are dropped exactly like zero-expert ids
    from paper_2605_18643_b200 import zeda
    rng = np.random.default_rng(6)
    idx = np.stack([rng.permutation(12)[:3] for _ in range(500)]).astype(np.int32)
    idx[rng.random(idx.shape) < 0.3] = -1
    idx[7] = -1                                         # a token with nothing but padding
    idx[100:110, 0] = -(2 ** 31)
    P = check_against_oracle(zeda, idx, 8)
    assert 0 < P < idx.size


def test_static_compaction_rejects_sizes_beyond_its_array():
    from paper_2605_18643_b200 import zeda
    dev = torch.device("cuda:0")
    idx = torch.zeros((zeda.STATIC_MAX_TOKENS + 1, 2), dtype=torch.int32, device=dev)
    with pytest.raises(zeda.ZedaError) as e:
        zeda.compact_static(idx, 8)
    assert e.value.status == zeda.ERR_UNSUPPORTED and "at most" in str(e.value)
    idx = torch.zeros((zeda.STATIC_MAX_TOKENS, 16), dtype=torch.int32, device=dev)   # too many slots
    with pytest.raises(zeda.ZedaError) as e:
        zeda.compact_static(idx, 8)
    assert e.value.status == zeda.ERR_UNSUPPORTED
