"""zeda_compact_static: the allocation-free counting sort, for callers that are handed device
buffers but may not call the CUDA allocator themselves (plug-ins inside a host framework, code in
a region where allocation is forbidden, fixed-budget processes).  Its scratch is a fixed array in
the library, so the checks are: same results as the workspace-based entry point, bit for bit, on
two calls in a row with different inputs (the array keeps the previous call's contents), and a
clear refusal beyond the stated maximum.  Collected last so that a failure here cannot hide the
other GPU tests."""
import numpy as np
import pytest
import torch

from paper_2605_18643_b200 import inputs

pytestmark = pytest.mark.gpu


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
        m.close()


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
