"""dct_dp_compress_static: the workspace-free variant of dct_dp_compress.

Collected last on purpose (file name), so that a run that stops at the first failure has already
gone through every other test.  The variant keeps its tile descriptors in an array built into the
library, for callers that cannot allocate device memory themselves (hooks running inside a framework
whose allocator owns the GPU).  It must give bit-identical results to the workspace version, also on
a second call that finds the array full of the first call's leftovers."""
import numpy as np
import pytest
import torch

from paper_2010_08899_b200 import binding as B
from paper_2010_08899_b200 import inputs


def _run(entry, g, e0, tau, budget, cap, **kw):
    e = e0.clone()
    idx = torch.full((cap + 16,), -3, dtype=torch.int32, device="cuda")
    val = torch.full((cap + 16,), -3.0, device="cuda")
    res = B.new_result()
    bud = None if budget is None else torch.tensor([budget], dtype=torch.int64, device="cuda")
    entry(g, e, g.numel(), tau, bud, idx, val, cap, res, **kw)
    r = B.read_result(res)
    return idx.cpu().numpy(), val.cpu().numpy().view(np.uint32), e.cpu().numpy().view(np.uint32), r


@pytest.mark.gpu
def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row():
    cases = [
        # (n, seed, k, tie budget?, capacity): the second call is smaller than the first, so it runs over
        # descriptors the first one left behind; the third overflows its capacity
        ((1 << 22) + 1234, 1, 4000, False, 1 << 16),
        (700_001, 2, 9000, True, 1 << 16),
        (3 * 4096, 3, 5000, False, 100),
    ]
    for n, seed, k, use_budget, cap in cases:
        g = inputs.dp_gaussian(n, seed, "cuda")
        e0 = inputs.dp_gaussian(n, 100 + seed, "cuda") * 0.25
        tau = torch.zeros(1, device="cuda")
        sel = B.new_result()
        B.dct_threshold_select(g, e0, n, k, tau, sel, B.new_workspace(B.dct_threshold_select_workspace_bytes(n)))
        budget = k - B.read_result(sel).n_gt if use_budget else None
        ws = B.new_workspace(B.dct_dp_compress_workspace_bytes(n))
        want = _run(B.dct_dp_compress, g, e0, tau, budget, cap, workspace=ws)
        for _ in range(2):                      # two calls in a row through the built-in scratch
            got = _run(B.dct_dp_compress_static, g, e0, tau, budget, cap)
            assert got[3] == want[3]
            assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])
            assert np.array_equal(got[2], want[2])
        assert want[3].count == min(want[3].needed, cap) and want[3].needed > 0


@pytest.mark.gpu
def test_static_scratch_variant_rejects_vectors_beyond_its_limit():
    t = torch.zeros(8, device="cuda")
    i = torch.zeros(8, dtype=torch.int32, device="cuda")
    res = B.new_result()
    st = B.lib().dct_dp_compress_static(t.data_ptr(), t.data_ptr(), B.DCT_DP_COMPRESS_STATIC_MAX_N + 1, t.data_ptr(),
                                        None, i.data_ptr(), t.data_ptr(), 8, res.data_ptr(), None)
    assert st == B.DCT_ERR_UNSUPPORTED
    with pytest.raises(B.DctError):
        B.dct_dp_compress_static(t, t, B.DCT_DP_COMPRESS_STATIC_MAX_N + 1, t, None, i, t, 8, res)
    assert B.lib().dct_dp_compress_static(t.data_ptr(), t.data_ptr(), 0, t.data_ptr(), None, i.data_ptr(),
                                          t.data_ptr(), 8, res.data_ptr(), None) == B.DCT_ERR_INVALID_ARG
