"""dct_dp_compress_static: the workspace-free variant of dct_dp_compress.

Collected last on purpose (file name), so that a run that stops at the first failure has already
gone through every other test.  The variant keeps its tile descriptors in an array built into the
library, for callers that cannot allocate device memory themselves (hooks running inside a framework
whose allocator owns the GPU).  It must give bit-identical results to the workspace version and to the
CPU oracle, also on a second call that finds the array full of the first call's leftovers, and it must
leave the amount of free device memory where it was."""
import numpy as np
import pytest
import torch

import oracle
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
        # and against the oracle directly
        e_h = e0.cpu().numpy().copy()
        o = oracle.dp_compress(g.cpu().numpy(), e_h, float(tau.cpu()), budget, cap)
        assert (got[3].count, got[3].needed) == (o.count, o.needed)
        assert np.array_equal(got[0][:o.count], o.idx) and np.array_equal(got[1][:o.count], o.val.view(np.uint32))
        assert np.array_equal(got[2], e_h.view(np.uint32))


@pytest.mark.gpu
@pytest.mark.parametrize("n", [B.DCT_DP_COMPRESS_STATIC_MAX_N, B.DCT_DP_COMPRESS_STATIC_MAX_N - 1234])
def test_static_scratch_variant_at_its_size_limit_allocates_nothing(n):
    """The largest vectors the built-in array serves (its last descriptors are in use), checked against the
    oracle; the second call must leave the free device memory exactly where it found it."""
    g = inputs.dp_mixture(n, 7, "cuda")
    e = inputs.dp_gaussian(n, 8, "cuda") * 0.001
    k = B.k_from_density(n, 1, 10_000)
    cap = 4 * k
    tau = torch.zeros(1, device="cuda")
    sel = B.new_result()
    B.dct_threshold_select(g, e, n, k, tau, sel, B.new_workspace(B.dct_threshold_select_workspace_bytes(n)))
    idx = torch.full((cap + 16,), -3, dtype=torch.int32, device="cuda")
    val = torch.full((cap + 16,), -3.0, device="cuda")
    res = B.new_result()
    g_h, e_h = g.cpu().numpy(), e.cpu().numpy().copy()
    e_first = e.clone()
    B.dct_dp_compress_static(g, e_first, n, tau, None, idx, val, cap, res)      # first call on the device: set-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    B.dct_dp_compress_static(g, e, n, tau, None, idx, val, cap, res)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    r = B.read_result(res)
    o = oracle.dp_compress(g_h, e_h, float(tau.cpu()), None, cap)
    assert r.status == B.DCT_OK and (r.count, r.needed) == (o.count, o.needed) and r.count >= k
    assert np.array_equal(idx[:r.count].cpu().numpy(), o.idx)
    assert np.array_equal(val[:r.count].cpu().numpy().view(np.uint32), o.val.view(np.uint32))
    assert np.array_equal(e.cpu().numpy().view(np.uint32), e_h.view(np.uint32))
    assert torch.equal(e, e_first)
    assert bool((idx[cap:] == -3).all())


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
