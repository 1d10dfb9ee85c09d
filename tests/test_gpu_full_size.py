"""Parity at the full sizes of the large configurations, in the launch configuration bench.py times.
The CPU oracle is slow at these sizes, so the number of compared iterations is small; every compared
output is still checked element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import binding as B
from paper_2010_08899_b200 import inputs
from tests import _gpu as G
from tests._util import bits32

pytestmark = pytest.mark.gpu


def _run_dp_config(gen, n, k, sel_seed, iter_seeds, capacity):
    g_sel = gen(n, sel_seed, G.DEV)
    tau_dev, r = G.select(g_sel, None, k)
    want = oracle.dp_select(g_sel.cpu().numpy(), None, k)
    assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0]
    assert (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq) and r.n_gt < k <= r.n_gt + r.n_eq
    del g_sel
    e_dev = torch.zeros(n, device=G.DEV)
    e = np.zeros(n, np.float32)
    ws = B.new_workspace(B.dct_dp_compress_workspace_bytes(n))
    counts = []
    for seed in iter_seeds:
        g_dev = gen(n, seed, G.DEV)
        w = oracle.dp_compress(g_dev.cpu().numpy(), e, want.tau, None, capacity)
        idx, val, rr = G.compress(g_dev, e_dev, tau_dev, None, capacity, ws=ws)
        assert rr.status == B.DCT_OK and rr.count == w.count == rr.needed == w.needed
        assert np.array_equal(idx, w.idx) and np.array_equal(bits32(val), bits32(w.val))
        assert np.array_equal(bits32(e_dev.cpu().numpy()), bits32(e))
        counts.append(rr.count)
        del g_dev
    return float(want.tau), counts


def test_config3_dp_dlrm_scale():
    """64 Mi fp32 gradients, DLRM-like blocks, Student-t(3)/sqrt(fan_in), density 0.1 %."""
    n = 64 << 20
    k = B.k_from_density(n, 1, 1000)
    assert k == 67_109
    tau, counts = _run_dp_config(inputs.dp_dlrm_like, n, k, 300, [301, 302, 303], n // 32)
    assert tau == pytest.approx(0.44, rel=0.1)
    assert counts[0] == pytest.approx(k, rel=0.05) and counts[-1] > counts[0]


def test_config5_dp_large():
    """2^30 fp32 gradients (4 GiB), mixture 0.99 N(0,1e-4) + 0.01 N(0,1), density 0.01 %."""
    n = 1 << 30
    k = B.k_from_density(n, 1, 10_000)
    assert k == 107_375
    tau, counts = _run_dp_config(inputs.dp_mixture, n, k, 500, [501, 502], n // 256)
    assert tau == pytest.approx(2.576, rel=0.02)
    assert counts[0] == pytest.approx(k, rel=0.05)
