"""Threshold life-span L = 1 (select and compress the same vector, exactly k survivors) against the
oracle's select followed by its compress with the tie budget k - n_gt."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import binding as B
from paper_2010_08899_b200 import inputs
from tests._util import bits32

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [1, 77, 4096, 50_001, (1 << 20) + 3])
def test_l1_mode_keeps_exactly_k(n):
    g_dev = inputs.quantize_mantissa(inputs.dp_gaussian(n, 31 + n % 7, "cuda"), 6)    # ties are common
    e_dev = inputs.quantize_mantissa(inputs.dp_gaussian(n, 41 + n % 5, "cuda") * 0.25, 6)
    ws = B.new_workspace(B.dct_dp_select_compress_workspace_bytes(n))
    e = e_dev.clone()
    e_ref = e_dev.cpu().numpy().copy()
    for it, k in enumerate(sorted({1, max(1, n // 50), max(1, n // 2), n})):
        for cap in (n, max(1, k - 1)):
            e_run, e_want = e.clone(), e_ref.copy()
            idx = torch.full((cap + 4,), -1, dtype=torch.int32, device="cuda")
            val = torch.full((cap + 4,), -1.0, device="cuda")
            tau, res = torch.zeros(1, device="cuda"), B.new_result()
            B.dct_dp_select_compress(g_dev, e_run, n, k, tau, idx, val, cap, res, ws)
            r = B.read_result(res)
            s = oracle.dp_select(g_dev.cpu().numpy(), e_want, k)
            w = oracle.dp_compress(g_dev.cpu().numpy(), e_want, s.tau, k - s.n_gt, cap)
            assert bits32(tau.cpu().numpy())[0] == bits32(s.tau)[0]
            assert (r.n_gt, r.n_eq, r.needed, r.count) == (s.n_gt, s.n_eq, k, min(k, cap))
            assert r.status == (B.DCT_OK if cap >= k else B.DCT_ERR_CAPACITY)
            assert np.array_equal(idx[:r.count].cpu().numpy(), w.idx)
            assert np.array_equal(bits32(val[:r.count].cpu().numpy()), bits32(w.val))
            assert np.array_equal(bits32(e_run.cpu().numpy()), bits32(e_want))
            assert bool((idx[cap:] == -1).all())
