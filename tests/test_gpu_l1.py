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


def _check_l1(g_dev, e_dev, n, k, cap, ws, name=""):
    e_run = e_dev.clone()
    e_want = e_dev.cpu().numpy().copy()
    g_host = g_dev.cpu().numpy()
    idx = torch.full((cap + 4,), -1, dtype=torch.int32, device="cuda")
    val = torch.full((cap + 4,), -1.0, device="cuda")
    tau, res = torch.zeros(1, device="cuda"), B.new_result()
    B.dct_dp_select_compress(g_dev, e_run, n, k, tau, idx, val, cap, res, ws)
    r = B.read_result(res)
    s = oracle.dp_select(g_host, e_want, k)
    w = oracle.dp_compress(g_host, e_want, s.tau, k - s.n_gt, cap)
    assert bits32(tau.cpu().numpy())[0] == bits32(s.tau)[0], name
    assert (r.n_gt, r.n_eq, r.needed, r.count) == (s.n_gt, s.n_eq, k, min(k, cap)), name
    assert r.status == (B.DCT_OK if cap >= k else B.DCT_ERR_CAPACITY), name
    assert np.array_equal(idx[:r.count].cpu().numpy(), w.idx), name
    assert np.array_equal(bits32(val[:r.count].cpu().numpy()), bits32(w.val)), name
    assert np.array_equal(bits32(e_run.cpu().numpy()), bits32(e_want)), name
    assert bool((idx[cap:] == -1).all()), name
    return e_run


def test_l1_one_pass_path_and_its_fallbacks():
    """From 2^25 elements the vector is streamed once: candidates above a sampled bound, exact select over them, a
    pass over the candidates.  The sample only steers: when it misjudges the vector (too few candidates, or more
    than the list holds) the plain select and compress run on the summed vector, with the same result."""
    n = (1 << 25) + 999
    stride = (n // (1 << 17)) & ~7
    sampled = (torch.arange(1 << 17, device="cuda")[:, None] * stride + torch.arange(8, device="cuda")[None, :]).reshape(-1)
    ws = B.new_workspace(B.dct_dp_select_compress_workspace_bytes(n))
    e0 = inputs.dp_gaussian(n, 71, "cuda") * 0.25
    base = inputs.dp_mixture(n, 90, "cuda")
    # (gradient, error, k, capacity)
    cases = {"iid, sparse k": (base, e0 * 0.01, 3356, 4000),
             "iid, capacity below k": (base, e0 * 0.01, 3356, 3000),
             "two iterations in a row": None,
             "heavy ties": (inputs.quantize_mantissa(inputs.dp_gaussian(n, 72, "cuda"), 3),
                            inputs.quantize_mantissa(e0, 3), 20_000, 20_000),
             "dense k: two operators": (base, e0 * 0.01, n // 4, n // 4)}
    big = inputs.dp_gaussian(n, 91, "cuda")
    big[sampled] = 1000.0 + inputs.dp_gaussian(sampled.numel(), 92, "cuda")
    cases["sample overestimates: too few candidates"] = (big, torch.zeros(n, device="cuda"), 10_000, 12_000)
    low = inputs.dp_gaussian(n, 93, "cuda")
    low[sampled] = 0.0
    cases["sample underestimates: the list overflows"] = (low, torch.zeros(n, device="cuda"), 5_000, 5_000)
    for name, case in cases.items():
        if case is None:
            e1 = _check_l1(base, e0 * 0.01, n, 3356, 4000, ws, name)          # the error of one call feeds the next
            _check_l1(inputs.dp_mixture(n, 94, "cuda"), e1, n, 3356, 4000, ws, name)
            continue
        g, e, k, cap = case
        _check_l1(g, e, n, k, cap, ws, name)


def test_l1_one_pass_unaligned_vectors():
    n = (1 << 25) + 5
    g = inputs.dp_mixture(n + 3, 95, "cuda")[3:]                              # 12 bytes off a 16-byte boundary
    e = (inputs.dp_gaussian(n + 1, 96, "cuda") * 0.001)[1:]
    ws = B.new_workspace(B.dct_dp_select_compress_workspace_bytes(n))
    _check_l1(g, e, n, 4000, 4096, ws)
