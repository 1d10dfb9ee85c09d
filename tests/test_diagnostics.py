"""Threshold diagnostics (Sec. 2.1 threshold plot, Sec. 2.2 mean-threshold plot, drift guard).

CPU part: the oracle functions pinned against things other than themselves (numpy partition / sort,
torch.topk, exact rational arithmetic, hand cases).  GPU part: the CUDA entry points against the oracle,
bit for bit (thresholds, counts) and to the stated bound (the binary64 mean)."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import inputs
from tests._util import bf16_bits


def _as_bf16_values(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


# ---------------------------------------------------------------------------------------------
# oracle pins (CPU)
# ---------------------------------------------------------------------------------------------

def test_oracle_select_multi_against_numpy_order_statistics():
    rng = np.random.default_rng(5)
    for n in (1, 7, 1000, 65537):
        g = rng.standard_normal(n).astype(np.float32)
        e = (0.1 * rng.standard_normal(n)).astype(np.float32)
        w = np.abs(g + e)                                  # one fp32 add, then the magnitude
        ks = sorted({1, max(1, n // 20), max(1, n // 10), max(1, n // 4), n})
        ks = ks[:4]
        r = oracle.dp_select_multi(g, e, ks)
        part = np.sort(w)                                  # ascending
        for q, k in enumerate(ks):
            assert r.tau[q] == part[n - k]
            assert int(r.n_gt[q]) == int((w > part[n - k]).sum())
            assert int(r.n_eq[q]) == int((w == part[n - k]).sum())
            assert int(r.n_gt[q]) < k <= int(r.n_gt[q]) + int(r.n_eq[q])


def test_oracle_select_multi_is_monotone_and_matches_closed_form_quantiles():
    # |N(0,1)|: the k-th largest of n sits at the (1 - k/n) quantile of the half-normal
    from scipy import stats
    n = 1 << 20
    g = inputs.dp_gaussian(n, 3, "cpu").numpy()
    ks = [n // 4, n // 10, n // 20]                        # 75 / 90 / 95 % sparsity, the paper's levels
    r = oracle.dp_select_multi(g, None, ks)
    assert r.tau[0] < r.tau[1] < r.tau[2]                  # the threshold grows with the sparsity
    for q, k in enumerate(ks):
        want = stats.halfnorm.ppf(1.0 - k / n)
        assert abs(float(r.tau[q]) - want) < 0.01


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_oracle_threshold_mean_against_topk_and_exact_rational_mean(dtype):
    rows, d = 37, 300
    x = inputs.mp_activations(rows, d, 11, dtype=torch.float32 if dtype == "f32" else torch.bfloat16,
                              device="cpu", col_scale_seed=12)
    sign = torch.where(inputs.dp_gaussian(rows * d, 13, "cpu").view(rows, d) > 0, 1.0, -1.0).to(x.dtype)
    x = (x * sign).contiguous()
    ks = [75, 30, 15, 1]
    xo = x.numpy() if dtype == "f32" else bf16_bits(x)
    r = oracle.mp_threshold_mean(xo, ks)
    for q, k in enumerate(ks):
        want = torch.topk(x.abs().float(), k, dim=1).values[:, -1].numpy()        # k-th largest magnitude
        got = r.tau[q] if dtype == "f32" else _as_bf16_values(r.tau[q])
        assert np.array_equal(got, want)
        exact = sum(Fraction(float(v)) for v in want) / rows                      # exact rational mean
        assert abs(Fraction(float(r.mean[q])) - exact) <= abs(exact) * Fraction(rows, 2 ** 52)
    assert r.mean[0] <= r.mean[1] <= r.mean[2] <= r.mean[3]


def test_oracle_threshold_mean_hand_case():
    # rows (1, -4, 2, 0) and (3, 0, 0, -1): 2nd largest magnitudes 2 and 1 -> mean 1.5; largest 4 and 3 -> 3.5
    x = np.array([[1, -4, 2, 0], [3, 0, 0, -1]], dtype=np.float32)
    r = oracle.mp_threshold_mean(x, [2, 1, 4])
    assert r.mean.tolist() == [1.5, 3.5, 0.0]
    assert r.tau.tolist() == [[2.0, 1.0], [4.0, 3.0], [0.0, 0.0]]


def test_oracle_drift_flag_cases():
    # ratio 5/4: inside while 80 <= needed <= 125 for k = 100
    assert [oracle.dp_drift_flag(v, 100, 5, 4) for v in (0, 79, 80, 100, 125, 126, 10 ** 9)] == [2, 2, 0, 0, 0, 1, 1]
    assert oracle.dp_drift_flag(7, 7, 1, 1) == 0 and oracle.dp_drift_flag(8, 7, 1, 1) == 1
    big = 2 ** 31 - 1
    assert oracle.dp_drift_flag(big, big, 2 ** 32 - 1, 2 ** 32 - 1) == 0        # no overflow in the products


# ---------------------------------------------------------------------------------------------
# CUDA path against the oracle (GPU)
# ---------------------------------------------------------------------------------------------

def _gpu():
    from paper_2010_08899_b200 import binding as B
    from tests import _gpu as G
    return B, G


def _select_multi(g, e, ks):
    B, G = _gpu()
    n, m = g.numel(), len(ks)
    tau = torch.full((m + 8,), -7.0, device=G.DEV)
    res = torch.zeros(5 * m, dtype=torch.int64, device=G.DEV)
    ws = B.new_workspace(B.dct_threshold_select_multi_workspace_bytes(n, m))
    B.dct_threshold_select_multi(g, e, n, ks, tau, res, ws)
    assert bool((tau[m:] == -7.0).all())
    out = [B.read_result(res[5 * q: 5 * q + 5]) for q in range(m)]
    return tau[:m].cpu().numpy(), out


@pytest.mark.gpu
@pytest.mark.parametrize("n", [1, 5, 8191, 8192, 100003, (1 << 22) + 17])
def test_gpu_select_multi_matches_oracle(n):
    B, G = _gpu()
    g = inputs.dp_dlrm_like(n, 21, G.DEV) if n > 1000 else inputs.dp_gaussian(n, 21, G.DEV)
    e = 0.25 * inputs.dp_gaussian(n, 22, G.DEV)
    ks = sorted({max(1, n // 4), max(1, n // 10), max(1, n // 20), max(1, n // 1000)}, reverse=True)
    for resid in (None, e):
        tau, res = _select_multi(g, resid, ks)
        want = oracle.dp_select_multi(g.cpu().numpy(), None if resid is None else resid.cpu().numpy(), ks)
        assert np.array_equal(tau.view(np.uint32), want.tau.view(np.uint32))
        for q in range(len(ks)):
            assert res[q].status == B.DCT_OK
            assert (res[q].n_gt, res[q].n_eq) == (int(want.n_gt[q]), int(want.n_eq[q]))


@pytest.mark.gpu
def test_gpu_select_multi_equals_single_select_with_ties_and_unaligned_input():
    B, G = _gpu()
    n = 300001
    g = inputs.quantize_mantissa(inputs.dp_gaussian(n + 1, 31, G.DEV), 3)[1:]      # 4-byte aligned only, heavy ties
    ks = [n // 20, n // 4, 1, n]                                                  # any order, both extremes
    tau, res = _select_multi(g, None, ks)
    for q, k in enumerate(ks):
        t1, r1 = G.select(g, None, k)
        assert tau[q] == float(t1[0])
        assert (res[q].n_gt, res[q].n_eq) == (r1.n_gt, r1.n_eq)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("rows,d,ld", [(1, 1, 1), (33, 301, 304), (2048, 1024, 1024), (700, 4096, 4096), (3, 32768, 32768),
                                       (5, 12287, 12288)])
def test_gpu_threshold_mean_matches_oracle(dtype, rows, d, ld):
    B, G = _gpu()
    x = inputs.mp_activations(rows, d, 41, dtype=dtype, device=G.DEV, col_scale_seed=42, ld=ld)
    ks = sorted({max(1, d // 4), max(1, d // 10), max(1, d // 20), 1}, reverse=True)
    m = len(ks)
    mean = torch.full((m + 4,), -1.0, dtype=torch.float64, device=G.DEV)
    tau = torch.zeros(m * rows + 16, dtype=dtype, device=G.DEV)
    B.dct_mp_threshold_mean(x, rows, d, ld, ks, mean, tau)
    want = oracle.mp_threshold_mean(G.to_oracle(x), ks, d=d)
    got_tau = G.as_np_bits(tau[: m * rows]).reshape(m, rows)
    assert np.array_equal(got_tau, want.tau.view(got_tau.dtype))
    assert bool((mean[m:] == -1.0).all()) and bool((tau[m * rows:] == 0).all())
    got = mean[:m].cpu().numpy()
    # thresholds of one batch lie within a few binades: every partial sum is exact in binary64, in any order
    assert np.array_equal(got, want.mean)
    # and the per-row thresholds are those of the forward pack
    _, _, tau_fwd, _ = G.mp_fwd(x, d, ks[0])
    assert np.array_equal(G.as_np_bits(tau_fwd), got_tau[0])


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("ks", [[205, 2048], [2048, 205], [1500, 410, 7]])
def test_gpu_threshold_mean_levels_inside_and_outside_the_fast_kernels(dtype, ks):
    """Levels up to 3/8 of the row are found by the forward kernels run for their thresholds alone; a level beyond
    that sends the whole call to the general kernel, whichever position it has in the list."""
    B, G = _gpu()
    rows, d = 333, 4096
    x = inputs.mp_activations(rows, d, 43, dtype=dtype, device=G.DEV, col_scale_seed=44)
    x[5] = 0
    x[6, 100:] = 0
    m = len(ks)
    mean = torch.zeros(m, dtype=torch.float64, device=G.DEV)
    tau = torch.zeros(m * rows, dtype=dtype, device=G.DEV)
    B.dct_mp_threshold_mean(x, rows, d, d, ks, mean, tau)
    want = oracle.mp_threshold_mean(G.to_oracle(x), ks, d=d)
    got_tau = G.as_np_bits(tau).reshape(m, rows)
    assert np.array_equal(got_tau, want.tau.view(got_tau.dtype))
    assert np.array_equal(mean.cpu().numpy(), want.mean)


@pytest.mark.gpu
def test_gpu_threshold_mean_inexact_sum_stays_within_the_stated_bound():
    B, G = _gpu()
    rows, d = 4096, 64
    x = inputs.mp_activations(rows, d, 51, device=G.DEV)
    scale = torch.pow(2.0, torch.arange(rows, device=G.DEV) % 97 - 48.0)          # thresholds spread over 97 binades
    x = (x * scale[:, None]).contiguous()
    ks = [8]
    mean = torch.zeros(1, dtype=torch.float64, device=G.DEV)
    tau = torch.zeros(rows, device=G.DEV)
    B.dct_mp_threshold_mean(x, rows, d, d, ks, mean, tau)
    want = oracle.mp_threshold_mean(x.cpu().numpy(), ks)
    assert np.array_equal(tau.cpu().numpy(), want.tau[0])
    exact = sum(Fraction(float(v)) for v in want.tau[0]) / rows
    for v in (float(mean[0]), float(want.mean[0])):
        assert abs(Fraction(v) - exact) <= exact * Fraction(rows, 2 ** 53)
    again = torch.zeros(1, dtype=torch.float64, device=G.DEV)
    B.dct_mp_threshold_mean(x, rows, d, d, ks, again, tau)
    assert float(again[0]) == float(mean[0])                                      # fixed order: same bits


@pytest.mark.gpu
def test_gpu_drift_check_follows_a_reused_threshold():
    """tau selected once and reused while the residual builds up: the survivor count climbs away from k
    and the check reports it, on the device."""
    B, G = _gpu()
    n, k = 1 << 20, 1024
    tau, r = G.select(inputs.dp_gaussian(n, 60, G.DEV), None, k)
    e = torch.zeros(n, device=G.DEV)
    idx = torch.empty(n // 8, dtype=torch.int32, device=G.DEV)
    val = torch.empty(n // 8, device=G.DEV)
    res = B.new_result()
    ws = B.new_workspace(B.dct_dp_compress_workspace_bytes(n))
    flag = torch.full((2,), 9, dtype=torch.int32, device=G.DEV)
    seen = []
    for it in range(6):
        g = inputs.dp_gaussian(n, 61 + it, G.DEV)
        B.dct_dp_compress(g, e, n, tau, None, idx, val, n // 8, res, ws)
        B.dct_dp_drift_check(res, k, 5, 4, flag)
        needed = B.read_result(res).needed
        assert int(flag[0]) == oracle.dp_drift_flag(needed, k, 5, 4) and int(flag[1]) == 9
        seen.append(int(flag[0]))
    assert seen[0] == 0 and seen[-1] == 1
    for needed, want in ((0, 2), (k, 0)):
        fake = torch.tensor([0, needed, needed, 0, 0], dtype=torch.int64, device=G.DEV)
        B.dct_dp_drift_check(fake, k, 5, 4, flag)
        assert int(flag[0]) == want


@pytest.mark.gpu
def test_gpu_diagnostics_reject_bad_arguments():
    B, G = _gpu()
    g = inputs.dp_gaussian(100, 1, G.DEV)
    tau = torch.zeros(8, device=G.DEV)
    res = torch.zeros(40, dtype=torch.int64, device=G.DEV)
    ws = B.new_workspace(B.dct_threshold_select_multi_workspace_bytes(100, 4))
    for ks in ([], [1, 2, 3, 4, 5], [0], [101]):
        with pytest.raises(B.DctError):
            B.dct_threshold_select_multi(g, None, 100, ks, tau, res, ws)
    with pytest.raises(B.DctError):
        B.dct_threshold_select_multi(g, None, 100, [5], tau, res, ws[:256])
    x = inputs.mp_activations(4, 16, 1, device=G.DEV)
    mean = torch.zeros(4, dtype=torch.float64, device=G.DEV)
    t = torch.zeros(64, device=G.DEV)
    for ks in ([], [0], [17]):
        with pytest.raises(B.DctError):
            B.dct_mp_threshold_mean(x, 4, 16, 16, ks, mean, t)
    flag = torch.zeros(1, dtype=torch.int32, device=G.DEV)
    for num, den in ((3, 4), (1, 0)):
        with pytest.raises(B.DctError):
            B.dct_dp_drift_check(B.new_result(), 10, num, den, flag)
