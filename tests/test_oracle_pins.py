"""Pins for the CPU oracle: it is checked against things other than itself.

* hand-worked fixtures of Algorithm 1 and Algorithm 2 (tests/golden/),
* brute-force rank counting (O(n^2), no sort) on tiny inputs,
* library routines on the special cases that reduce to them
  (torch.kthvalue / torch.topk / amax / amin / take_along_dim),
* closed-form Gaussian quantiles for the synthetic workloads,
* the invariants the definitions fix (conservation, exact counts, tie rule).
"""
import numpy as np
import pytest
import torch
from scipy import stats

import oracle
from paper_2010_08899_b200 import inputs
from tests._util import read_golden, bits32, bf16_bits


# ----------------------------------------------------------------------------
# hand-worked fixtures
# ----------------------------------------------------------------------------

def test_dp_worked_example():
    g = read_golden("dct_dp_worked_example.txt")
    wg = g["w_grad"].astype(np.float32)
    e0 = g["e_grad"].astype(np.float32)
    k = int(g["k"][0])
    for full in (True, False):
        sel = oracle.dp_select(wg, e0, k, full_sort=full)
        assert float(sel.tau) == g["tau"][0]
        assert sel.n_gt == int(g["n_gt"][0]) and sel.n_eq == int(g["n_eq"][0])
    # literal mask I(|W| >= tau)
    e = e0.copy()
    r = oracle.dp_compress(wg, e, sel.tau, None, capacity=8)
    assert r.idx.tolist() == g["literal_idx"].astype(int).tolist()
    assert r.val.tolist() == g["literal_val"].tolist()
    assert e.tolist() == g["literal_e_new"].tolist()
    assert r.count == r.needed == 4
    # tie budget k - n_gt: exactly k survivors, lowest index wins
    e = e0.copy()
    r = oracle.dp_compress(wg, e, sel.tau, int(g["budget"][0]), capacity=8)
    assert r.idx.tolist() == g["budget_idx"].astype(int).tolist()
    assert r.val.tolist() == g["budget_val"].tolist()
    assert e.tolist() == g["budget_e_new"].tolist()
    assert r.count == k
    # the error-feedback sum itself
    assert (wg + e0).tolist() == g["w"].tolist()


def test_mp_worked_example():
    g = read_golden("dct_mp_worked_example.txt")
    d, k = int(g["d"][0]), int(g["k"][0])
    x = np.stack([g["x_act_0"], g["x_act_1"]]).astype(np.float32)
    gx = np.stack([g["x_grad_0"], g["x_grad_1"]]).astype(np.float32)
    assert x.shape == (2, d)
    f = oracle.mp_fwd(x, k)
    assert f.cols.tolist() == [g["cols_0"].astype(int).tolist(), g["cols_1"].astype(int).tolist()]
    assert f.vals.tolist() == [g["vals_0"].tolist(), g["vals_1"].tolist()]
    assert f.tau.tolist() == [g["tau_0"][0], g["tau_1"][0]]
    b = oracle.mp_bwd(gx, f.cols)
    assert b.tolist() == [g["gvals_0"].tolist(), g["gvals_1"].tolist()]
    # same through the bf16 entry points (all fixture values are exact in bf16)
    xb = bf16_bits(torch.from_numpy(x).to(torch.bfloat16))
    gb = bf16_bits(torch.from_numpy(gx).to(torch.bfloat16))
    fb = oracle.mp_fwd(xb, k)
    assert np.array_equal(fb.cols, f.cols)
    assert np.array_equal(fb.vals, bf16_bits(torch.from_numpy(f.vals).to(torch.bfloat16)))
    assert np.array_equal(fb.tau, bf16_bits(torch.from_numpy(f.tau).to(torch.bfloat16)))
    assert np.array_equal(oracle.mp_bwd(gb, fb.cols),
                          bf16_bits(torch.from_numpy(b).to(torch.bfloat16)))


# ----------------------------------------------------------------------------
# DP threshold select
# ----------------------------------------------------------------------------

def _brute_kth_largest(mag, k):
    """The unique v in mag with #{mag > v} < k <= #{mag >= v}; O(n^2), no sorting."""
    for v in mag:
        gt = int((mag > v).sum())
        ge = int((mag >= v).sum())
        if gt < k <= ge:
            return v, gt, ge - gt
    raise AssertionError("no order statistic found")


@pytest.mark.parametrize("n", [1, 2, 7, 64, 257])
def test_select_brute_force_every_k(n):
    rng = np.random.default_rng(n)
    # few distinct magnitudes, both signs: many ties
    g = (rng.integers(-6, 7, size=n) * 0.25).astype(np.float32)
    e = (rng.integers(-3, 4, size=n) * 0.125).astype(np.float32)
    w = (g + e).astype(np.float32)
    mag = np.abs(w)
    for k in range(1, n + 1):
        v, gt, eq = _brute_kth_largest(mag, k)
        for full in (True, False):
            s = oracle.dp_select(g, e, k, full_sort=full)
            assert float(s.tau) == float(v) and s.n_gt == gt and s.n_eq == eq
            assert s.n_gt < k <= s.n_gt + s.n_eq
            assert not np.signbit(s.tau)


def test_select_matches_library_kthvalue_and_topk():
    n = 50_000
    g = inputs.dp_gaussian(n, 11)
    e = inputs.dp_gaussian(n, 12) * 0.1
    w = (g + e).abs()
    for k in (1, 2, 50, 1000, n // 2, n - 1, n):
        s = oracle.dp_select(g.numpy(), e.numpy(), k)
        kth = torch.kthvalue(w, n - k + 1).values.item()      # k-th largest = (n-k+1)-th smallest
        top = torch.topk(w, k).values[-1].item()
        assert float(s.tau) == kth == top
    s1 = oracle.dp_select(g.numpy(), e.numpy(), 1)
    sn = oracle.dp_select(g.numpy(), e.numpy(), n)
    assert float(s1.tau) == torch.amax(w).item()
    assert float(sn.tau) == torch.amin(w).item()
    # residual absent == residual of zeros
    s0 = oracle.dp_select(g.numpy(), None, 77)
    sz = oracle.dp_select(g.numpy(), np.zeros(n, np.float32), 77)
    assert s0 == sz


def test_select_full_sort_equals_nth_element():
    for seed in range(5):
        g = inputs.quantize_mantissa(inputs.dp_gaussian(4096, seed), 3).numpy()
        for k in (1, 5, 100, 2048, 4096):
            assert oracle.dp_select(g, None, k, True) == oracle.dp_select(g, None, k, False)


def test_select_closed_form_quantiles():
    """tau on the synthetic workloads against the analytic quantile of the distribution."""
    # Gaussian: P(|z| > tau) = k/n  ->  tau = isf(k / 2n)
    n, k = 1 << 20, 1024
    g = inputs.dp_gaussian(n, 0).numpy()
    tau = float(oracle.dp_select(g, None, k).tau)
    assert tau == pytest.approx(stats.norm.isf(k / (2 * n)), rel=0.01)
    # mixture 0.99 N(0,1e-4) + 0.01 N(0,1) at density 1e-4: only the wide component reaches
    # the tail, P(|z| > tau) * 0.01 = 1e-4 -> tau = isf(0.005) = 2.576
    n = 1 << 22
    k = -(-n // 10_000)
    g = inputs.dp_mixture(n, 500).numpy()
    tau = float(oracle.dp_select(g, None, k).tau)
    assert tau == pytest.approx(stats.norm.isf(0.005), rel=0.05)
    # Student-t(3) blocks scaled by 1/sqrt(fan_in): tau solves sum_b f_b P(|t3| > tau sqrt(fan_b)) = density
    n = 1 << 22
    k = -(-n // 1000)
    scale = inputs.dlrm_like_scale(n).numpy().astype(np.float64)
    fans, counts = np.unique(np.round(1.0 / scale ** 2).astype(int), return_counts=True)
    frac = counts / n

    def tail(t):
        return float(sum(f * 2 * stats.t.sf(t * np.sqrt(fi), 3) for f, fi in zip(frac, fans)))
    lo, hi = 0.0, 10.0
    for _ in range(80):
        mid = 0.5 * (lo + hi)
        lo, hi = (mid, hi) if tail(mid) > 1e-3 else (lo, mid)
    g = inputs.dp_dlrm_like(n, 300).numpy()
    tau = float(oracle.dp_select(g, None, k).tau)
    assert tau == pytest.approx(0.5 * (lo + hi), rel=0.05)


def test_select_special_values():
    # +-0 are one magnitude; denormals order below the smallest normal; sign never matters
    g = np.array([0.0, -0.0, 1e-45, -1e-40, 1.17549435e-38, -3.0, 3.0], dtype=np.float32)
    s = oracle.dp_select(g, None, 2)
    assert float(s.tau) == 3.0 and s.n_gt == 0 and s.n_eq == 2
    s = oracle.dp_select(g, None, 3)
    assert bits32(s.tau) == bits32(np.float32(1.17549435e-38))
    s = oracle.dp_select(g, None, 4)
    assert bits32(s.tau) == bits32(np.float32(1e-40))
    s = oracle.dp_select(g, None, 7)
    assert bits32(s.tau) == 0 and s.n_eq == 2 and s.n_gt == 5
    # all-equal magnitudes with alternating signs: every k gives the same tau
    g = np.tile(np.array([2.5, -2.5], dtype=np.float32), 50)
    for k in (1, 37, 100):
        s = oracle.dp_select(g, None, k)
        assert float(s.tau) == 2.5 and s.n_gt == 0 and s.n_eq == 100
    # denormal sums are kept (no flush to zero): 1e-40 + 1e-40 is the larger of two magnitudes
    g = np.array([1e-40, 1.5e-40], dtype=np.float32)
    e = np.array([1e-40, 0.0], dtype=np.float32)
    s = oracle.dp_select(g, e, 1)
    assert bits32(s.tau) == bits32(np.float32(1e-40) + np.float32(1e-40))
    with pytest.raises(ValueError):
        oracle.dp_select(g, None, 0)
    with pytest.raises(ValueError):
        oracle.dp_select(g, None, 3)


# ----------------------------------------------------------------------------
# DP compress
# ----------------------------------------------------------------------------

def _check_compress_invariants(g, e_old, e_new, r, tau, capacity, budget=None):
    n = g.size
    w = (g + e_old).astype(np.float32)              # Algorithm 1, error feedback
    mag = np.abs(w)
    tau = np.float32(tau)
    # (i) ascending indices, (ii) survivors are at or above tau
    assert np.all(np.diff(r.idx.astype(np.int64)) > 0)
    assert np.all(np.abs(r.val) >= tau)
    # (iv) conservation, bit for bit:  scatter(idx, val) + E' == W with  E' == +0 at sent slots
    sent = np.zeros(n, dtype=np.float32)
    sent[r.idx] = r.val
    is_sent = np.zeros(n, dtype=bool)
    is_sent[r.idx] = True
    assert np.array_equal(bits32(sent)[is_sent], bits32(w)[is_sent])
    assert np.all(bits32(e_new)[is_sent] == 0)
    assert np.array_equal(bits32(e_new)[~is_sent], bits32(w)[~is_sent])
    # (v) counts
    n_ge = int((mag >= tau).sum())
    n_gt = int((mag > tau).sum())
    needed = n_ge if budget is None else n_gt + min(budget, n_ge - n_gt)
    assert r.needed == needed
    assert r.count == min(needed, capacity) == r.idx.size
    # (iii) nothing at or above tau is left behind unless the budget or the capacity kept it back
    if budget is None and needed <= capacity:
        assert np.all(np.abs(e_new) < tau) or tau == 0


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_compress_invariants_random(seed):
    n = 10_007
    g = inputs.dp_gaussian(n, seed).numpy()
    e_old = (inputs.dp_gaussian(n, 100 + seed) * 0.3).numpy()
    tau = oracle.dp_select(g, e_old, 100).tau
    for cap in (n, 100, 99, 1, 0):
        e = e_old.copy()
        r = oracle.dp_compress(g, e, tau, None, cap)
        _check_compress_invariants(g, e_old, e, r, tau, cap)
    # first `capacity` survivors in index order are the ones emitted
    e = e_old.copy()
    full = oracle.dp_compress(g, e, tau, None, n)
    e = e_old.copy()
    part = oracle.dp_compress(g, e, tau, None, 40)
    assert np.array_equal(part.idx, full.idx[:40]) and np.array_equal(part.val, full.val[:40])


def test_compress_tie_budget_gives_exactly_k():
    n = 5000
    g = inputs.quantize_mantissa(inputs.dp_gaussian(n, 5), 2).numpy()   # heavy ties
    e_old = np.zeros(n, np.float32)
    for k in (1, 10, 333, 2500, n):
        s = oracle.dp_select(g, e_old, k)
        assert k in (1, n) or s.n_eq > 1
        e = e_old.copy()
        r = oracle.dp_compress(g, e, s.tau, k - s.n_gt, n)
        assert r.count == k
        _check_compress_invariants(g, e_old, e, r, s.tau, n, budget=k - s.n_gt)
        # lowest index wins among ties: the tied survivors are the first ones in index order
        tied_all = np.flatnonzero(np.abs(g) == s.tau)
        tied_sent = r.idx[np.abs(r.val) == s.tau]
        assert np.array_equal(tied_sent, tied_all[:k - s.n_gt])
        # literal rule keeps all ties
        e = e_old.copy()
        r = oracle.dp_compress(g, e, s.tau, None, n)
        assert r.count == s.n_gt + s.n_eq


def test_compress_error_feedback_accumulates():
    """Across iterations the residual carries exactly what was not sent:
    sum of everything sent + final residual == sum of all gradients (exact in this dyadic example)."""
    n = 4096
    rng = np.random.default_rng(3)
    e = np.zeros(n, np.float32)
    total_in = np.zeros(n, np.float64)
    total_sent = np.zeros(n, np.float64)
    for it in range(6):
        g = (rng.integers(-8, 9, size=n) / 8.0).astype(np.float32)   # dyadic: every add is exact
        total_in += g
        r = oracle.dp_compress(g, e, np.float32(1.5), None, n)
        total_sent[r.idx] += r.val
    assert np.array_equal(total_sent + e, total_in)
    assert np.all(np.abs(e) < 1.5)


def test_compress_special_values():
    # -0.0 that is not sent stays -0.0; a sent slot becomes +0.0; tau = 0 sends everything, zeros included
    g = np.array([-0.0, 0.0, -2.0, 1e-40, 5.0], dtype=np.float32)
    e = np.array([-0.0, 0.0, 0.0, 1e-40, -5.0], dtype=np.float32)
    e1 = e.copy()
    r = oracle.dp_compress(g, e1, np.float32(1.0), None, 5)
    assert r.idx.tolist() == [2] and r.val.tolist() == [-2.0]
    assert bits32(e1).tolist() == [0x80000000, 0, 0, int(bits32(np.float32(1e-40) + np.float32(1e-40))[0]), 0]
    e2 = e.copy()
    r = oracle.dp_compress(g, e2, np.float32(0.0), None, 5)
    assert r.idx.tolist() == [0, 1, 2, 3, 4]
    assert bits32(r.val)[0] == 0x80000000 and np.all(bits32(e2) == 0)
    # a negative tau means its magnitude
    e3 = e.copy()
    r = oracle.dp_compress(g, e3, np.float32(-1.0), None, 5)
    assert r.idx.tolist() == [2]


# ----------------------------------------------------------------------------
# MP forward / backward
# ----------------------------------------------------------------------------

def _check_mp_row_definition(xrow_key, cols, k):
    """Definition of the row mask without sorting: exactly k columns; every kept key >= every
    dropped key; among keys equal to the threshold, kept columns all precede dropped ones."""
    d = xrow_key.size
    cols = cols.astype(np.int64)
    assert cols.size == k and np.all(np.diff(cols) > 0) and cols[0] >= 0 and cols[-1] < d
    kept = np.zeros(d, bool)
    kept[cols] = True
    tau = xrow_key[kept].min()
    if k < d:
        assert tau >= xrow_key[~kept].max()
        tied_kept = np.flatnonzero(kept & (xrow_key == tau))
        tied_drop = np.flatnonzero(~kept & (xrow_key == tau))
        if tied_drop.size:
            assert tied_kept.max() < tied_drop.min()
    return tau


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mp_fwd_definition_with_ties(dtype):
    rows, d = 64, 96
    x = inputs.mp_activations(rows, d, 7, col_scale_seed=8)
    x = inputs.quantize_mantissa(x, 2) * torch.where(inputs.dp_gaussian(rows * d, 9).view(rows, d) > 0, 1.0, -1.0)
    if dtype == "bf16":
        xa = bf16_bits(x.to(torch.bfloat16))
        key = (xa & 0x7FFF).astype(np.int64)
    else:
        xa = x.numpy()
        key = (bits32(xa) & 0x7FFFFFFF).astype(np.int64)
    for k in (1, 2, 5, 48, 95, 96):
        f = oracle.mp_fwd(xa, k)
        for i in range(rows):
            tau_key = _check_mp_row_definition(key[i], f.cols[i], k)
            assert int(f.tau[i].view(np.uint32 if dtype == "f32" else np.uint16)) == tau_key
            assert np.array_equal(f.vals[i], xa[i, f.cols[i].astype(np.int64)])


def test_mp_fwd_matches_library_topk_when_tie_free():
    rows, d, k = 128, 1000, 37
    x = inputs.dp_gaussian(rows * d, 21).view(rows, d)        # continuous: no ties, both signs
    f = oracle.mp_fwd(x.numpy(), k)
    top = torch.topk(x.abs(), k, dim=1)
    want = torch.sort(top.indices, dim=1).values.numpy()
    assert np.array_equal(f.cols.astype(np.int64), want)
    assert np.array_equal(f.tau, top.values[:, -1].numpy())
    assert np.array_equal(f.vals, torch.gather(x, 1, torch.from_numpy(want)).numpy())


def test_mp_fwd_relu_rows_with_few_nonzeros_and_padding():
    # ld > d: padding columns hold a huge value and must never be selected
    rows, d, ld, k = 32, 50, 64, 40
    x = inputs.mp_activations(rows, d, 31, ld=ld).numpy()
    assert np.all(x[:, d:] > 1e29)
    f = oracle.mp_fwd(x, k, d=d)
    assert f.cols.max() < d
    for i in range(rows):
        nz = np.flatnonzero(x[i, :d] > 0)
        assert nz.size < k                                     # ~50 % zeros, k = 80 % of d
        zeros = np.setdiff1d(np.arange(d), nz)[:k - nz.size]   # lowest-column zeros fill the rest
        assert np.array_equal(f.cols[i].astype(np.int64), np.sort(np.concatenate([nz, zeros])))
        assert f.tau[i] == 0


def test_mp_bwd_is_a_gather_and_reuses_the_mask():
    rows, d, k = 40, 200, 17
    x = inputs.mp_activations(rows, d, 41).numpy()
    gx = inputs.mp_gradients(rows, d, 42).numpy()
    f = oracle.mp_fwd(x, k)
    cols_before = f.cols.copy()
    gv = oracle.mp_bwd(gx, f.cols)
    assert np.array_equal(f.cols, cols_before)
    want = torch.take_along_dim(torch.from_numpy(gx), torch.from_numpy(f.cols.astype(np.int64)), dim=1).numpy()
    assert np.array_equal(bits32(gv), bits32(want))
    # dense reconstruction: scattering the packed gradients back gives X_grad .* M, whose support lies inside the
    # mask of X_act .* M and which agrees with X_grad on every kept column
    m_f = np.zeros((rows, d), bool)
    np.put_along_axis(m_f, f.cols.astype(np.int64), True, axis=1)
    assert np.all(m_f.sum(1) == k)
    dense_b = np.zeros((rows, d), np.float32)
    np.put_along_axis(dense_b, f.cols.astype(np.int64), gv, axis=1)
    assert np.array_equal(bits32(dense_b), bits32(np.where(m_f, gx, np.float32(0))))
    assert not np.any((dense_b != 0) & ~m_f)
    # bf16
    gb = bf16_bits(torch.from_numpy(gx).to(torch.bfloat16))
    assert np.array_equal(oracle.mp_bwd(gb, f.cols), np.take_along_axis(gb, f.cols.astype(np.int64), axis=1))
    # a column outside the row is refused
    bad = f.cols.copy()
    bad[0, 0] = d
    with pytest.raises(ValueError):
        oracle.mp_bwd(gx, bad)


def test_mp_invalid_arguments():
    x = np.zeros((2, 8), np.float32)
    with pytest.raises(ValueError):
        oracle.mp_fwd(x, 0)
    with pytest.raises(ValueError):
        oracle.mp_fwd(x, 9)
