"""GPU parity of DCT-DP (threshold select, hard threshold + error feedback + compaction)
against the CPU oracle: bit-exact on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import binding as B
from paper_2010_08899_b200 import inputs
from tests import _gpu as G
from tests._util import bits32

pytestmark = pytest.mark.gpu

SIZES = [1, 2, 3, 31, 127, 4095, 4096, 4097, 8193, 12345, 100003, (1 << 18) + 5]


def _compare_compress(g_dev, e_dev, tau_dev, budget, capacity):
    """Run both sides from the same (g, e_old); e_dev is updated in place. Returns the GPU result."""
    g = g_dev.cpu().numpy()
    e = e_dev.cpu().numpy().copy()
    tau = tau_dev.cpu().numpy()[0]
    want = oracle.dp_compress(g, e, tau, budget, capacity)
    idx, val, r = G.compress(g_dev, e_dev, tau_dev, budget, capacity)
    assert r.needed == want.needed and r.count == want.count
    assert r.status == (B.DCT_ERR_CAPACITY if want.needed > capacity else B.DCT_OK)
    assert np.array_equal(idx, want.idx)
    assert np.array_equal(bits32(val), bits32(want.val))
    assert np.array_equal(bits32(e_dev.cpu().numpy()), bits32(e))
    return r


@pytest.mark.parametrize("n", SIZES)
def test_select_and_compress_odd_sizes(n):
    g_dev = inputs.dp_gaussian(n, 1000 + n, G.DEV)
    e_dev = inputs.dp_gaussian(n, 2000 + n, G.DEV) * 0.25
    g, e = g_dev.cpu().numpy(), e_dev.cpu().numpy()
    for k in sorted({1, min(n, 2), max(1, n // 1000), max(1, n // 20), max(1, n // 2), n}):
        for res_dev, res in ((None, None), (e_dev, e)):
            tau_dev, r = G.select(g_dev, res_dev, k)
            want = oracle.dp_select(g, res, k)
            assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0]
            assert (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq)
        # compress with the threshold of (g + e), literal rule and exact-k rule
        for budget in (None, k - want.n_gt):
            for cap in sorted({n, max(want.n_gt + want.n_eq - 1, 0), 0}):
                ee = e_dev.clone()
                _compare_compress(g_dev, ee, tau_dev, budget, cap)


@pytest.mark.parametrize("offset", [1, 2, 3])
def test_misaligned_pointers(offset):
    n = 20_001
    g_dev = G.offset_copy(inputs.dp_gaussian(n, 5, G.DEV), offset)
    e_dev = G.offset_copy(inputs.dp_gaussian(n, 6, G.DEV), (offset + 1) % 4)
    assert g_dev.data_ptr() % 16 != 0
    k = 200
    tau_dev, r = G.select(g_dev, e_dev, k)
    want = oracle.dp_select(g_dev.cpu().numpy(), e_dev.cpu().numpy(), k)
    assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0] and (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq)
    _compare_compress(g_dev, e_dev, tau_dev, None, n)


@pytest.mark.parametrize("offset", [1, 2, 3])
@pytest.mark.parametrize("n", [3, 4093, 4096, 20_001, 3 * 4096 - 2, (1 << 21) + 7])
def test_gradient_and_residual_at_the_same_odd_offset(offset, n):
    """Views at the same element offset into two flat buffers: both vectors sit 4, 8 or 12 bytes past a 16-byte
    boundary.  The elements next to them in the buffers (before the first, after the last) are left alone, the
    indices count from the vector's own first element, ties and a capacity that cuts the list off work as ever."""
    gbuf = inputs.dp_gaussian(n + 8, 15 + n % 7, G.DEV)
    ebuf = inputs.dp_gaussian(n + 8, 16 + n % 5, G.DEV) * 0.5
    if n > 1000:
        gbuf = inputs.quantize_mantissa(gbuf, 4)
        ebuf = torch.zeros_like(ebuf)
    g_dev, e_view = gbuf[offset:offset + n], ebuf[offset:offset + n]
    assert g_dev.data_ptr() % 16 == 4 * offset and e_view.data_ptr() % 16 == 4 * offset
    around = ebuf.clone()
    for k in sorted({1, max(1, n // 50), n}):
        tau_dev, r = G.select(g_dev, e_view, k)
        want = oracle.dp_select(g_dev.cpu().numpy(), e_view.cpu().numpy(), k)
        assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0] and (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq)
        for budget, cap in ((None, n), (k - r.n_gt, n), (None, max(1, k // 2))):
            ebuf.copy_(around)
            _compare_compress(g_dev, e_view, tau_dev, budget, cap)
            assert torch.equal(ebuf[:offset], around[:offset]) and torch.equal(ebuf[offset + n:], around[offset + n:])


def test_heavy_ties_and_exact_k():
    n = 300_000
    g_dev = inputs.quantize_mantissa(inputs.dp_gaussian(n, 77, G.DEV), 2)
    e_dev = torch.zeros(n, device=G.DEV)
    g = g_dev.cpu().numpy()
    for k in (1, 10, 3000, n // 3, n):
        tau_dev, r = G.select(g_dev, None, k)
        want = oracle.dp_select(g, None, k)
        assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0] and (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq)
        ee = e_dev.clone()
        rr = _compare_compress(g_dev, ee, tau_dev, k - r.n_gt, n)
        assert rr.count == k                                   # exactly k survivors with the tie budget
        ee = e_dev.clone()
        rr = _compare_compress(g_dev, ee, tau_dev, None, n)
        assert rr.count == r.n_gt + r.n_eq                     # the literal mask keeps every tie
        ee = e_dev.clone()
        _compare_compress(g_dev, ee, tau_dev, 0, n)            # budget 0: strictly-greater only


@pytest.mark.parametrize("kind", ["gaussian", "dense_and_sparse_stretches", "ties"])
def test_dense_survivors_many_tiles_per_cta(kind):
    """Every persistent CTA takes a dozen tiles and most tiles have hundreds to thousands of survivors: the
    shared-memory ring wraps, fills up (the compute warps wait for their drain warps and count the tiles they
    hold ahead of their turn) and carries tiles of every density up to all 4096 elements."""
    n = (1 << 24) + 4096 + 3
    g_dev = inputs.dp_gaussian(n, 31, G.DEV)
    if kind == "dense_and_sparse_stretches":                   # stretches of 1..40 tiles, alternately scaled up and down
        gen = torch.Generator().manual_seed(5)
        edges = torch.cumsum(torch.randint(1, 41, (2000,), generator=gen) * 4096, 0)
        scale = torch.ones(n)
        lo = 0
        for j, hi in enumerate(edges.tolist()):
            if lo >= n:
                break
            scale[lo:hi] = 8.0 if j % 2 else 0.05
            lo = hi
        g_dev = g_dev * scale.to(G.DEV)
    if kind == "ties":
        g_dev = inputs.quantize_mantissa(g_dev, 1)
    e0 = inputs.dp_gaussian(n, 32, G.DEV) * 0.3
    if kind == "ties":
        e0 = torch.zeros(n, device=G.DEV)
    g = g_dev.cpu().numpy()
    for k in (n // 8, n // 4, n // 2, n):
        tau_dev, r = G.select(g_dev, e0, k)
        want = oracle.dp_select(g, e0.cpu().numpy(), k)
        assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0] and (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq)
        _compare_compress(g_dev, e0.clone(), tau_dev, None, n)
        if kind == "ties":
            rr = _compare_compress(g_dev, e0.clone(), tau_dev, k - r.n_gt, n)
            assert rr.count == k
    # an output that is too small: the survivors past the capacity go back into the residual, by the million
    tau_dev, r = G.select(g_dev, e0, n // 4)
    rr = _compare_compress(g_dev, e0.clone(), tau_dev, None, n // 16)
    assert rr.status == B.DCT_ERR_CAPACITY and rr.count == n // 16


def test_dense_survivors_with_error_feedback_over_iterations():
    """A threshold of 5 % kept over eight iterations: the residual fills up and about 15 % of the elements pass."""
    n = (1 << 23) + 100
    g0 = inputs.dp_gaussian(n, 40, G.DEV)
    tau_dev, _ = G.select(g0, None, n // 20)
    e_dev = torch.zeros(n, device=G.DEV)
    counts = []
    for t in range(8):
        g_dev = inputs.dp_gaussian(n, 41 + t, G.DEV)
        counts.append(_compare_compress(g_dev, e_dev, tau_dev, None, n).count)
    assert counts[0] == pytest.approx(n / 20, rel=0.05) and counts[-1] > 2.5 * counts[0]


def test_degenerate_vectors():
    n = 10_000
    cases = {
        "all_equal": torch.full((n,), 2.5),
        "alternating_sign": torch.tensor([1.25, -1.25]).repeat(n // 2),
        "all_zero": torch.zeros(n),
        "signed_zeros": torch.tensor([0.0, -0.0]).repeat(n // 2),
        "denormals": torch.arange(n, dtype=torch.float32) * 1e-42 * torch.tensor([1.0, -1.0]).repeat(n // 2),
        "one_outlier": torch.cat([torch.full((n - 1,), 1e-3), torch.tensor([1e30])]),
    }
    for name, g_cpu in cases.items():
        g_dev = g_cpu.to(G.DEV)
        for e_cpu in (torch.zeros(n), g_cpu.flip(0) * 0.5):
            e_dev = e_cpu.to(G.DEV)
            for k in (1, 17, n // 2, n):
                tau_dev, r = G.select(g_dev, e_dev, k)
                want = oracle.dp_select(g_cpu.numpy(), e_cpu.numpy(), k)
                assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0], name
                assert (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq), name
                for budget in (None, k - r.n_gt):
                    for cap in (n, 5):
                        _compare_compress(g_dev, e_dev.clone(), tau_dev, budget, cap)


def test_config1_dp_tiny():
    """N = 2^20 ~ N(0,1), k = 1024: one select, then 8 compress iterations with error feedback."""
    n, k = 1 << 20, 1024
    g0 = inputs.dp_gaussian(n, 0, G.DEV)
    tau_dev, r = G.select(g0, None, k)
    want = oracle.dp_select(g0.cpu().numpy(), None, k)
    assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0] and (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq)
    assert float(want.tau) == pytest.approx(3.29, abs=0.05)
    e_dev = torch.zeros(n, device=G.DEV)
    e = np.zeros(n, np.float32)
    counts = []
    for t in range(1, 9):
        g_dev = inputs.dp_gaussian(n, t, G.DEV)
        w = oracle.dp_compress(g_dev.cpu().numpy(), e, want.tau, None, n // 8)
        idx, val, rr = G.compress(g_dev, e_dev, tau_dev, None, n // 8)
        assert rr.status == B.DCT_OK and rr.count == w.count == rr.needed
        assert np.array_equal(idx, w.idx) and np.array_equal(bits32(val), bits32(w.val))
        assert np.array_equal(bits32(e_dev.cpu().numpy()), bits32(e))
        counts.append(rr.count)
    assert counts[0] == pytest.approx(1024, rel=0.15) and counts[-1] > 30 * counts[0]   # density grows under EF


def test_repeated_runs_are_bit_identical():
    n = (1 << 21) + 77
    g_dev = inputs.dp_gaussian(n, 9, G.DEV)
    e0 = inputs.dp_gaussian(n, 10, G.DEV) * 0.5
    tau_dev, _ = G.select(g_dev, e0, 50_000)
    first = None
    for _ in range(10):
        e = e0.clone()
        idx, val, r = G.compress(g_dev, e, tau_dev, None, 100_000)
        got = (idx.tobytes(), val.tobytes(), e.cpu().numpy().tobytes(), r)
        first = first or got
        assert got == first


def test_workspace_reuse_and_garbage_workspace():
    n = 50_000
    g_dev = inputs.dp_gaussian(n, 3, G.DEV)
    tau_dev, _ = G.select(g_dev, None, 500)
    ws = B.new_workspace(B.dct_dp_compress_workspace_bytes(n))
    ws.fill_(0xFF)                                             # stale descriptors must not matter
    e = np.zeros(n, np.float32)
    want = oracle.dp_compress(g_dev.cpu().numpy(), e, tau_dev.cpu().numpy()[0], None, n)
    for _ in range(3):
        e_dev = torch.zeros(n, device=G.DEV)
        idx, val, r = G.compress(g_dev, e_dev, tau_dev, None, n, ws=ws)
        assert np.array_equal(idx, want.idx) and r.count == want.count


def test_bounded_wait_gives_up_cleanly():
    """Tile 0 is never processed (testing ticket offset), so tile 1's look-back finds a descriptor
    nobody writes: the wait must run out, report DCT_ERR_TIMEOUT, keep the residual conservative
    and leave the context usable."""
    n = 3 * 4096
    g_dev = inputs.dp_gaussian(n, 4, G.DEV)
    e_dev = torch.zeros(n, device=G.DEV)
    tau_dev = torch.tensor([1.0], device=G.DEV)
    try:
        B.dct_debug_configure(spin_limit=2000, first_ticket=1)
        idx, val, r = G.compress(g_dev, e_dev, tau_dev, None, n)
    finally:
        B.dct_debug_configure()
    assert r.status == B.DCT_ERR_TIMEOUT
    # tiles 1 and 2 ran: nothing of theirs was sent, so their residual is all of w = g + 0
    got = e_dev.cpu().numpy()
    assert np.array_equal(bits32(got[4096:]), bits32(g_dev.cpu().numpy()[4096:]))
    # and the next normal call works
    e_dev.zero_()
    _compare_compress(g_dev, e_dev, tau_dev, None, n)


def test_host_buffer_entry_point():
    n, cap = 200_000, 20_000
    g_host = inputs.dp_gaussian(n, 21).pin_memory()
    g_dev = torch.empty(n, device=G.DEV)
    e_dev = inputs.dp_gaussian(n, 22, G.DEV) * 0.1
    e = e_dev.cpu().numpy().copy()
    tau_dev = torch.tensor([2.0], device=G.DEV)
    idx_dev = torch.empty(cap, dtype=torch.int32, device=G.DEV)
    val_dev = torch.empty(cap, device=G.DEV)
    idx_host = torch.empty(cap, dtype=torch.int32).pin_memory()
    val_host = torch.empty(cap).pin_memory()
    res_dev, res_host = B.new_result(), torch.zeros(5, dtype=torch.int64).pin_memory()
    ws = B.new_workspace(B.dct_dp_compress_workspace_bytes(n))
    r = B.dct_dp_compress_host(g_host, g_dev, e_dev, n, tau_dev, None, idx_dev, val_dev, cap, idx_host, val_host,
                               res_dev, res_host, ws)
    want = oracle.dp_compress(g_host.numpy(), e, np.float32(2.0), None, cap)
    assert r.count == want.count and r.status == B.DCT_OK
    assert np.array_equal(idx_host.numpy()[:r.count], want.idx)
    assert np.array_equal(bits32(val_host.numpy()[:r.count]), bits32(want.val))
    assert np.array_equal(bits32(e_dev.cpu().numpy()), bits32(e))


def test_select_sampled_path_and_its_fallbacks():
    """From 2^25 elements the select reads the vector once, guided by a sample of 2^17 groups of 8
    neighbours.  The sample only steers: when it misjudges the vector (too few or far too many
    candidates, a band that misses rank k) or cannot be used, the plain passes must give the same exact answer."""
    n = (1 << 25) + 999
    stride = (n // (1 << 17)) & ~7
    sampled = (torch.arange(1 << 17, device=G.DEV)[:, None] * stride + torch.arange(8, device=G.DEV)[None, :]).reshape(-1)
    assert int(sampled.max()) < n
    base = inputs.dp_mixture(n, 90, G.DEV)
    cases = {}
    cases["iid, sparse k"] = (base, 3356)
    cases["dense k: bounds on both sides of tau"] = (base, n // 4)
    cases["dense k, 5 %"] = (base, n // 20)
    cases["dense k, 1.5 %"] = (base, n // 64)
    cases["dense k, ties around tau"] = (inputs.quantize_mantissa(base, 3), n // 10)
    cases["k of half the vector: no sample"] = (base, n // 2 + 1)
    big_at_sampled = inputs.dp_gaussian(n, 91, G.DEV)
    big_at_sampled[sampled] = 1000.0 + inputs.dp_gaussian(sampled.numel(), 92, G.DEV)
    cases["sample overestimates: too few candidates"] = (big_at_sampled, 10_000)
    zero_at_sampled = inputs.dp_gaussian(n, 93, G.DEV)
    zero_at_sampled[sampled] = 0.0
    cases["sample underestimates: candidates overflow"] = (zero_at_sampled, 5_000)
    # dense k with a sample that says nothing about the rest: the band misses rank k on one side or the other
    cases["dense k, sample too large: rank k lies below the band"] = (big_at_sampled, n // 10)
    cases["dense k, sample too small: rank k lies above the band"] = (zero_at_sampled, n // 10)
    shifted = inputs.dp_gaussian(n, 94, G.DEV)
    shifted[sampled] *= 1.02                                   # the band sits a little too high: part of it is used
    cases["dense k, sample slightly off"] = (shifted, n // 10)
    for name, (g, k) in cases.items():
        tau_dev, r = G.select(g, None, k)
        want = oracle.dp_select(g.cpu().numpy(), None, k)
        assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0], name
        assert (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq), name
