"""Decompression (the receiving end of the two "send" steps): oracle pins on CPU, GPU parity, and the
round trips  unpack(pack(x)) == x .* M  and  decompress(compress(g, e)) + e' == g + e."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import inputs
from tests._util import read_golden, bits32, bf16_bits


# ----------------------------------------------------------------------------------------------
# oracle pins (no GPU)
# ----------------------------------------------------------------------------------------------

def test_oracle_dp_decompress_worked_example_and_library_scatter():
    g = read_golden("dct_dp_worked_example.txt")
    n = g["w"].size
    idx = g["literal_idx"].astype(np.int32)
    val = g["literal_val"].astype(np.float32)
    dense = np.full(n, 7.0, np.float32)
    oracle.dp_decompress(idx, val, dense, accumulate=False)
    # W_hat = W .* M of the fixture: W at the kept indices, zero elsewhere; W_hat + E' == W
    want = np.where(np.isin(np.arange(n), idx), g["w"], 0.0).astype(np.float32)
    assert np.array_equal(dense, want)
    assert np.array_equal(dense + g["literal_e_new"].astype(np.float32), g["w"].astype(np.float32))
    # accumulate == numpy's scatter-add on a vector that already holds something
    rng = np.random.default_rng(0)
    base = rng.standard_normal(1000).astype(np.float32)
    idx = np.sort(rng.choice(1000, 137, replace=False)).astype(np.int32)
    val = rng.standard_normal(137).astype(np.float32)
    got = base.copy()
    oracle.dp_decompress(idx, val, got, accumulate=True)
    want = base.copy()
    np.add.at(want, idx, val)
    assert np.array_equal(bits32(got), bits32(want))
    got2 = base.copy()
    oracle.dp_decompress(idx, val, got2, accumulate=False)
    want2 = np.zeros(1000, np.float32)
    want2[idx] = val
    assert np.array_equal(bits32(got2), bits32(want2))
    with pytest.raises(ValueError):
        oracle.dp_decompress(np.array([1000], np.int32), np.array([1.0], np.float32), got2, False)
    with pytest.raises(ValueError):
        oracle.dp_decompress(np.array([-1], np.int32), np.array([1.0], np.float32), got2, True)


def test_oracle_dp_round_trip_conserves_the_gradient():
    n = 20_011
    gvec = inputs.dp_gaussian(n, 3).numpy()
    e_old = (inputs.dp_gaussian(n, 4) * 0.3).numpy()
    tau = oracle.dp_select(gvec, e_old, 300).tau
    e = e_old.copy()
    r = oracle.dp_compress(gvec, e, tau, None, n)
    dense = np.empty(n, np.float32)
    oracle.dp_decompress(r.idx, r.val, dense, accumulate=False)
    w = (gvec + e_old).astype(np.float32)
    # sent + residual == gradient + old residual, element by element (x + 0 is exact)
    assert np.array_equal(dense + e, w)
    assert np.count_nonzero(dense) == r.count


def test_oracle_mp_unpack_worked_example_and_library_scatter():
    g = read_golden("dct_mp_worked_example.txt")
    d, k = int(g["d"][0]), int(g["k"][0])
    x = np.stack([g["x_act_0"], g["x_act_1"]]).astype(np.float32)
    f = oracle.mp_fwd(x, k)
    dense = oracle.mp_unpack(f.cols, f.vals, d)
    # X_act .* M of the fixture, written out by hand
    want = np.array([[0, 3, -3, 0, 0, 0, -5, 0], [-4, 0, 0, 0, 0, 0, 0.5, 0]], np.float32)
    assert np.array_equal(dense, want)
    # random case against numpy's put_along_axis, fp32 and bf16, with padding columns
    rows, d, ld, k = 33, 100, 104, 9
    xs = inputs.mp_activations(rows, d, 5, ld=ld).numpy()
    f = oracle.mp_fwd(xs, k, d=d)
    want = np.zeros((rows, ld), np.float32)
    np.put_along_axis(want, f.cols.astype(np.int64), f.vals, axis=1)
    assert np.array_equal(bits32(oracle.mp_unpack(f.cols, f.vals, d, ld)), bits32(want))
    mask = np.zeros((rows, ld), bool)
    np.put_along_axis(mask, f.cols.astype(np.int64), True, axis=1)
    assert np.array_equal(oracle.mp_unpack(f.cols, f.vals, d, ld), np.where(mask, xs, 0.0))   # x .* M
    xb = bf16_bits(torch.from_numpy(xs).to(torch.bfloat16))
    fb = oracle.mp_fwd(xb, k, d=d)
    wantb = np.zeros((rows, ld), np.uint16)
    np.put_along_axis(wantb, fb.cols.astype(np.int64), fb.vals, axis=1)
    assert np.array_equal(oracle.mp_unpack(fb.cols, fb.vals, d, ld), wantb)
    bad = f.cols.copy()
    bad[0, 0] = d
    with pytest.raises(ValueError):
        oracle.mp_unpack(bad, f.vals, d, ld)


# ----------------------------------------------------------------------------------------------
# GPU parity
# ----------------------------------------------------------------------------------------------

@pytest.mark.gpu
@pytest.mark.parametrize("n", [1, 5, 1023, 1024, 4097, 100_003, (1 << 21) + 7])
def test_gpu_dp_decompress_matches_oracle_and_round_trips(n):
    from paper_2010_08899_b200 import binding as B
    from tests import _gpu as G
    g_dev = inputs.dp_gaussian(n, 50 + n % 97, G.DEV)
    e_dev = inputs.dp_gaussian(n, 60 + n % 89, G.DEV) * 0.25
    w = (g_dev + e_dev)
    for k in sorted({1, max(1, n // 100), max(1, n // 3)}):
        tau_dev, _ = G.select(g_dev, e_dev, k)
        for cap in (n, max(1, k // 2)):
            e = e_dev.clone()
            idx = torch.full((cap + 8,), -9, dtype=torch.int32, device=G.DEV)
            val = torch.full((cap + 8,), -9.0, device=G.DEV)
            packed = B.new_result()
            B.dct_dp_compress(g_dev, e, n, tau_dev, None, idx, val, cap, packed,
                              B.new_workspace(B.dct_dp_compress_workspace_bytes(n)))
            count = B.read_result(packed).count
            for offset in (0, 1):                       # aligned and misaligned dense vector
                buf = torch.full((n + 8 + offset,), 5.0, device=G.DEV)
                dense = buf[offset:offset + n]
                res = B.new_result()
                B.dct_dp_decompress(idx, val, packed, cap, dense, n, False, res)
                assert B.read_result(res).status == B.DCT_OK
                want = np.full(n, 5.0, np.float32)
                oracle.dp_decompress(idx[:count].cpu().numpy(), val[:count].cpu().numpy(), want, False)
                assert np.array_equal(bits32(dense.cpu().numpy()), bits32(want))
                assert bool((buf[offset + n:] == 5.0).all()) and bool((buf[:offset] == 5.0).all())
                # round trip: what was sent plus what was kept is the error-fed gradient
                assert torch.equal(dense + e, w)
            # accumulate into a vector that already holds something
            base = inputs.dp_gaussian(n, 70, G.DEV)
            acc = base.clone()
            res = B.new_result()
            B.dct_dp_decompress(idx, val, packed, cap, acc, n, True, res)
            want = base.cpu().numpy().copy()
            oracle.dp_decompress(idx[:count].cpu().numpy(), val[:count].cpu().numpy(), want, True)
            assert np.array_equal(bits32(acc.cpu().numpy()), bits32(want))


@pytest.mark.gpu
def test_gpu_dp_decompress_reports_bad_indices_without_touching_anything_else():
    from paper_2010_08899_b200 import binding as B
    n = 5000
    idx = torch.tensor([3, 17, 4999, 5000, 70000], dtype=torch.int32, device="cuda")
    val = torch.tensor([1.0, 2.0, 3.0, 4.0, 5.0], device="cuda")
    packed = torch.tensor([0, 5, 5, 0, 0], dtype=torch.int64, device="cuda")
    buf = torch.full((n + 64,), 9.0, device="cuda")
    res = B.new_result()
    B.dct_dp_decompress(idx, val, packed, 5, buf[:n], n, False, res)
    assert B.read_result(res).status == B.DCT_ERR_BAD_MASK
    want = torch.zeros(n, device="cuda")
    want[3], want[17], want[4999] = 1.0, 2.0, 3.0
    assert torch.equal(buf[:n], want) and bool((buf[n:] == 9.0).all())


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("rows,d,ld,k", [(1, 1, 1, 1), (37, 33, 40, 5), (64, 1000, 1000, 50), (300, 4096, 4096, 205),
                                         (9, 4097, 4101, 400),
                                         # short rows with few kept columns: a thread per 16-byte unit
                                         (70001, 64, 64, 3), (5003, 64, 72, 16), (3001, 128, 136, 6), (2000, 256, 256, 2),
                                         (999, 32, 32, 32), (777, 8, 8, 1),
                                         # just beyond that kernel's reach
                                         (3000, 128, 128, 32), (1000, 512, 512, 25)])
def test_gpu_mp_unpack_matches_oracle_and_round_trips(dtype, rows, d, ld, k):
    from paper_2010_08899_b200 import binding as B
    from tests import _gpu as G
    x = inputs.mp_activations(rows, d, 5 + d, dtype=dtype, device=G.DEV, col_scale_seed=6 + d, ld=ld)
    gx = inputs.mp_gradients(rows, d, 7 + d, dtype=dtype, device=G.DEV, ld=ld)
    cols, vals, _, _ = G.mp_fwd(x, d, k)
    gv, _ = G.mp_bwd(gx, d, cols)
    for src, packed in ((x, vals), (gx, gv)):
        dense = torch.full((rows, ld), 3.0, dtype=dtype, device=G.DEV)
        res = B.new_result()
        B.dct_mp_unpack(cols.contiguous(), packed.contiguous(), rows, d, ld, k, dense, res)
        assert B.read_result(res).status == B.DCT_OK
        want = oracle.mp_unpack(cols.cpu().numpy(), G.to_oracle(packed), d, ld)
        got = G.as_np_bits(dense)
        assert np.array_equal(got[:, :d], want[:, :d].view(got.dtype))
        if ld > d:                                       # padding columns are left alone
            assert bool((dense[:, d:] == 3.0).all())
        # round trip: X .* M
        mask = torch.zeros(rows, ld, dtype=torch.bool, device=G.DEV)
        mask.scatter_(1, cols.long(), True)
        assert torch.equal(dense[:, :d], torch.where(mask, src, torch.zeros_like(src))[:, :d])


@pytest.mark.gpu
@pytest.mark.parametrize("accumulate", [False, True])
@pytest.mark.parametrize("bad_idx", [[3, -1, 10], [3, 70000, 10], [10, 5], [7, 7], [0, 1, 2, 2, 9]])
def test_gpu_dp_decompress_checks_the_whole_index_list(bad_idx, accumulate):
    """A negative or too-large index in the middle of the list, an unsorted pair and a duplicate are all reported,
    whichever CTA's range they fall into, and nothing outside the vector is touched."""
    from paper_2010_08899_b200 import binding as B
    n = 300_000                                     # several CTA ranges
    filler = list(range(20_000, 20_000 + 40_000, 7))  # a valid ascending run after the bad entries
    good = [i for i in bad_idx if 0 <= i < n]
    idx_list = bad_idx + [i for i in filler if i > max(good)]
    idx = torch.tensor(idx_list, dtype=torch.int32, device="cuda")
    val = torch.arange(1, len(idx_list) + 1, dtype=torch.float32, device="cuda")
    packed = torch.tensor([0, len(idx_list), len(idx_list), 0, 0], dtype=torch.int64, device="cuda")
    buf = torch.full((n + 64,), 9.0, device="cuda")
    res = B.new_result()
    B.dct_dp_decompress(idx, val, packed, len(idx_list), buf[:n], n, accumulate, res)
    assert B.read_result(res).status == B.DCT_ERR_BAD_MASK
    assert bool((buf[n:] == 9.0).all())
    # the same list without its faults is accepted
    ok = sorted(set(good) | {i for i in filler if i > max(good)})
    idx2 = torch.tensor(ok, dtype=torch.int32, device="cuda")
    packed2 = torch.tensor([0, len(ok), len(ok), 0, 0], dtype=torch.int64, device="cuda")
    res2 = B.new_result()
    B.dct_dp_decompress(idx2, val[:len(ok)].contiguous(), packed2, len(ok), buf[:n], n, accumulate, res2)
    assert B.read_result(res2).status == B.DCT_OK


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_gpu_mp_unpack_of_short_rows_rejects_out_of_range_and_takes_any_order(dtype):
    """The thread-per-unit kernel for short rows: a column past the row is skipped and reported, the other entries of
    the row are placed, and the columns of a row need not be ascending."""
    from paper_2010_08899_b200 import binding as B
    rows, d, k = 4, 64, 3
    cols = torch.tensor([[0, 1, 2], [3, 64, 5], [63, 7, 8], [-1, 10, 9]], dtype=torch.int16, device="cuda")
    vals = torch.arange(1, rows * k + 1, dtype=torch.float32, device="cuda").view(rows, k).to(dtype)
    dense = torch.full((rows, d), 2.0, dtype=dtype, device="cuda")
    res = B.new_result()
    B.dct_mp_unpack(cols, vals, rows, d, d, k, dense, res)
    assert B.read_result(res).status == B.DCT_ERR_BAD_MASK
    want = torch.zeros(rows, d, device="cuda")
    want[0, 0], want[0, 1], want[0, 2] = 1, 2, 3
    want[1, 3], want[1, 5] = 4, 6
    want[2, 63], want[2, 7], want[2, 8] = 7, 8, 9
    want[3, 10], want[3, 9] = 11, 12
    assert torch.equal(dense.float(), want)


@pytest.mark.gpu
def test_gpu_mp_unpack_rejects_out_of_range_columns():
    from paper_2010_08899_b200 import binding as B
    rows, d, k = 4, 50, 3
    cols = torch.tensor([[0, 1, 2], [3, 50, 5], [6, 7, 8], [-1, 10, 11]], dtype=torch.int16, device="cuda")
    vals = torch.arange(1, rows * k + 1, dtype=torch.float32, device="cuda").view(rows, k)
    dense = torch.full((rows, d), 2.0, device="cuda")
    res = B.new_result()
    B.dct_mp_unpack(cols, vals, rows, d, d, k, dense, res)
    assert B.read_result(res).status == B.DCT_ERR_BAD_MASK
    want = torch.zeros(rows, d, device="cuda")
    want[0, 0], want[0, 1], want[0, 2] = 1, 2, 3
    want[1, 3], want[1, 5] = 4, 6
    want[2, 6], want[2, 7], want[2, 8] = 7, 8, 9
    want[3, 10], want[3, 11] = 11, 12
    assert torch.equal(dense, want)
