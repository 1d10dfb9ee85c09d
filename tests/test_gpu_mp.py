"""GPU parity of DCT-MP (per-row top-k + forward pack, backward pack through the same mask)
against the CPU oracle: bit-exact on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import binding as B
from paper_2010_08899_b200 import inputs
from tests import _gpu as G

pytestmark = pytest.mark.gpu


def _compare_fwd_bwd(x_dev, gx_dev, d, k, want_rows=False):
    rows = x_dev.shape[0]
    want = oracle.mp_fwd(G.to_oracle(x_dev), k, d=d)
    cols, vals, tau, rws = G.mp_fwd(x_dev, d, k, want_rows=want_rows)
    assert np.array_equal(cols.cpu().numpy(), want.cols)
    assert np.array_equal(G.as_np_bits(vals), want.vals.view(G.as_np_bits(vals).dtype))
    assert np.array_equal(G.as_np_bits(tau), want.tau.view(G.as_np_bits(tau).dtype))
    if want_rows:
        assert np.array_equal(rws.cpu().numpy(), np.repeat(np.arange(rows, dtype=np.int32)[:, None], k, 1))
    if gx_dev is not None:
        cols_before = cols.clone()
        gv, r = G.mp_bwd(gx_dev, d, cols)
        assert r.status == B.DCT_OK
        assert torch.equal(cols, cols_before)                  # the mask is consumed unchanged
        want_g = oracle.mp_bwd(G.to_oracle(gx_dev), want.cols, d=d)
        assert np.array_equal(G.as_np_bits(gv), want_g.view(G.as_np_bits(gv).dtype))
    return cols


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d,ld", [(1, 1), (7, 7), (33, 40), (1000, 1000), (1024, 1024), (4097, 4100),
                                  (5000, 5000), (32768, 32768)])
def test_mp_odd_shapes(dtype, d, ld):
    rows = 37 if d < 8192 else 5
    x = inputs.mp_activations(rows, d, 50 + d, dtype=dtype, device=G.DEV, col_scale_seed=60 + d, ld=ld)
    gx = inputs.mp_gradients(rows, d, 70 + d, dtype=dtype, device=G.DEV, ld=ld)
    for k in sorted({1, min(d, 2), max(1, d // 20), max(1, d // 2), max(1, d - 1), d}):
        cols = _compare_fwd_bwd(x, gx, d, k, want_rows=(k == 1))
        assert int(cols.max()) < d


@pytest.mark.parametrize("dtype,d", [(torch.float32, 12288), (torch.float32, 11800), (torch.bfloat16, 24576),
                                     (torch.bfloat16, 24000)])
def test_mp_rows_of_just_under_48_kib_in_the_general_kernel(dtype, d):
    """A row of 44 to 48 KiB fits the shared memory a kernel gets without asking only if the kernel had no static
    shared memory of its own: the general kernel (k = d / 2 is beyond every fast path) must ask for more there too."""
    rows = 9
    x = inputs.mp_activations(rows, d, 61 + d, dtype=dtype, device=G.DEV, col_scale_seed=62 + d)
    gx = inputs.mp_gradients(rows, d, 63 + d, dtype=dtype, device=G.DEV)
    _compare_fwd_bwd(x, gx, d, d // 2)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_mp_misaligned_rows(dtype):
    rows, d, ld, k = 20, 301, 303, 31
    x = inputs.mp_activations(rows, d, 5, dtype=dtype, device=G.DEV, ld=ld)
    gx = inputs.mp_gradients(rows, d, 6, dtype=dtype, device=G.DEV, ld=ld)
    xo = G.offset_copy(x, 1).view(rows, ld)
    go = G.offset_copy(gx, 3).view(rows, ld)
    _compare_fwd_bwd(xo, go, d, k)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_mp_ties_signs_and_degenerate_rows(dtype):
    rows, d = 64, 2048
    sign = torch.where(inputs.dp_gaussian(rows * d, 1, G.DEV).view(rows, d) > 0, 1.0, -1.0)
    x = inputs.quantize_mantissa(inputs.mp_activations(rows, d, 2, device=G.DEV, col_scale_seed=3), 1) * sign
    x[0] = 0.0                                   # all zero: pure lowest-column rule
    x[1] = 3.0                                   # all equal
    x[2] = torch.tensor([1.5, -1.5], device=G.DEV).repeat(d // 2)
    x[3] = 0.0
    x[3, 5] = -1e30                              # one outlier, rest zeros
    x[4] = torch.arange(d, device=G.DEV) * 1e-42   # denormals (fp32) / zeros after bf16 rounding
    x = x.to(dtype).contiguous()
    gx = inputs.mp_gradients(rows, d, 4, dtype=dtype, device=G.DEV)
    for k in (1, 64, 102, 1024, d):
        _compare_fwd_bwd(x, gx, d, k)


def test_config2_mp_small():
    """2048 x 1024 fp32, ReLU of N(0,1), k = 64; plus a tie-injected copy."""
    rows, d, k = 2048, 1024, 64
    x = inputs.mp_activations(rows, d, 100, device=G.DEV)
    gx = inputs.mp_gradients(rows, d, 101, device=G.DEV)
    zero_frac = float((x == 0).float().mean())
    assert 0.45 < zero_frac < 0.55
    _compare_fwd_bwd(x, gx, d, k, want_rows=True)
    _compare_fwd_bwd(inputs.quantize_mantissa(x, 4), gx, d, k)


def test_config4_mp_production_width():
    """16384 x 4096 bf16, ReLU of N(0,1) with per-column LogNormal scale, k = 205 (5 %)."""
    rows, d, k = 16384, 4096, 205
    assert k == B.k_from_sparsity(d, 95, 100)
    x = inputs.mp_activations(rows, d, 410, dtype=torch.bfloat16, device=G.DEV, col_scale_seed=400)
    gx = inputs.mp_gradients(rows, d, 420, dtype=torch.bfloat16, device=G.DEV)
    cols = _compare_fwd_bwd(x, gx, d, k)
    # ties at tau_i are the common case in bf16: make sure the input really exercises them
    keys = (x.view(torch.int16).to(torch.int32) & 0x7FFF)
    kth = torch.topk(keys, k, dim=1).values[:, -1:]
    tied_rows = ((keys == kth).sum(1) > 1).float().mean().item()
    assert tied_rows > 0.2
    assert cols.shape == (rows, k)


def test_bwd_rejects_out_of_range_columns():
    rows, d, k = 8, 100, 4
    gx = inputs.mp_gradients(rows, d, 1, device=G.DEV)
    cols = torch.tensor([[0, 1, 2, 3]] * rows, dtype=torch.int16, device=G.DEV)
    cols[3, 2] = 100
    cols[5, 0] = -1
    gv, r = G.mp_bwd(gx, d, cols)
    assert r.status == B.DCT_ERR_BAD_MASK
    want = torch.gather(gx, 1, cols.long().clamp(0, d - 1))
    want[3, 2] = 0
    want[5, 0] = 0
    assert torch.equal(gv, want)


def test_mp_host_buffer_entry_point():
    rows, d, k = 256, 512, 26
    x = inputs.mp_activations(rows, d, 7, dtype=torch.bfloat16).pin_memory()
    gx = inputs.mp_gradients(rows, d, 8, dtype=torch.bfloat16).pin_memory()
    dev = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt, device=G.DEV)
    host = lambda *s, dt=torch.bfloat16: torch.empty(*s, dtype=dt).pin_memory()
    cols_h, vals_h, gv_h = host(rows * k, dt=torch.int16), host(rows * k), host(rows * k)
    res_h = torch.zeros(5, dtype=torch.int64).pin_memory()
    B.dct_mp_pack_host(x, gx, dev(rows, d), dev(rows, d), rows, d, d, k, dev(rows * k, dt=torch.int16),
                       dev(rows * k), dev(rows * k), cols_h, vals_h, gv_h, B.new_result(), res_h)
    want = oracle.mp_fwd(G.to_oracle(x), k)
    assert np.array_equal(cols_h.numpy().reshape(rows, k), want.cols)
    assert np.array_equal(G.as_np_bits(vals_h).reshape(rows, k), want.vals)
    assert np.array_equal(G.as_np_bits(gv_h).reshape(rows, k), oracle.mp_bwd(G.to_oracle(gx), want.cols))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_mp_rows_with_wildly_different_scales(dtype):
    """The warp-per-row kernels guess each row's bound from the previous row's threshold; rows whose
    scales jump by orders of magnitude make that guess useless in both directions (too few / far too
    many candidates), which must only cost time, never change the result."""
    # enough rows that every warp of the persistent grid meets several of them, and a scale pattern whose
    # period (7) shares no factor with the number of warps, so consecutive rows of a warp differ in scale
    rows, d, k = 9002, 4096, 205
    x = inputs.mp_activations(rows, d, 77, dtype=torch.float32, device=G.DEV, col_scale_seed=78)
    scale = torch.tensor([1.0, 300.0, 0.004, 17.0, 1e-3, 1e4, 1.0], device=G.DEV).repeat(rows // 7)
    x = (x * scale[:, None]).to(dtype).contiguous()
    x[5] = 0                                    # a dead sample between live ones
    x[6, ::7] = 2.0                             # heavy ties right after it
    gx = inputs.mp_gradients(rows, d, 79, dtype=dtype, device=G.DEV)
    for kk in (k, 64, 256):
        _compare_fwd_bwd(x, gx, d, kk)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [256, 512, 768, 1280, 1536, 1792, 2560, 3072, 3584, 4096])
def test_mp_warp_per_row_widths(dtype, d):
    """Every row width the warp-per-row kernels are instantiated for, both dtypes, with k on both sides of
    their limits (k <= d/8 and 224, k <= d/4 and 448)."""
    rows = 300
    x = inputs.mp_activations(rows, d, 11 + d, dtype=dtype, device=G.DEV, col_scale_seed=12 + d)
    x[7] = 0
    x[8] = 1.0
    x[9, ::3] = -2.5
    gx = inputs.mp_gradients(rows, d, 13 + d, dtype=dtype, device=G.DEV)
    for k in sorted({1, max(1, d // 20), d // 10, d // 8, d // 5, min(d // 4, 448), min(d // 4, 448) + 1}):
        _compare_fwd_bwd(x, gx, d, k)


def test_mp_f32_keys_that_differ_only_in_the_low_bits():
    """fp32 rows whose magnitudes share their upper 16 bits in large groups: the 15-bit bucket of tau_i
    then holds many members, and the order inside it is decided by the lower 16 bits alone (few members:
    ranked through the list; more than 64: bit by bit), with exact ties on top."""
    rows, d, k = 600, 4096, 205
    g = torch.Generator(device=G.DEV).manual_seed(5)
    hi = torch.randint(0x3F00, 0x3F10, (rows, d), generator=g, device=G.DEV, dtype=torch.int32)       # 16 buckets only
    lo = torch.randint(0, 1 << 16, (rows, d), generator=g, device=G.DEV, dtype=torch.int32)
    lo[100:200] &= 0xFF00                                   # coarse lower bits: exact ties inside the bucket
    lo[200:300] = 0                                         # bf16-valued fp32: every member of a bucket ties
    sign = torch.randint(0, 2, (rows, d), generator=g, device=G.DEV, dtype=torch.int32) << 31
    x = ((hi << 16) | lo | sign).view(torch.float32).contiguous()
    x[300:400, 1000:] = 0.0                                 # ~1000 live columns: buckets of ~60 members
    gx = inputs.mp_gradients(rows, d, 6, device=G.DEV)
    for kk in (k, 17, 448, 1024, 2048):
        _compare_fwd_bwd(x, gx, d, kk)


@pytest.mark.parametrize("d,k_limit", [(256, 20), (512, 40), (768, 48), (1024, 64)])
def test_mp_bf16_narrow_rows_several_per_warp(d, k_limit):
    """Rows of at most 1024 bf16 columns stay in registers, 4 / 2 / 1 of them per warp: row counts that leave
    the last warp partly filled, k on both sides of the path's limit, and rows that force each of its
    fall-backs (no previous threshold, threshold far from the previous one, ties that overflow the list,
    dead rows) next to ordinary ones in the same warp."""
    for rows in (1, 3, 37, 1001):
        x = inputs.mp_activations(rows, d, 21 + d + rows, dtype=torch.float32, device=G.DEV, col_scale_seed=22 + d)
        scale = torch.tensor([1.0, 250.0, 0.01, 1.0, 3.0], device=G.DEV).repeat(rows // 5 + 1)[:rows]
        x = x * scale[:, None]
        if rows > 30:
            x[4] = 0.0                                  # dead row
            x[9] = 1.5                                  # every element ties
            x[10, ::2] = -7.0                           # half the row ties above everything else
            x[17] = inputs.quantize_mantissa(x[17], 1)  # coarse values
        x = x.to(torch.bfloat16).contiguous()
        gx = inputs.mp_gradients(rows, d, 23 + d, dtype=torch.bfloat16, device=G.DEV)
        for k in sorted({1, max(1, d // 20), k_limit, k_limit + 1}):
            _compare_fwd_bwd(x, gx, d, k)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [264, 1000, 2000, 3000, 4000, 4088])
def test_mp_warp_per_row_widths_between_the_buffer_sizes(dtype, d):
    """Rows whose width is a multiple of 16 bytes but not of 256 columns sit zero-padded in the next larger
    buffer of the warp-per-row kernels: the padding must never be selected, not even by rows with fewer than
    k non-zeros (ties at zero go to the lowest columns) or rows of equal values."""
    rows = 203
    x = inputs.mp_activations(rows, d, 31 + d, dtype=dtype, device=G.DEV, col_scale_seed=32 + d)
    x[5] = 0.0                                   # dead row: the first k columns
    x[6] = -0.75                                 # all equal
    x[7] = 0.0
    x[7, d - 3:] = 1.0                           # three non-zeros at the very end, zeros elsewhere
    x[8, : d - 8] = 0.0                          # only the last 8 columns alive
    gx = inputs.mp_gradients(rows, d, 33 + d, dtype=dtype, device=G.DEV)
    for k in sorted({1, 7, d // 20, d // 8, min(d // 4, 448)}):
        cols = _compare_fwd_bwd(x, gx, d, k)
        assert int(cols.max()) < d


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("d", [512, 1024, 2000, 4096])
def test_mp_dense_k(dtype, d):
    """k from a quarter to half of the row (75 % sparsity and below): up to 3/8 of the row tau_i is pinned between
    two bounds at most 64 keys apart (beyond, the general kernel serves).  Rows whose scale jumps by orders of
    magnitude make the window move several times; ties, dead rows and rows with fewer than k non-zeros (tau_i = 0:
    the first zeros fill the row's slots) take the remaining branches."""
    rows = 2500
    x = inputs.mp_activations(rows, d, 51 + d, dtype=torch.float32, device=G.DEV, col_scale_seed=52 + d)
    sign = torch.where(inputs.dp_gaussian(rows * d, 53 + d, G.DEV).view(rows, d) > 0, 1.0, -1.0)
    scale = torch.tensor([1.0, 40.0, 1.0, 1e-3, 1e4, 1.0, 1.0], device=G.DEV).repeat(rows // 7 + 1)[:rows]
    x = x * sign * scale[:, None]
    x[3] = 0.0                                      # dead row
    x[4] = 2.0                                      # every element ties
    x[5, d // 3:] = 0.0                             # fewer than d/2 non-zeros
    x[6] = inputs.quantize_mantissa(x[6], 1)        # few distinct values
    x[7] = 3.0e38                                   # the top of the range
    x = x.to(dtype).contiguous()
    gx = inputs.mp_gradients(rows, d, 54 + d, dtype=dtype, device=G.DEV)
    for k in sorted({d // 4 + 1, d // 3, d // 2, min(d // 2, 1280)}):
        _compare_fwd_bwd(x, gx, d, k)


@pytest.mark.parametrize("d", [1024, 4096])
def test_mp_dense_k_clustered_columns_and_many_ties(d):
    """In the bf16 kernel for denser k every lane walks the kept bits of its own span of the row: rows whose kept
    columns sit in one part of the row (some lanes hold nearly everything, others nothing), rows of a few distinct
    values (every row has many ties at tau_i, spread over the lanes, of which only some are kept; windows that
    have to be narrowed), and k that is not a multiple of 32."""
    rows = 900
    x = inputs.mp_activations(rows, d, 71 + d, dtype=torch.float32, device=G.DEV, col_scale_seed=72 + d)
    third = d // 3
    x[0::6, third:] = 0.0                            # only the first third is alive
    x[1::6, :d - third] = 0.0                        # only the last third
    x[2::6, third // 2:d - third // 2] = 0.0         # both ends, nothing in the middle
    x[3::6] = inputs.quantize_mantissa(x[3::6], 2)   # a handful of distinct values per binade: ties everywhere
    x[4::6] = torch.round(x[4::6] * 4.0) / 4.0       # multiples of 0.25, most of them 0
    x = x.to(torch.bfloat16).contiguous()
    gx = inputs.mp_gradients(rows, d, 73 + d, dtype=torch.bfloat16, device=G.DEV)
    for k in sorted({d // 4 + 3, third - 5, third, third + 1, min(d // 2 - 1, 1279), min(d // 2, 1280)}):
        cols = _compare_fwd_bwd(x, gx, d, k)
        assert int(cols.max()) < d


@pytest.mark.parametrize("d,k", [(1024, 256), (2048, 512), (4096, 1024), (4096, 1280)])
def test_mp_dense_k_multiple_of_256_writes_whole_words(d, k):
    """With 4-byte aligned outputs the bf16 kernel for denser k stores its staged entries in pairs (4-byte words of
    either output, plus the optional row ids); an output that starts 2 bytes off goes to the general kernel.  Both
    give the oracle's result, and neither writes outside its rows * k slots."""
    rows = 333
    x = inputs.mp_activations(rows, d, 81 + d, dtype=torch.bfloat16, device=G.DEV, col_scale_seed=82 + d)
    x[5] = 0.5                                       # every element ties: the first k columns win
    want = oracle.mp_fwd(G.to_oracle(x), k, d=d)
    cols, vals, tau, rws = G.mp_fwd(x, d, k, want_rows=True)
    assert np.array_equal(cols.cpu().numpy(), want.cols)
    assert np.array_equal(G.as_np_bits(vals), want.vals.view(np.uint16))
    assert np.array_equal(rws.cpu().numpy(), np.repeat(np.arange(rows, dtype=np.int32)[:, None], k, 1))
    # outputs one element (2 bytes) off a 16-byte boundary
    cols_buf = torch.full((rows * k + 9,), -1, dtype=torch.int16, device=G.DEV)
    vals_buf = torch.full((rows * k + 9,), 99.0, dtype=torch.bfloat16, device=G.DEV)
    res = B.new_result()
    B.dct_mp_topk_pack_fwd(x, rows, d, d, k, cols_buf[1:], vals_buf[1:], None, None, res)
    assert B.read_result(res).status == B.DCT_OK
    assert np.array_equal(cols_buf[1:1 + rows * k].view(rows, k).cpu().numpy(), want.cols)
    assert np.array_equal(G.as_np_bits(vals_buf[1:1 + rows * k].view(rows, k)), want.vals.view(np.uint16))
    assert int(cols_buf[0]) == -1 and bool((cols_buf[1 + rows * k:] == -1).all())
    assert float(vals_buf[0]) == 99.0 and bool((vals_buf[1 + rows * k:] == 99.0).all())


@pytest.mark.parametrize("d", [5000, 6144, 8000, 8192])
def test_mp_bf16_wide_rows(d):
    """bf16 rows of more than 4096 and up to 8192 columns take the warp-per-row kernels too (buffers of 6144
    and 8192 columns): sparse k with 10 and 20 candidates per lane, dense k, and the degenerate rows."""
    rows = 700
    x = inputs.mp_activations(rows, d, 61 + d, dtype=torch.float32, device=G.DEV, col_scale_seed=62 + d)
    scale = torch.tensor([1.0, 30.0, 1e-2, 1.0, 1.0], device=G.DEV).repeat(rows // 5 + 1)[:rows]
    x = x * scale[:, None]
    x[3] = 0.0
    x[4] = -1.25
    x[5, 100:] = 0.0
    x[6] = inputs.quantize_mantissa(x[6], 2)
    x = x.to(torch.bfloat16).contiguous()
    gx = inputs.mp_gradients(rows, d, 63 + d, dtype=torch.bfloat16, device=G.DEV)
    for k in sorted({1, d // 40, d // 20, d // 10, 1000, 1280}):
        cols = _compare_fwd_bwd(x, gx, d, k)
        assert int(cols.max()) < d


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("d,ld", [(32, 32), (64, 64), (64, 72), (96, 96), (128, 128), (128, 136), (192, 200), (256, 256),
                                  (256, 264), (320, 320), (384, 384), (512, 512), (512, 640)])
def test_mp_many_short_rows(dtype, d, ld):
    """Many short rows (the widths of the paper's recommendation-model layers), more than one round of any
    persistent grid and not a multiple of 32: contiguous and strided rows, sparse and denser k, rows of very
    different scales (a guess taken from a previous row fails in both directions), dead rows, rows where
    everything ties, rows with fewer than k non-zeros, rows of a few distinct values, rows with huge values
    (thresholds at the top of the key range), and in fp32 denormal rows and rows whose values differ only in
    their lower key bits."""
    rows = 32 * 148 * 3 + 21
    x = inputs.mp_activations(rows, d, 291 + d, dtype=torch.float32, device=G.DEV, col_scale_seed=292 + d, ld=ld)
    sign = torch.where(inputs.dp_gaussian(rows * ld, 293 + d, G.DEV).view(rows, ld) > 0, 1.0, -1.0)
    scale = torch.tensor([1.0, 30.0, 1e-2, 1.0, 1e3, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0], device=G.DEV)
    scale = scale.repeat(rows // 11 + 1)[:rows]
    x = x * sign * scale[:, None]
    x[3] = 0.0
    x[4] = -1.25
    x[5, 9:] = 0.0
    x[6] = inputs.quantize_mantissa(x[6], 1)
    x[7::50] = inputs.quantize_mantissa(x[7::50], 2)
    x[8] = 3.0e38
    x[9, ::3] = 3.3e38
    x[13, 1:] = 0.0                                     # one non-zero: the first zeros, never a column past the row, fill up
    x[10] = x[10] * 1e-41                               # fp32: denormals, every key in bucket 0 (bf16: zeros)
    x[11::50] = inputs.quantize_mantissa(x[11::50], 9)  # fp32: several members per bucket, ties inside it
    x[12::50] = 1.0 + torch.arange(ld, device=G.DEV) * 2.0 ** -22     # fp32: one bucket holds the whole row
    x[rows - 1] = 0.5
    x = x.to(dtype).contiguous()
    gx = inputs.mp_gradients(rows, d, 294 + d, dtype=dtype, device=G.DEV, ld=ld)
    for k in sorted({1, 2, d // 20, d // 10, d // 8, d // 4, d // 2, d - 1, d}):
        cols = _compare_fwd_bwd(x, gx, d, k, want_rows=(k == 2))
        assert int(cols.max()) < d


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("d,ld,shift", [(1, 1, 0), (7, 7, 0), (33, 40, 0), (64, 64, 1), (100, 100, 0), (127, 131, 0),
                                        (128, 128, 3), (250, 250, 0), (256, 260, 0), (257, 257, 1), (500, 500, 0),
                                        (512, 516, 0), (512, 512, 1), (513, 513, 0), (1000, 1004, 0), (1001, 1001, 0),
                                        (1024, 1024, 1)])
def test_mp_short_rows_at_any_width_stride_and_address(dtype, d, ld, shift):
    """Rows of up to 1024 columns that do not start on 16-byte boundaries or are not whole 16-byte units (odd widths, odd
    strides, a matrix that starts `shift` elements into its buffer): every k, rows of different scales, dead rows,
    ties, fewer than k non-zeros; the columns past the end of a row are never read as part of it."""
    rows = (16 * 148 * 2 if d <= 512 else 16 * 148) + 5
    buf = torch.full((rows * ld + shift + 8,), 7.0e30, dtype=torch.float32, device=G.DEV)   # huge values around the rows
    x = inputs.mp_activations(rows, d, 391 + d, dtype=torch.float32, device=G.DEV, col_scale_seed=392 + d, ld=ld)
    sign = torch.where(inputs.dp_gaussian(rows * ld, 393 + d, G.DEV).view(rows, ld) > 0, 1.0, -1.0)
    scale = torch.tensor([1.0, 30.0, 1e-2, 1.0, 1e3, 1.0, 1.0], device=G.DEV).repeat(rows // 7 + 1)[:rows]
    x = x * sign * scale[:, None]
    x[3] = 0.0
    x[4] = -1.25
    x[5, 2:] = 0.0
    x[6] = inputs.quantize_mantissa(x[6], 1)
    x[:, d:] = 7.0e30                                  # the padding between rows must never win
    buf[shift:shift + rows * ld] = x.reshape(-1)
    xs = buf.to(dtype)[shift:shift + rows * ld].view(rows, ld)
    gx = inputs.mp_gradients(rows, d, 394 + d, dtype=dtype, device=G.DEV, ld=ld)
    for k in sorted({1, max(1, d // 20), max(1, d // 4), max(1, d // 2), d}):
        cols = _compare_fwd_bwd(xs, gx, d, k)
        assert int(cols.max()) < d


@pytest.mark.parametrize("d", [516, 768, 1024, 1540, 2048, 2052, 4096, 4100, 8192, 12000, 16384, 24580, 32768])
def test_mp_f32_rows_wider_than_512(d):
    """fp32 rows of more than 512 columns that the sparse warp-per-row kernel leaves out (every k beyond 4096
    columns, the denser k up to 4096) are packed by a CTA per row, a lane looking after 32 or 64 columns: sparse and
    denser k, rows of very different scales (the window has to move), dead rows, rows where everything ties, rows
    with fewer than k non-zeros, rows of tiny values inside bucket 0, rows of a few distinct values (many members in
    one bucket, ties inside it), and more rows than CTAs, so that every CTA works through several rows."""
    rows = 900 if d <= 8192 else 400
    x = inputs.mp_activations(rows, d, 191 + d, dtype=torch.float32, device=G.DEV, col_scale_seed=192 + d)
    sign = torch.where(inputs.dp_gaussian(rows * d, 193 + d, G.DEV).view(rows, d) > 0, 1.0, -1.0)
    scale = torch.tensor([1.0, 30.0, 1e-2, 1.0, 1e3, 1.0, 1.0], device=G.DEV).repeat(rows // 7 + 1)[:rows]
    x = x * sign * scale[:, None]
    x[3] = 0.0
    x[4] = -1.25
    x[5, 300:] = 0.0
    x[6] = inputs.quantize_mantissa(x[6], 1)
    x[7::50] = inputs.quantize_mantissa(x[7::50], 2)
    x[8] = 3.0e38
    x[9] = x[9] * 1e-41                          # denormals: every key in bucket 0
    x[10, 100:] = x[10, 100:] * 1e-42
    x[11::50] = inputs.quantize_mantissa(x[11::50], 9)    # few distinct values inside a bucket
    x = x.contiguous()
    gx = inputs.mp_gradients(rows, d, 194 + d, dtype=torch.float32, device=G.DEV)
    for k in sorted({d // 7, min(d // 4 + 1, 4095), 3 * d // 8} | ({1, 33, d // 20} if d > 4096 else set())):
        cols = _compare_fwd_bwd(x, gx, d, k, want_rows=(k == 33))
        assert int(cols.max()) < d


@pytest.mark.parametrize("d", [3080, 4096, 5120, 6152, 8192, 8200, 12288, 16384, 20000, 32768])
def test_mp_bf16_rows_wider_than_3072(d):
    """bf16 rows of more than 3072 columns are packed by a CTA per row (2 to 8 warps, a lane looking after 64 columns
    up to 8192 columns, after 128 beyond) wherever the sparse warp-per-row kernel does not apply: sparse and denser
    k, rows of very different scales (the window has to move), dead rows, rows where everything ties, rows with
    fewer than k non-zeros, rows of a few distinct values (crowded windows and the exact mode), and more rows than
    CTAs, so that every CTA works through several rows."""
    rows = 1500 if d <= 16384 else 700
    x = inputs.mp_activations(rows, d, 91 + d, dtype=torch.float32, device=G.DEV, col_scale_seed=92 + d)
    sign = torch.where(inputs.dp_gaussian(rows * d, 93 + d, G.DEV).view(rows, d) > 0, 1.0, -1.0)
    scale = torch.tensor([1.0, 30.0, 1e-2, 1.0, 1e3, 1.0, 1.0], device=G.DEV).repeat(rows // 7 + 1)[:rows]
    x = x * sign * scale[:, None]
    x[3] = 0.0
    x[4] = -1.25
    x[5, 300:] = 0.0
    x[6] = inputs.quantize_mantissa(x[6], 1)
    x[7::50] = inputs.quantize_mantissa(x[7::50], 2)
    x[8] = 3.0e38
    x = x.to(torch.bfloat16).contiguous()
    gx = inputs.mp_gradients(rows, d, 94 + d, dtype=torch.bfloat16, device=G.DEV)
    for k in sorted({1, 33, d // 20, d // 8, min(d // 4 + 1, 2299), 3 * d // 8}):
        cols = _compare_fwd_bwd(x, gx, d, k, want_rows=(k == 33))
        assert int(cols.max()) < d
