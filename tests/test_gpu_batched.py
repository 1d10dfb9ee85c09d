"""dct_dp_compress_batched: every layer of a batched call must come out exactly as the oracle's (and the
single-vector call's) result for that layer -- own threshold, own error, own output, own counts."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import binding as B
from paper_2010_08899_b200 import inputs
from tests import _gpu as G
from tests._util import bits32

pytestmark = pytest.mark.gpu


def _make_layers(sizes, seed, misalign=(), dense=False):
    layers = []
    for j, n in enumerate(sizes):
        g = inputs.dp_gaussian(n, seed + 3 * j, G.DEV) * (0.1 + j % 5)
        e = inputs.dp_gaussian(n, seed + 3 * j + 1, G.DEV) * 0.2
        if j in misalign:
            g, e = G.offset_copy(g, 1), G.offset_copy(e, 3)
        k = max(1, n // (20 + 7 * (j % 4)))
        if dense:
            k = max(1, n // (1 + j % 5))                      # all, a half, a third, ... of the elements pass
        tau, sel = G.select(g, e, k)
        cap = n if j % 3 else max(1, k // 2)                 # every third layer overflows its capacity
        budget = None if j % 2 else torch.tensor([k - sel.n_gt], dtype=torch.int64, device=G.DEV)
        layers.append(dict(grad=g, residual=e, n=n, tau=tau.clone(), tie_budget=budget, capacity=cap,
                           idx_out=torch.full((cap + 8,), -7, dtype=torch.int32, device=G.DEV),
                           val_out=torch.full((cap + 8,), -7.0, device=G.DEV), result=B.new_result()))
    return layers


@pytest.mark.parametrize("sizes,misalign", [
    ([1], ()), ([5000], ()), ([4096, 4096], ()),
    ([131072, 16384, 1048576, 524288, 131072, 256, 3, 8191, 12289], ()),        # DLRM-like mix plus odd sizes
    ([70001, 4096 * 3, 100, 262144 + 5, 9999], (0, 3)),                         # some layers not 16-byte aligned
    ([(1 << 20) + 17] * 3 + [64] * 40, (41,)),
])
def test_batched_equals_per_layer_oracle(sizes, misalign):
    layers = _make_layers(sizes, 1000 + len(sizes), misalign)
    want = []
    for a in layers:
        e = a["residual"].cpu().numpy().copy()
        bud = None if a["tie_budget"] is None else int(a["tie_budget"].item())
        want.append((oracle.dp_compress(a["grad"].cpu().numpy(), e, a["tau"].cpu().numpy()[0], bud, a["capacity"]), e))
    ws = B.new_workspace(B.dct_dp_compress_batched_workspace_bytes(sizes))
    ws.fill_(0xAB)                                            # stale workspace contents must not matter
    B.dct_dp_compress_batched(layers, ws)
    for a, (w, e_want) in zip(layers, want):
        r = B.read_result(a["result"])
        cap = a["capacity"]
        assert (r.count, r.needed) == (w.count, w.needed)
        assert r.status == (B.DCT_ERR_CAPACITY if w.needed > cap else B.DCT_OK)
        assert np.array_equal(a["idx_out"][:r.count].cpu().numpy(), w.idx)
        assert np.array_equal(bits32(a["val_out"][:r.count].cpu().numpy()), bits32(w.val))
        assert bool((a["idx_out"][r.count:] == -7).all()) and bool((a["val_out"][r.count:] == -7.0).all())
        assert np.array_equal(bits32(a["residual"].cpu().numpy()), bits32(e_want))


def test_batched_dense_layers_many_tiles_per_cta():
    """Layers of up to a thousand tiles in which a fifth to all of the elements pass: the ring of the streaming
    kernel fills up and the tiles a waiting CTA counts ahead of their turn belong to the next layer now and then."""
    sizes = [(1 << 21) + 5, 1 << 22, 4096 * 700, (1 << 20) + 4096, 4096 * 3, 4096 * 333 + 1, 1 << 21]
    layers = _make_layers(sizes, 77, dense=True)
    ws = B.new_workspace(B.dct_dp_compress_batched_workspace_bytes(sizes))
    want = []
    for a in layers:
        e = a["residual"].cpu().numpy().copy()
        bud = None if a["tie_budget"] is None else int(a["tie_budget"].item())
        want.append((oracle.dp_compress(a["grad"].cpu().numpy(), e, a["tau"].cpu().numpy()[0], bud, a["capacity"]), e))
    B.dct_dp_compress_batched(layers, ws)
    for a, (w, e_want) in zip(layers, want):
        r = B.read_result(a["result"])
        assert (r.count, r.needed) == (w.count, w.needed)
        assert r.status == (B.DCT_ERR_CAPACITY if w.needed > a["capacity"] else B.DCT_OK)
        assert np.array_equal(a["idx_out"][:r.count].cpu().numpy(), w.idx)
        assert np.array_equal(bits32(a["val_out"][:r.count].cpu().numpy()), bits32(w.val))
        assert np.array_equal(bits32(a["residual"].cpu().numpy()), bits32(e_want))


@pytest.mark.parametrize("dense", [False, True])
def test_batched_layers_inside_two_flat_buffers(dense):
    """The layers of a model as views into one flat gradient buffer and one flat residual buffer: an odd-sized tensor
    shifts every layer behind it off the 16-byte boundaries, gradient and residual alike.  Every layer must come out as
    the oracle's, and what lies between the layers (and before the first, after the last) must be left alone."""
    sizes = [4096 * 3 + 1, 250, 1 << 20, 7, 65536 + 3, 4096, 100_000, 4095, 4096 * 2 + 2, (1 << 21) + 5, 33]
    gaps = [0, 1, 0, 0, 2, 0, 0, 3, 0, 0, 0]            # unused elements behind a layer (another tensor's, say)
    total = sum(sizes) + sum(gaps) + 8
    g_flat = inputs.dp_gaussian(total, 501, G.DEV)
    e_flat = inputs.dp_gaussian(total, 502, G.DEV) * 0.2
    e_before = e_flat.clone()
    layers, spans, off = [], [], 1                      # the first layer starts one element into the buffers
    for j, (n, gap) in enumerate(zip(sizes, gaps)):
        g, e = g_flat[off:off + n], e_flat[off:off + n]
        assert g.data_ptr() % 16 == e.data_ptr() % 16
        k = max(1, n // (3 if dense else 40))
        tau, sel = G.select(g, e, k)
        cap = n if j % 3 else max(1, k // 2)
        budget = None if j % 2 else torch.tensor([k - sel.n_gt], dtype=torch.int64, device=G.DEV)
        layers.append(dict(grad=g, residual=e, n=n, tau=tau.clone(), tie_budget=budget, capacity=cap,
                           idx_out=torch.full((cap + 8,), -7, dtype=torch.int32, device=G.DEV),
                           val_out=torch.full((cap + 8,), -7.0, device=G.DEV), result=B.new_result()))
        spans.append((off, off + n))
        off += n + gap
    # the thresholds of all layers in one batched select, from the same views
    sel_layers = [dict(grad=a["grad"], residual=a["residual"], n=a["n"], k=max(1, a["n"] // (3 if dense else 40)),
                       tau_out=torch.zeros(1, device=G.DEV), result=B.new_result()) for a in layers]
    ws_sel = B.new_workspace(B.dct_threshold_select_batched_workspace_bytes(len(sizes)))
    B.dct_threshold_select_batched(sel_layers, ws_sel)
    for a, sl in zip(layers, sel_layers):
        w = oracle.dp_select(a["grad"].cpu().numpy(), a["residual"].cpu().numpy(), sl["k"])
        r = B.read_result(sl["result"])
        assert bits32(sl["tau_out"].cpu().numpy())[0] == bits32(w.tau)[0] and (r.n_gt, r.n_eq) == (w.n_gt, w.n_eq)
    want = []
    for a in layers:
        e = a["residual"].cpu().numpy().copy()
        bud = None if a["tie_budget"] is None else int(a["tie_budget"].item())
        want.append((oracle.dp_compress(a["grad"].cpu().numpy(), e, a["tau"].cpu().numpy()[0], bud, a["capacity"]), e))
    ws = B.new_workspace(B.dct_dp_compress_batched_workspace_bytes(sizes))
    ws.fill_(0xCD)
    B.dct_dp_compress_batched(layers, ws)
    for a, (w, e_want) in zip(layers, want):
        r = B.read_result(a["result"])
        assert (r.count, r.needed) == (w.count, w.needed)
        assert r.status == (B.DCT_ERR_CAPACITY if w.needed > a["capacity"] else B.DCT_OK)
        assert np.array_equal(a["idx_out"][:r.count].cpu().numpy(), w.idx)
        assert np.array_equal(bits32(a["val_out"][:r.count].cpu().numpy()), bits32(w.val))
        assert bool((a["idx_out"][r.count:] == -7).all())
        assert np.array_equal(bits32(a["residual"].cpu().numpy()), bits32(e_want))
    outside = torch.ones(total, dtype=torch.bool, device=G.DEV)
    for lo, hi in spans:
        outside[lo:hi] = False
    assert torch.equal(e_flat[outside], e_before[outside])


def test_batched_rejects_bad_layers_on_the_host():
    layers = _make_layers([5000, 6000], 7)
    ws = B.new_workspace(B.dct_dp_compress_batched_workspace_bytes([5000, 6000]))
    with pytest.raises(B.DctError):
        B.dct_dp_compress_batched(layers, ws[:256])
    bad = dict(layers[1])
    bad["residual"] = bad["grad"]                              # aliasing
    with pytest.raises(B.DctError):
        B.dct_dp_compress_batched([layers[0], bad], ws)
    assert B.dct_dp_compress_batched_workspace_bytes([0]) == 0


def _select_layers(sizes, seed, misalign=(), with_residual=True):
    layers = []
    for j, n in enumerate(sizes):
        g = inputs.dp_dlrm_like(n, seed + 3 * j, G.DEV) * (0.1 + j % 5) if n > 64 else inputs.dp_gaussian(n, seed + 3 * j, G.DEV)
        e = inputs.dp_gaussian(n, seed + 3 * j + 1, G.DEV) * 0.05 if (with_residual and j % 3 != 2) else None
        if j % 4 == 1:
            g = inputs.quantize_mantissa(g, 3)                  # heavy ties in some layers
        if j in misalign:
            g = G.offset_copy(g, 1)
            e = None if e is None else G.offset_copy(e, 3)
        k = [1, max(1, n // 1000), max(1, n // 20), max(1, n // 4), n][j % 5]
        layers.append(dict(grad=g, residual=e, n=n, k=k, tau_out=torch.full((3,), -7.0, device=G.DEV),
                           result=B.new_result()))
    return layers


@pytest.mark.parametrize("sizes,misalign", [
    ([1], ()), ([8192], ()), ([8193, 1, 8191], ()),
    ([131072, 16384, 1048576, 524288, 131072, 256, 3, 8191, 12289], ()),        # DLRM-like mix plus odd sizes
    ([70001, 4096 * 3, 100, 262144 + 5, 9999], (0, 3)),                         # some layers not 16-byte aligned
    ([(1 << 21) + 17] * 2 + [64] * 300, (41,)),                                 # more layers than CTAs, tiny ones
])
def test_batched_select_equals_per_layer_oracle(sizes, misalign):
    """dct_threshold_select_batched: every layer's threshold and counts as the oracle (and the single-vector
    select) give them for that layer alone."""
    layers = _select_layers(sizes, 3000 + len(sizes), misalign)
    ws = B.new_workspace(B.dct_threshold_select_batched_workspace_bytes(len(sizes)))
    ws.fill_(0xCD)                                            # stale workspace contents must not matter
    B.dct_threshold_select_batched(layers, ws)
    for j, a in enumerate(layers):
        e = None if a["residual"] is None else a["residual"].cpu().numpy()
        want = oracle.dp_select(a["grad"].cpu().numpy(), e, a["k"])
        r = B.read_result(a["result"])
        assert r.status == B.DCT_OK, j
        assert bits32(a["tau_out"][:1].cpu().numpy())[0] == bits32(want.tau)[0], j
        assert (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq), j
        assert bool((a["tau_out"][1:] == -7.0).all()), j
    # the same call again on the same workspace gives the same answer
    first = [a["tau_out"][:1].clone() for a in layers]
    B.dct_threshold_select_batched(layers, ws)
    assert all(torch.equal(a["tau_out"][:1], t) for a, t in zip(layers, first))


def test_batched_select_feeds_batched_compress():
    """The layer-wise scheme end to end: thresholds of all layers in one call, then all layers compressed in
    one call with the tie budgets k - n_gt: exactly k survivors per layer."""
    sizes = [131072, 16384, 262144, 65536, 131072, 256]
    sel = _select_layers(sizes, 4000, with_residual=True)
    for a in sel:
        a["k"] = max(1, a["n"] // 100)
        if a["residual"] is None:
            a["residual"] = torch.zeros(a["n"], device=G.DEV)
    B.dct_threshold_select_batched(sel, B.new_workspace(B.dct_threshold_select_batched_workspace_bytes(len(sizes))))
    layers = []
    for a in sel:
        r = B.read_result(a["result"])
        budget = torch.tensor([a["k"] - r.n_gt], dtype=torch.int64, device=G.DEV)
        layers.append(dict(grad=a["grad"], residual=a["residual"], n=a["n"], tau=a["tau_out"][:1].clone(),
                           tie_budget=budget, capacity=a["n"],
                           idx_out=torch.empty(a["n"], dtype=torch.int32, device=G.DEV),
                           val_out=torch.empty(a["n"], device=G.DEV), result=B.new_result()))
    B.dct_dp_compress_batched(layers, B.new_workspace(B.dct_dp_compress_batched_workspace_bytes(sizes)))
    for a, s in zip(layers, sel):
        r = B.read_result(a["result"])
        assert (r.status, r.count, r.needed) == (B.DCT_OK, s["k"], s["k"])


def test_batched_select_rejects_bad_layers_on_the_host():
    g = inputs.dp_gaussian(100, 1, G.DEV)
    ok = dict(grad=g, residual=None, n=100, k=5, tau_out=torch.zeros(1, device=G.DEV), result=B.new_result())
    ws = B.new_workspace(B.dct_threshold_select_batched_workspace_bytes(2))
    for bad in (dict(ok, k=0), dict(ok, k=101), dict(ok, n=0)):
        with pytest.raises(B.DctError):
            B.dct_threshold_select_batched([ok, bad], ws)
    with pytest.raises(B.DctError):
        B.dct_threshold_select_batched([ok, ok], ws[:256])
