"""Seeded random sweep of shapes, survivor targets, dtypes, strides, alignments and value patterns:
every case is compared with the oracle bit for bit.  The fixed cases of the other test files aim at
known corners; this file looks for the unknown ones (a shape that straddles two code paths, an odd
combination of stride and width, a value pattern nobody thought of)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2010_08899_b200 import binding as B
from paper_2010_08899_b200 import inputs
from tests import _gpu as G
from tests._util import bits32

pytestmark = pytest.mark.gpu

# DCT_SWEEP_SEED=<int> in the environment runs the sweep on another set of cases
SEED = int(os.environ.get("DCT_SWEEP_SEED", "0"))


def _mp_case(rng: np.random.Generator, case: int):
    dtype = torch.float32 if rng.integers(2) else torch.bfloat16
    # widths: the warp-per-row widths (multiples of 256) and their neighbours, plus anything else
    pick = rng.integers(4)
    if pick == 0:
        d = 256 * int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 10, 12, 14, 16]))
    elif pick == 1:
        d = 256 * int(rng.integers(1, 17)) + int(rng.integers(-3, 4))
    elif pick == 2:
        d = int(rng.integers(1, 300))
    else:
        d = int(rng.integers(300, 9000))
    d = max(1, d)
    ld = d + (int(rng.integers(0, 3)) * int(rng.choice([1, 4, 8])) if rng.integers(2) else 0)
    rows = int(rng.integers(1, 700)) if d <= 4096 else int(rng.integers(1, 40))
    if d <= 2048 and rng.integers(6) == 0:              # enough rows that every warp meets several in a row
        rows = int(rng.integers(4000, 12000))
    kmode = rng.integers(5)
    k = [1, max(1, d // 20), max(1, d // 8), max(1, d // 4), int(rng.integers(1, d + 1))][kmode]
    k = min(k + int(rng.integers(0, 2)), d)
    x = inputs.mp_activations(rows, d, 1000 + case, dtype=torch.float32, device=G.DEV,
                              col_scale_seed=(2000 + case) if rng.integers(2) else None, ld=ld)
    pattern = rng.integers(5)
    if pattern == 1:                                   # signed
        x = x * torch.where(inputs.dp_gaussian(rows * ld, 3000 + case, G.DEV).view(rows, ld) > 0, 1.0, -1.0)
    elif pattern == 2:                                 # coarse values: many ties
        x = inputs.quantize_mantissa(x, int(rng.integers(1, 6)))
    elif pattern == 3:                                 # row scales over many binades
        x = x * torch.pow(2.0, torch.randint(-30, 30, (rows, 1), device=G.DEV,
                                             generator=torch.Generator(G.DEV).manual_seed(case)).float())
    elif pattern == 4:                                 # mostly dead rows
        x = x * (inputs.dp_gaussian(rows * ld, 4000 + case, G.DEV).view(rows, ld) > 1.0)
    x = x.to(dtype).contiguous()
    gx = inputs.mp_gradients(rows, d, 5000 + case, dtype=dtype, device=G.DEV, ld=ld)
    if rng.integers(4) == 0:                           # rows that start off a 16-byte boundary
        x = G.offset_copy(x, int(rng.integers(1, 4))).view(rows, ld)
        gx = G.offset_copy(gx, int(rng.integers(1, 4))).view(rows, ld)
    return x, gx, d, k


@pytest.mark.parametrize("chunk", range(16))
def test_mp_random_cases(chunk):
    rng = np.random.default_rng(100 + chunk + 1000 * SEED)
    for case in range(chunk * 12 + 10000 * SEED, chunk * 12 + 12 + 10000 * SEED):
        x, gx, d, k = _mp_case(rng, case)
        what = f"case {case}: {tuple(x.shape)} d={d} k={k} {x.dtype}"
        want = oracle.mp_fwd(G.to_oracle(x), k, d=d)
        cols, vals, tau, _ = G.mp_fwd(x, d, k)
        assert np.array_equal(cols.cpu().numpy(), want.cols), what
        assert np.array_equal(G.as_np_bits(vals), want.vals.view(G.as_np_bits(vals).dtype)), what
        assert np.array_equal(G.as_np_bits(tau), want.tau.view(G.as_np_bits(tau).dtype)), what
        gv, r = G.mp_bwd(gx, d, cols)
        assert r.status == B.DCT_OK, what
        want_g = oracle.mp_bwd(G.to_oracle(gx), want.cols, d=d)
        assert np.array_equal(G.as_np_bits(gv), want_g.view(G.as_np_bits(gv).dtype)), what


@pytest.mark.parametrize("chunk", range(10))
def test_dp_random_cases(chunk):
    rng = np.random.default_rng(200 + chunk + 1000 * SEED)
    for case in range(chunk * 6 + 10000 * SEED, chunk * 6 + 6 + 10000 * SEED):
        n = int(rng.choice([int(rng.integers(1, 5000)), int(rng.integers(5000, 200_000)),
                            4096 * int(rng.integers(1, 300)) + int(rng.integers(-2, 3)),
                            int(rng.integers(200_000, 3_000_000))]))
        n = max(1, n)
        gen = [inputs.dp_gaussian, inputs.dp_mixture, inputs.dp_dlrm_like][int(rng.integers(3))]
        off = int(rng.integers(0, 4)) if rng.integers(3) == 0 else 0
        g = G.offset_copy(gen(n, 6000 + case, G.DEV), off)
        e0 = G.offset_copy(0.3 * inputs.dp_gaussian(n, 7000 + case, G.DEV), off)
        if rng.integers(3) == 0:
            g = inputs.quantize_mantissa(g, int(rng.integers(1, 8)))
        k = int([1, max(1, n // 1000), max(1, n // 50), max(1, n // 3), n][int(rng.integers(5))])
        what = f"case {case}: n={n} k={k} offset={off} {gen.__name__}"
        tau_dev, r = G.select(g, e0, k)
        want = oracle.dp_select(g.cpu().numpy(), e0.cpu().numpy(), k)
        assert bits32(tau_dev.cpu().numpy())[0] == bits32(want.tau)[0], what
        assert (r.n_gt, r.n_eq) == (want.n_gt, want.n_eq), what
        budget = None if rng.integers(2) else k - r.n_gt
        cap = int([n, max(1, k // 2), k + 7][int(rng.integers(3))])
        e_dev = e0.clone()
        e_cpu = e0.cpu().numpy().copy()
        w = oracle.dp_compress(g.cpu().numpy(), e_cpu, want.tau, budget, cap)
        idx, val, rr = G.compress(g, e_dev, tau_dev, budget, cap)
        assert (rr.count, rr.needed) == (w.count, w.needed), what
        assert rr.status == (B.DCT_OK if w.needed <= cap else B.DCT_ERR_CAPACITY), what
        assert np.array_equal(idx, w.idx[:w.count]) and np.array_equal(bits32(val), bits32(w.val[:w.count])), what
        assert np.array_equal(bits32(e_dev.cpu().numpy()), bits32(e_cpu)), what
