"""Seeded synthetic inputs shaped like the paper's workloads.

This module serves both the CUDA path's tests/benchmark and the CPU oracle's
tests.  It holds none of the method's arithmetic: it only draws random
gradients and activations.  Every generator takes a seed and a torch device and
is deterministic for that (seed, device kind) pair; a test always hands the very
same buffer to both sides, so parity never depends on regenerating an input.

Shapes follow the experiments of the paper: gradient vectors of fully connected
layers compressed at 95-99.99 % sparsity (Sec. 2.1, Sec. 3.3), activations taken
after a ReLU so that about half of the entries are exactly zero (Remark 1), of
which a few per cent are kept per sample (Sec. 2.2).
"""
from __future__ import annotations

import math
from typing import List, Tuple

import torch

# One repeat of the DLRM-like dense stack: (fan_out, fan_in) of every weight
# matrix of a bottom MLP 512-256-64 and a top MLP 1024-1024-512-256-1.
DLRM_LIKE_LAYERS: List[Tuple[int, int]] = [
    (256, 512), (64, 256),
    (1024, 1024), (512, 1024), (256, 512), (1, 256),
]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def dp_gaussian(n: int, seed: int, device="cpu") -> torch.Tensor:
    """fp32 gradient vector ~ N(0, 1)."""
    return torch.randn(n, generator=_gen(seed, device), device=device, dtype=torch.float32)


def dp_mixture(n: int, seed: int, device="cpu", chunk: int = 1 << 27) -> torch.Tensor:
    """fp32 gradient vector ~ 0.99 N(0, 1e-4) + 0.01 N(0, 1), drawn in chunks to bound temporaries."""
    g = _gen(seed, device)
    out = torch.empty(n, device=device, dtype=torch.float32)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        z = torch.randn(m, generator=g, device=device, dtype=torch.float32)
        u = torch.rand(m, generator=g, device=device, dtype=torch.float32)
        out[lo:lo + m] = torch.where(u < 0.01, z, z * 0.01)
    return out


def dlrm_like_scale(n: int, device="cpu") -> torch.Tensor:
    """Per-element 1/sqrt(fan_in) of the concatenated dense-layer blocks, tiled to n elements."""
    parts = [torch.full((fo * fi,), 1.0 / math.sqrt(fi), dtype=torch.float32, device=device)
             for fo, fi in DLRM_LIKE_LAYERS]
    one = torch.cat(parts)
    reps = (n + one.numel() - 1) // one.numel()
    return one.repeat(reps)[:n].contiguous()


def dp_dlrm_like(n: int, seed: int, device="cpu", chunk: int = 1 << 26) -> torch.Tensor:
    """fp32 gradients of concatenated dense layers: Student-t(nu=3) scaled per block by 1/sqrt(fan_in)."""
    g = _gen(seed, device)
    scale = dlrm_like_scale(n, device)
    out = torch.empty(n, device=device, dtype=torch.float32)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        z = torch.randn(4, m, generator=g, device=device, dtype=torch.float32)
        t3 = z[0] / torch.sqrt((z[1] * z[1] + z[2] * z[2] + z[3] * z[3]) / 3.0)
        out[lo:lo + m] = t3 * scale[lo:lo + m]
    return out


def mp_activations(rows: int, d: int, seed: int, dtype=torch.float32, device="cpu",
                   col_scale_seed=None, ld=None) -> torch.Tensor:
    """Post-ReLU activation matrix [rows, ld]: max(N(0,1), +0) times an optional per-column
    LogNormal(0,1) scale, rounded to ``dtype``.  Columns d..ld-1 (padding) are filled with a
    large value so that a kernel that reads past d is caught."""
    ld = d if ld is None else ld
    x = torch.randn(rows, d, generator=_gen(seed, device), device=device, dtype=torch.float32)
    x = torch.clamp_min(x, 0.0) + 0.0  # +0.0 for clipped entries
    if col_scale_seed is not None:
        c = torch.exp(torch.randn(d, generator=_gen(col_scale_seed, device), device=device,
                                  dtype=torch.float32))
        x = x * c
    out = torch.full((rows, ld), 1.0e30, device=device, dtype=torch.float32)
    out[:, :d] = x
    return out.to(dtype).contiguous()


def mp_gradients(rows: int, d: int, seed: int, dtype=torch.float32, device="cpu", ld=None) -> torch.Tensor:
    """Backward gradient matrix [rows, ld] ~ N(0,1), rounded to ``dtype``."""
    ld = d if ld is None else ld
    x = torch.randn(rows, ld, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return x.to(dtype).contiguous()


def quantize_mantissa(x: torch.Tensor, keep_bits: int) -> torch.Tensor:
    """Round-toward-zero fp32 values to ``keep_bits`` mantissa bits: a cheap way to force many ties."""
    assert x.dtype == torch.float32
    mask = -(1 << (23 - keep_bits))
    return (x.view(torch.int32) & mask).view(torch.float32)
