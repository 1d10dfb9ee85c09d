"""Helpers for the GPU parity tests: call the C ABI through the binding with guard words
around every output buffer, and bring results to numpy for comparison with the oracle."""
import numpy as np
import torch

from paper_2010_08899_b200 import binding as B

GUARD = 64            # guard elements after every output buffer
DEV = "cuda"


def _guarded(n, dtype, fill):
    t = torch.full((n + GUARD,), fill, dtype=dtype, device=DEV)
    return t


def _guard_ok(t, n, fill):
    return bool((t[n:] == fill).all().item())


def offset_copy(t: torch.Tensor, offset_elems: int) -> torch.Tensor:
    """A device copy of ``t`` that starts ``offset_elems`` elements past a 256-byte boundary."""
    buf = torch.empty(t.numel() + offset_elems + 64, dtype=t.dtype, device=DEV)
    base = (-buf.data_ptr() % 256) // t.element_size()
    view = buf[base + offset_elems: base + offset_elems + t.numel()]
    view.copy_(t.reshape(-1))
    return view


def select(grad: torch.Tensor, residual, k: int):
    n = grad.numel()
    tau = _guarded(1, torch.float32, -7.0)
    res = B.new_result()
    ws = B.new_workspace(B.dct_threshold_select_workspace_bytes(n))
    B.dct_threshold_select(grad, residual, n, k, tau, res, ws)
    r = B.read_result(res)
    assert r.status == B.DCT_OK
    assert _guard_ok(tau, 1, -7.0)
    return tau[:1], r


def compress(grad, residual, tau_dev, budget, capacity, ws=None):
    """Runs dct_dp_compress in place on ``residual``; returns (idx, val, Result) as numpy."""
    n = grad.numel()
    idx = _guarded(capacity, torch.int32, -12345)
    val = _guarded(capacity, torch.float32, -777.0)
    res = B.new_result()
    if ws is None:
        ws = B.new_workspace(B.dct_dp_compress_workspace_bytes(n))
    bud = None if budget is None else torch.tensor([budget], dtype=torch.int64, device=DEV)
    B.dct_dp_compress(grad, residual, n, tau_dev, bud, idx, val, capacity, res, ws)
    r = B.read_result(res)
    assert _guard_ok(idx, capacity, -12345) and _guard_ok(val, capacity, -777.0), "write past capacity"
    # entries at and beyond count are untouched
    assert bool((idx[r.count:capacity] == -12345).all().item())
    return idx[:r.count].cpu().numpy(), val[:r.count].cpu().numpy(), r


def mp_fwd(x: torch.Tensor, d: int, k: int, want_rows=False, want_tau=True):
    rows, ld = x.shape
    cols = _guarded(rows * k, torch.int16, -1)
    vals = _guarded(rows * k, x.dtype, 99.0)
    rws = _guarded(rows * k, torch.int32, -5) if want_rows else None
    tau = _guarded(rows, x.dtype, 99.0) if want_tau else None
    res = B.new_result()
    B.dct_mp_topk_pack_fwd(x, rows, d, ld, k, cols, vals, rws, tau, res)
    assert B.read_result(res).status == B.DCT_OK
    assert _guard_ok(cols, rows * k, -1) and _guard_ok(vals, rows * k, 99.0)
    if tau is not None:
        assert _guard_ok(tau, rows, 99.0)
    if rws is not None:
        assert _guard_ok(rws, rows * k, -5)
    return cols[:rows * k].view(rows, k), vals[:rows * k].view(rows, k), \
        (None if tau is None else tau[:rows]), (None if rws is None else rws[:rows * k].view(rows, k))


def mp_bwd(gx: torch.Tensor, d: int, cols: torch.Tensor):
    rows, ld = gx.shape
    k = cols.shape[1]
    gv = _guarded(rows * k, gx.dtype, 99.0)
    res = B.new_result()
    B.dct_mp_pack_bwd(gx, rows, d, ld, k, cols.contiguous(), gv, res)
    r = B.read_result(res)
    assert _guard_ok(gv, rows * k, 99.0)
    return gv[:rows * k].view(rows, k), r


def as_np_bits(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> numpy array of its bit patterns (uint32 for fp32, uint16 for bf16)."""
    t = t.contiguous().cpu()
    if t.dtype == torch.float32:
        return t.numpy().view(np.uint32)
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    raise TypeError(t.dtype)


def to_oracle(t: torch.Tensor) -> np.ndarray:
    """Device tensor -> the array type the oracle takes (float32, or uint16 bits for bf16)."""
    t = t.contiguous().cpu()
    if t.dtype == torch.float32:
        return t.numpy()
    return t.view(torch.int16).numpy().view(np.uint16)
