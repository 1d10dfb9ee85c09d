"""Python binding of the C ABI in ``include/dct.h``: argument marshalling only.

Every function here has the name and the argument order of its C counterpart,
takes torch tensors (used purely as device or host buffers), checks dtype and
contiguity, and passes raw pointers to ``libdct_b200.so``.  No step of the
method runs in Python or in PyTorch.  If the shared library cannot be loaded
the import of a symbol fails loudly: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import NamedTuple, Optional

import torch

from . import build as _build

DCT_OK, DCT_ERR_INVALID_ARG, DCT_ERR_WORKSPACE, DCT_ERR_UNSUPPORTED = 0, 1, 2, 3
DCT_ERR_CUDA, DCT_ERR_CAPACITY, DCT_ERR_TIMEOUT, DCT_ERR_BAD_MASK = 4, 5, 6, 7
DCT_F32, DCT_BF16 = 0, 1

RESULT_BYTES = 40          # sizeof(dct_result_t)

# every symbol include/dct.h declares
EXPORTED_SYMBOLS = (
    "dct_status_string", "dct_last_cuda_error",
    "dct_threshold_select_workspace_bytes", "dct_dp_compress_workspace_bytes",
    "dct_threshold_select", "dct_dp_compress", "dct_mp_topk_pack_fwd", "dct_mp_pack_bwd",
    "dct_dp_compress_host", "dct_mp_pack_host", "dct_threshold_select_host", "dct_debug_configure",
    "dct_dp_compress_static", "dct_dp_decompress", "dct_mp_unpack",
    "dct_dp_select_compress", "dct_dp_select_compress_workspace_bytes",
    "dct_dp_compress_batched", "dct_dp_compress_batched_workspace_bytes",
    "dct_threshold_select_multi", "dct_threshold_select_multi_workspace_bytes",
    "dct_mp_threshold_mean", "dct_dp_drift_check",
    "dct_threshold_select_batched", "dct_threshold_select_batched_workspace_bytes",
    "dct_threshold_select_shard_workspace_bytes", "dct_threshold_select_shard_begin",
    "dct_threshold_select_shard_pass", "dct_threshold_select_shard_advance",
    "dct_threshold_select_shard_sampled_workspace_bytes", "dct_threshold_select_shard_sampled_begin",
    "dct_threshold_select_shard_sampled_pass", "dct_threshold_select_shard_sampled_advance",
)

_vp, _u64, _u32, _sz, _int = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_size_t, ctypes.c_int
_lib = None


class DctError(RuntimeError):
    def __init__(self, where: str, status: int):
        self.status = status
        name = lib().dct_status_string(status).decode()
        extra = ""
        if status == DCT_ERR_CUDA:
            extra = ": " + lib().dct_last_cuda_error().decode()
        super().__init__(f"{where}: {name}{extra}")


def library_path() -> str:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """Load (building first if the sources are newer) the CUDA library.  Raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing and could not be built: the DCT kernels have no fallback")
    L = ctypes.CDLL(path)
    L.dct_status_string.restype = ctypes.c_char_p
    L.dct_status_string.argtypes = [_int]
    L.dct_last_cuda_error.restype = ctypes.c_char_p
    L.dct_last_cuda_error.argtypes = []
    for f in (L.dct_threshold_select_workspace_bytes, L.dct_dp_compress_workspace_bytes):
        f.restype = _sz
        f.argtypes = [_u64]
    L.dct_threshold_select.restype = _int
    L.dct_threshold_select.argtypes = [_vp, _vp, _u64, _u64, _vp, _vp, _vp, _sz, _vp]
    L.dct_dp_compress.restype = _int
    L.dct_dp_compress.argtypes = [_vp, _vp, _u64, _vp, _vp, _vp, _vp, _u64, _vp, _vp, _sz, _vp]
    L.dct_dp_select_compress_workspace_bytes.restype = _sz
    L.dct_dp_select_compress_workspace_bytes.argtypes = [_u64]
    L.dct_dp_select_compress.restype = _int
    L.dct_dp_select_compress.argtypes = [_vp, _vp, _u64, _u64, _vp, _vp, _vp, _u64, _vp, _vp, _sz, _vp]
    L.dct_dp_compress_batched_workspace_bytes.restype = _sz
    L.dct_dp_compress_batched_workspace_bytes.argtypes = [_vp, _u32]
    L.dct_dp_compress_batched.restype = _int
    L.dct_dp_compress_batched.argtypes = [_vp, _u32, _vp, _sz, _vp]
    L.dct_dp_decompress.restype = _int
    L.dct_dp_decompress.argtypes = [_vp, _vp, _vp, _u64, _vp, _u64, _int, _vp, _vp]
    L.dct_mp_unpack.restype = _int
    L.dct_mp_unpack.argtypes = [_vp, _vp, _int, _u32, _u32, _u32, _u32, _vp, _vp, _vp]
    L.dct_dp_compress_static.restype = _int
    L.dct_dp_compress_static.argtypes = [_vp, _vp, _u64, _vp, _vp, _vp, _vp, _u64, _vp, _vp]
    L.dct_mp_topk_pack_fwd.restype = _int
    L.dct_mp_topk_pack_fwd.argtypes = [_vp, _int, _u32, _u32, _u32, _u32, _vp, _vp, _vp, _vp, _vp, _vp]
    L.dct_mp_pack_bwd.restype = _int
    L.dct_mp_pack_bwd.argtypes = [_vp, _int, _u32, _u32, _u32, _u32, _vp, _vp, _vp, _vp]
    L.dct_dp_compress_host.restype = _int
    L.dct_dp_compress_host.argtypes = [_vp, _vp, _vp, _u64, _vp, _vp, _vp, _vp, _u64, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
    L.dct_threshold_select_host.restype = _int
    L.dct_threshold_select_host.argtypes = [_vp, _vp, _vp, _u64, _u64, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
    L.dct_mp_pack_host.restype = _int
    L.dct_mp_pack_host.argtypes = [_vp, _vp, _vp, _vp, _int, _u32, _u32, _u32, _u32,
                                   _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
    L.dct_threshold_select_multi_workspace_bytes.restype = _sz
    L.dct_threshold_select_multi_workspace_bytes.argtypes = [_u64, _u32]
    L.dct_threshold_select_multi.restype = _int
    L.dct_threshold_select_multi.argtypes = [_vp, _vp, _u64, _vp, _u32, _vp, _vp, _vp, _sz, _vp]
    L.dct_mp_threshold_mean.restype = _int
    L.dct_mp_threshold_mean.argtypes = [_vp, _int, _u32, _u32, _u32, _vp, _u32, _vp, _vp, _vp]
    L.dct_dp_drift_check.restype = _int
    L.dct_dp_drift_check.argtypes = [_vp, _u64, _u32, _u32, _vp, _vp]
    L.dct_threshold_select_batched_workspace_bytes.restype = _sz
    L.dct_threshold_select_batched_workspace_bytes.argtypes = [_u32]
    L.dct_threshold_select_batched.restype = _int
    L.dct_threshold_select_batched.argtypes = [_vp, _u32, _vp, _sz, _vp]
    L.dct_threshold_select_shard_workspace_bytes.restype = _sz
    L.dct_threshold_select_shard_workspace_bytes.argtypes = []
    L.dct_threshold_select_shard_begin.restype = _int
    L.dct_threshold_select_shard_begin.argtypes = [_u64, _vp, _sz, _vp]
    L.dct_threshold_select_shard_pass.restype = _int
    L.dct_threshold_select_shard_pass.argtypes = [_vp, _vp, _u64, _u32, _vp, _vp, _vp]
    L.dct_threshold_select_shard_advance.restype = _int
    L.dct_threshold_select_shard_advance.argtypes = [_vp, _u32, _vp, _vp, _vp, _vp]
    L.dct_threshold_select_shard_sampled_workspace_bytes.restype = _sz
    L.dct_threshold_select_shard_sampled_workspace_bytes.argtypes = [_u64]
    L.dct_threshold_select_shard_sampled_begin.restype = _int
    L.dct_threshold_select_shard_sampled_begin.argtypes = [_u64, _u64, _u64, _vp, _sz, _vp]
    L.dct_threshold_select_shard_sampled_pass.restype = _int
    L.dct_threshold_select_shard_sampled_pass.argtypes = [_vp, _vp, _u64, _u32, _vp, _vp, _vp]
    L.dct_threshold_select_shard_sampled_advance.restype = _int
    L.dct_threshold_select_shard_sampled_advance.argtypes = [_vp, _u32, _vp, _vp, _vp, _vp]
    L.dct_debug_configure.restype = None
    L.dct_debug_configure.argtypes = [_u32, _u32]
    _lib = L
    return L


# ----------------------------------------------------------------------------
# marshalling helpers
# ----------------------------------------------------------------------------

def _p(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _need(t: torch.Tensor, dtype, name: str, cuda: bool = True):
    if t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if cuda and not t.is_cuda:
        raise ValueError(f"{name}: must be a CUDA tensor")
    if not cuda and t.is_cuda:
        raise ValueError(f"{name}: must be a host tensor")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DCT_F32
    if t.dtype == torch.bfloat16:
        return DCT_BF16
    raise TypeError(f"unsupported dtype {t.dtype}: float32 or bfloat16")


def _check(where: str, status: int):
    if status != DCT_OK:
        raise DctError(where, status)


class Result(NamedTuple):
    status: int
    count: int
    needed: int
    n_gt: int
    n_eq: int


def new_result(device="cuda") -> torch.Tensor:
    """A device buffer holding one dct_result_t."""
    return torch.zeros(RESULT_BYTES // 8, dtype=torch.int64, device=device)


def read_result(result: torch.Tensor) -> Result:
    """Copy a result block to the host (synchronises) and decode it."""
    r = result.cpu().tolist()
    return Result(r[0] & 0xFFFFFFFF, r[1], r[2], r[3], r[4])


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned device workspace of at least ``nbytes`` bytes."""
    t = torch.empty(max(nbytes, 256) + 256, dtype=torch.uint8, device=device)
    off = (-t.data_ptr()) % 256
    return t[off:off + max(nbytes, 256)]


def k_from_sparsity(n: int, eta_num: int, eta_den: int) -> int:
    """Survivor target for a sparsity factor eta = eta_num/eta_den (fraction dropped):
    k = n - floor(n * eta), in exact integer arithmetic (Algorithm 1 / 2, threshold index)."""
    if not (0 <= eta_num <= eta_den and eta_den > 0):
        raise ValueError("need 0 <= eta <= 1")
    return n - (n * eta_num) // eta_den


def k_from_density(n: int, den_num: int, den_den: int) -> int:
    """Survivor target for a kept fraction den_num/den_den: k = ceil(n * density)."""
    return -((-n * den_num) // den_den)


# ----------------------------------------------------------------------------
# the C entry points
# ----------------------------------------------------------------------------

def dct_threshold_select_workspace_bytes(n: int) -> int:
    return lib().dct_threshold_select_workspace_bytes(n)


def dct_dp_compress_workspace_bytes(n: int) -> int:
    return lib().dct_dp_compress_workspace_bytes(n)


def dct_threshold_select(grad, residual, n, k, tau_out, result, workspace, stream=None) -> None:
    _need(grad, torch.float32, "grad")
    if residual is not None:
        _need(residual, torch.float32, "residual")
    _need(tau_out, torch.float32, "tau_out")
    _need(result, torch.int64, "result")
    _need(workspace, torch.uint8, "workspace")
    if grad.numel() < n or (residual is not None and residual.numel() < n) or result.numel() * 8 < RESULT_BYTES:
        raise ValueError("buffer smaller than n")
    _check("dct_threshold_select",
           lib().dct_threshold_select(_p(grad), _p(residual), n, k, _p(tau_out), _p(result),
                                      _p(workspace), workspace.numel(), _stream(stream)))


def dct_dp_compress(grad, residual, n, tau, tie_budget, idx_out, val_out, capacity, result, workspace,
                    stream=None) -> None:
    _need(grad, torch.float32, "grad")
    _need(residual, torch.float32, "residual")
    _need(tau, torch.float32, "tau")
    if tie_budget is not None:
        _need(tie_budget, torch.int64, "tie_budget")
    _need(idx_out, torch.int32, "idx_out")
    _need(val_out, torch.float32, "val_out")
    _need(result, torch.int64, "result")
    _need(workspace, torch.uint8, "workspace")
    if grad.numel() < n or residual.numel() < n or idx_out.numel() < capacity or val_out.numel() < capacity:
        raise ValueError("buffer smaller than n / capacity")
    _check("dct_dp_compress",
           lib().dct_dp_compress(_p(grad), _p(residual), n, _p(tau), _p(tie_budget), _p(idx_out), _p(val_out),
                                 capacity, _p(result), _p(workspace), workspace.numel(), _stream(stream)))


DCT_DP_COMPRESS_STATIC_MAX_N = 1 << 27


def dct_dp_compress_static(grad, residual, n, tau, tie_budget, idx_out, val_out, capacity, result, stream=None) -> None:
    """dct_dp_compress for callers that have no workspace to give: the scratch is an array built into the
    library (n <= DCT_DP_COMPRESS_STATIC_MAX_N).  Calls on one device share that array, so do not let two
    of them overlap on the GPU; the first call per device should happen outside stream capture."""
    _need(grad, torch.float32, "grad")
    _need(residual, torch.float32, "residual")
    _need(tau, torch.float32, "tau")
    if tie_budget is not None:
        _need(tie_budget, torch.int64, "tie_budget")
    _need(idx_out, torch.int32, "idx_out")
    _need(val_out, torch.float32, "val_out")
    _need(result, torch.int64, "result")
    if n <= DCT_DP_COMPRESS_STATIC_MAX_N and (grad.numel() < n or residual.numel() < n or
                                              idx_out.numel() < capacity or val_out.numel() < capacity):
        raise ValueError("buffer smaller than n / capacity")
    _check("dct_dp_compress_static",
           lib().dct_dp_compress_static(_p(grad), _p(residual), n, _p(tau), _p(tie_budget), _p(idx_out),
                                        _p(val_out), capacity, _p(result), _stream(stream)))


def dct_mp_topk_pack_fwd(x_act, rows, d, ld, k, cols_out, vals_out, rows_out=None, tau_out=None, result=None,
                         stream=None) -> None:
    code = _dtype_code(x_act)
    _need(x_act, x_act.dtype, "x_act")
    _need(cols_out, torch.int16, "cols_out")
    _need(vals_out, x_act.dtype, "vals_out")
    if rows_out is not None:
        _need(rows_out, torch.int32, "rows_out")
    if tau_out is not None:
        _need(tau_out, x_act.dtype, "tau_out")
    if result is not None:
        _need(result, torch.int64, "result")
    if ld >= d and rows >= 1 and k >= 1:
        if (x_act.numel() < (rows - 1) * ld + d or cols_out.numel() < rows * k or vals_out.numel() < rows * k or
                (rows_out is not None and rows_out.numel() < rows * k) or
                (tau_out is not None and tau_out.numel() < rows)):
            raise ValueError("buffer smaller than rows x ld / rows x k")
    _check("dct_mp_topk_pack_fwd",
           lib().dct_mp_topk_pack_fwd(_p(x_act), code, rows, d, ld, k, _p(cols_out), _p(vals_out), _p(rows_out),
                                      _p(tau_out), _p(result), _stream(stream)))


def dct_mp_pack_bwd(x_grad, rows, d, ld, k, cols, gvals_out, result=None, stream=None) -> None:
    code = _dtype_code(x_grad)
    _need(x_grad, x_grad.dtype, "x_grad")
    _need(cols, torch.int16, "cols")
    _need(gvals_out, x_grad.dtype, "gvals_out")
    if result is not None:
        _need(result, torch.int64, "result")
    if ld >= d and rows >= 1 and k >= 1:
        if x_grad.numel() < (rows - 1) * ld + d or cols.numel() < rows * k or gvals_out.numel() < rows * k:
            raise ValueError("buffer smaller than rows x ld / rows x k")
    _check("dct_mp_pack_bwd",
           lib().dct_mp_pack_bwd(_p(x_grad), code, rows, d, ld, k, _p(cols), _p(gvals_out), _p(result),
                                 _stream(stream)))


def dct_dp_decompress(idx, val, packed, capacity, dense, n, accumulate, result, stream=None) -> None:
    _need(idx, torch.int32, "idx")
    _need(val, torch.float32, "val")
    _need(packed, torch.int64, "packed")
    _need(dense, torch.float32, "dense")
    _need(result, torch.int64, "result")
    if idx.numel() < capacity or val.numel() < capacity or dense.numel() < n:
        raise ValueError("buffer smaller than capacity / n")
    _check("dct_dp_decompress",
           lib().dct_dp_decompress(_p(idx), _p(val), _p(packed), capacity, _p(dense), n, 1 if accumulate else 0,
                                   _p(result), _stream(stream)))


def dct_mp_unpack(cols, vals, rows, d, ld, k, dense_out, result=None, stream=None) -> None:
    code = _dtype_code(vals)
    _need(cols, torch.int16, "cols")
    _need(vals, vals.dtype, "vals")
    _need(dense_out, vals.dtype, "dense_out")
    if result is not None:
        _need(result, torch.int64, "result")
    if ld >= d and rows >= 1 and k >= 1:
        if cols.numel() < rows * k or vals.numel() < rows * k or dense_out.numel() < (rows - 1) * ld + d:
            raise ValueError("buffer smaller than rows x k / rows x ld")
    _check("dct_mp_unpack",
           lib().dct_mp_unpack(_p(cols), _p(vals), code, rows, d, ld, k, _p(dense_out), _p(result), _stream(stream)))


def dct_dp_compress_host(grad_host, grad_dev, residual_dev, n, tau_dev, tie_budget_dev, idx_dev, val_dev, capacity,
                         idx_host, val_host, result_dev, result_host, workspace, stream=None) -> Result:
    """Returns the decoded host copy of the result block; DCT_ERR_CAPACITY is reported there, not raised."""
    _need(grad_host, torch.float32, "grad_host", cuda=False)
    _need(grad_dev, torch.float32, "grad_dev")
    _need(residual_dev, torch.float32, "residual_dev")
    _need(idx_host, torch.int32, "idx_host", cuda=False)
    _need(val_host, torch.float32, "val_host", cuda=False)
    _need(result_host, torch.int64, "result_host", cuda=False)
    _need(idx_dev, torch.int32, "idx_dev")
    _need(val_dev, torch.float32, "val_dev")
    if min(grad_host.numel(), grad_dev.numel(), residual_dev.numel()) < n or \
            min(idx_host.numel(), val_host.numel(), idx_dev.numel(), val_dev.numel()) < capacity:
        raise ValueError("buffer smaller than n / capacity")
    st = lib().dct_dp_compress_host(_p(grad_host), _p(grad_dev), _p(residual_dev), n, _p(tau_dev),
                                    _p(tie_budget_dev), _p(idx_dev), _p(val_dev), capacity, _p(idx_host),
                                    _p(val_host), _p(result_dev), _p(result_host), _p(workspace),
                                    workspace.numel(), _stream(stream))
    if st not in (DCT_OK, DCT_ERR_CAPACITY):
        raise DctError("dct_dp_compress_host", st)
    r = result_host.tolist()
    return Result(r[0] & 0xFFFFFFFF, r[1], r[2], r[3], r[4])


def dct_threshold_select_host(grad_host, grad_dev, residual_dev, n, k, tau_dev, tau_host, result_dev, result_host,
                              workspace, stream=None) -> Result:
    _need(grad_host, torch.float32, "grad_host", cuda=False)
    _need(grad_dev, torch.float32, "grad_dev")
    _need(tau_dev, torch.float32, "tau_dev")
    _need(result_host, torch.int64, "result_host", cuda=False)
    if min(grad_host.numel(), grad_dev.numel()) < n:
        raise ValueError("buffer smaller than n")
    _check("dct_threshold_select_host",
           lib().dct_threshold_select_host(_p(grad_host), _p(grad_dev), _p(residual_dev), n, k, _p(tau_dev),
                                           _p(tau_host), _p(result_dev), _p(result_host), _p(workspace),
                                           workspace.numel(), _stream(stream)))
    r = result_host.tolist()
    return Result(r[0] & 0xFFFFFFFF, r[1], r[2], r[3], r[4])


def dct_mp_pack_host(x_act_host, x_grad_host, x_act_dev, x_grad_dev, rows, d, ld, k, cols_dev, vals_dev, gvals_dev,
                     cols_host, vals_host, gvals_host, result_dev, result_host, stream=None) -> None:
    code = _dtype_code(x_act_host)
    for t, nm in ((x_act_host, "x_act_host"), (x_grad_host, "x_grad_host"), (vals_host, "vals_host"),
                  (gvals_host, "gvals_host")):
        _need(t, x_act_host.dtype, nm, cuda=False)
    for t, nm in ((x_act_dev, "x_act_dev"), (x_grad_dev, "x_grad_dev"), (vals_dev, "vals_dev"),
                  (gvals_dev, "gvals_dev")):
        _need(t, x_act_host.dtype, nm)
    _need(cols_dev, torch.int16, "cols_dev")
    _need(cols_host, torch.int16, "cols_host", cuda=False)
    _need(result_host, torch.int64, "result_host", cuda=False)
    if min(x_act_host.numel(), x_grad_host.numel(), x_act_dev.numel(), x_grad_dev.numel()) < rows * ld or \
            min(cols_dev.numel(), vals_dev.numel(), gvals_dev.numel(), cols_host.numel(), vals_host.numel(),
                gvals_host.numel()) < rows * k:
        raise ValueError("buffer smaller than rows x ld / rows x k")
    _check("dct_mp_pack_host",
           lib().dct_mp_pack_host(_p(x_act_host), _p(x_grad_host), _p(x_act_dev), _p(x_grad_dev), code, rows, d, ld,
                                  k, _p(cols_dev), _p(vals_dev), _p(gvals_dev), _p(cols_host), _p(vals_host),
                                  _p(gvals_host), _p(result_dev), _p(result_host), _stream(stream)))


def dct_debug_configure(spin_limit: int = 1 << 21, first_ticket: int = 0) -> None:
    """Testing knobs: iteration limit of device-side waits, and the first tile ticket of dct_dp_compress
    (a non-zero value leaves tile 0 unprocessed so that the bounded wait can be seen to give up)."""
    lib().dct_debug_configure(spin_limit, first_ticket)


def dct_dp_select_compress_workspace_bytes(n: int) -> int:
    return lib().dct_dp_select_compress_workspace_bytes(n)


def dct_dp_select_compress(grad, residual, n, k, tau_out, idx_out, val_out, capacity, result, workspace,
                           stream=None) -> None:
    """Threshold life-span L = 1: select on grad + residual, then compress the same vector with the tie
    budget k - n_gt, all on the stream."""
    _need(grad, torch.float32, "grad")
    _need(residual, torch.float32, "residual")
    _need(tau_out, torch.float32, "tau_out")
    _need(idx_out, torch.int32, "idx_out")
    _need(val_out, torch.float32, "val_out")
    _need(result, torch.int64, "result")
    _need(workspace, torch.uint8, "workspace")
    if grad.numel() < n or residual.numel() < n or idx_out.numel() < capacity or val_out.numel() < capacity:
        raise ValueError("buffer smaller than n / capacity")
    _check("dct_dp_select_compress",
           lib().dct_dp_select_compress(_p(grad), _p(residual), n, k, _p(tau_out), _p(idx_out), _p(val_out),
                                        capacity, _p(result), _p(workspace), workspace.numel(), _stream(stream)))


class _DpLayer(ctypes.Structure):          # dct_dp_layer_t
    _fields_ = [("grad", _vp), ("residual", _vp), ("n", _u64), ("tau", _vp), ("tie_budget", _vp),
                ("idx_out", _vp), ("val_out", _vp), ("capacity", _u64), ("result", _vp)]


def dct_dp_compress_batched_workspace_bytes(sizes) -> int:
    arr = (_u64 * len(sizes))(*sizes)
    return lib().dct_dp_compress_batched_workspace_bytes(arr, len(sizes))


def dct_dp_layer_table(layers):
    """Marshal a sequence of layer dicts (keys of dct_dp_layer_t: grad, residual, n, tau, tie_budget or None,
    idx_out, val_out, capacity, result) into the host array the C call takes.  Build it once per model."""
    table = (_DpLayer * len(layers))()
    for slot, a in zip(table, layers):
        _need(a["grad"], torch.float32, "grad")
        _need(a["residual"], torch.float32, "residual")
        _need(a["tau"], torch.float32, "tau")
        if a.get("tie_budget") is not None:
            _need(a["tie_budget"], torch.int64, "tie_budget")
        _need(a["idx_out"], torch.int32, "idx_out")
        _need(a["val_out"], torch.float32, "val_out")
        _need(a["result"], torch.int64, "result")
        n, cap = a["n"], a["capacity"]
        if a["grad"].numel() < n or a["residual"].numel() < n or a["idx_out"].numel() < cap or a["val_out"].numel() < cap:
            raise ValueError("buffer smaller than n / capacity")
        slot.grad, slot.residual, slot.n, slot.tau = _p(a["grad"]), _p(a["residual"]), n, _p(a["tau"])
        slot.tie_budget = _p(a.get("tie_budget"))
        slot.idx_out, slot.val_out, slot.capacity, slot.result = _p(a["idx_out"]), _p(a["val_out"]), cap, _p(a["result"])
    return table


def dct_dp_compress_batched(layers, workspace, stream=None) -> None:
    """``layers``: a table from dct_dp_layer_table, or the sequence of layer dicts it is built from."""
    table = layers if isinstance(layers, ctypes.Array) else dct_dp_layer_table(layers)
    _need(workspace, torch.uint8, "workspace")
    _check("dct_dp_compress_batched",
           lib().dct_dp_compress_batched(table, len(table), _p(workspace), workspace.numel(), _stream(stream)))


# ----------------------------------------------------------------------------
# threshold diagnostics
# ----------------------------------------------------------------------------

DCT_DIAG_MAX_QUANTILES = 4


def dct_threshold_select_multi_workspace_bytes(n: int, m: int) -> int:
    return lib().dct_threshold_select_multi_workspace_bytes(n, m)


def dct_threshold_select_multi(grad, residual, n, ks, tau_out, results, workspace, stream=None) -> None:
    """Thresholds of one vector for the survivor targets ``ks`` (a host sequence) out of the same three
    passes; tau_out [m] fp32 and results [m * 5] int64 (one dct_result_t per rank) are device tensors."""
    _need(grad, torch.float32, "grad")
    if residual is not None:
        _need(residual, torch.float32, "residual")
    _need(tau_out, torch.float32, "tau_out")
    _need(results, torch.int64, "results")
    _need(workspace, torch.uint8, "workspace")
    m = len(ks)
    if grad.numel() < n or (residual is not None and residual.numel() < n):
        raise ValueError("buffer smaller than n")
    if tau_out.numel() < m or results.numel() * 8 < m * RESULT_BYTES:
        raise ValueError("tau_out / results smaller than m")
    arr = (_u64 * max(m, 1))(*ks)
    _check("dct_threshold_select_multi",
           lib().dct_threshold_select_multi(_p(grad), _p(residual), n, arr, m, _p(tau_out), _p(results),
                                            _p(workspace), workspace.numel(), _stream(stream)))


def dct_mp_threshold_mean(x_act, rows, d, ld, ks, mean_out, tau_out, stream=None) -> None:
    """mean_out[q] = mean over the rows of the ks[q]-th largest |x[i, :d]|; tau_out [m * rows] receives the
    per-row thresholds.  Nothing is sparsified."""
    code = _dtype_code(x_act)
    _need(x_act, x_act.dtype, "x_act")
    _need(mean_out, torch.float64, "mean_out")
    _need(tau_out, x_act.dtype, "tau_out")
    m = len(ks)
    if x_act.numel() < (rows - 1) * ld + d:
        raise ValueError("x_act smaller than rows x ld")
    if mean_out.numel() < m or tau_out.numel() < m * rows:
        raise ValueError("mean_out / tau_out smaller than m / m * rows")
    arr = (_u32 * max(m, 1))(*ks)
    _check("dct_mp_threshold_mean",
           lib().dct_mp_threshold_mean(_p(x_act), code, rows, d, ld, arr, m, _p(mean_out), _p(tau_out),
                                       _stream(stream)))


def dct_dp_drift_check(compress_result, k, ratio_num, ratio_den, flag_out, stream=None) -> None:
    """flag_out[0] = 1 / 2 / 0: the survivor count of the last compress call is above k * ratio / below
    k / ratio / inside.  Device to device, on the stream."""
    _need(compress_result, torch.int64, "compress_result")
    _need(flag_out, torch.int32, "flag_out")
    _check("dct_dp_drift_check",
           lib().dct_dp_drift_check(_p(compress_result), k, ratio_num, ratio_den, _p(flag_out), _stream(stream)))


# ----------------------------------------------------------------------------
# thresholds of all layers at once
# ----------------------------------------------------------------------------

class _SelectLayer(ctypes.Structure):      # dct_select_layer_t
    _fields_ = [("grad", _vp), ("residual", _vp), ("n", _u64), ("k", _u64), ("tau_out", _vp), ("result", _vp)]


def dct_threshold_select_batched_workspace_bytes(num_layers: int) -> int:
    return lib().dct_threshold_select_batched_workspace_bytes(num_layers)


def dct_select_layer_table(layers):
    """Marshal a sequence of layer dicts (keys of dct_select_layer_t: grad, residual or None, n, k, tau_out,
    result) into the host array the C call takes."""
    table = (_SelectLayer * len(layers))()
    for slot, a in zip(table, layers):
        _need(a["grad"], torch.float32, "grad")
        if a.get("residual") is not None:
            _need(a["residual"], torch.float32, "residual")
        _need(a["tau_out"], torch.float32, "tau_out")
        _need(a["result"], torch.int64, "result")
        if a["grad"].numel() < a["n"] or (a.get("residual") is not None and a["residual"].numel() < a["n"]):
            raise ValueError("buffer smaller than n")
        slot.grad, slot.residual, slot.n, slot.k = _p(a["grad"]), _p(a.get("residual")), a["n"], a["k"]
        slot.tau_out, slot.result = _p(a["tau_out"]), _p(a["result"])
    return table


def dct_threshold_select_batched(layers, workspace, stream=None) -> None:
    """``layers``: a table from dct_select_layer_table, or the sequence of layer dicts it is built from."""
    table = layers if isinstance(layers, ctypes.Array) else dct_select_layer_table(layers)
    _need(workspace, torch.uint8, "workspace")
    _check("dct_threshold_select_batched",
           lib().dct_threshold_select_batched(table, len(table), _p(workspace), workspace.numel(), _stream(stream)))


# --------------------------------------------------------------------------------------------
# one vector range-partitioned over several ranks: the select with one small all-reduce per radix pass
# --------------------------------------------------------------------------------------------

SHARD_PASSES = 3
SHARD_BINS = 2048


def sharded_select_rounds(local_histogram, advance, all_reduce_sum, rounds=None):
    """The rounds of the range-partitioned select, free of any device code so that the exchange can be exercised on
    CPU ranks: per round ``local_histogram(p)`` returns this rank's 2048 counts, ``all_reduce_sum(h)`` returns
    (or turns ``h`` into) their sum over the ranks, and ``advance(p, h)`` lets the rank act on the sum.  Three rounds
    (the radix passes) by default; the sampled variant has six (SHARD_SAMPLED_ROUNDS)."""
    for p in range(SHARD_PASSES if rounds is None else rounds):
        h = local_histogram(p)
        summed = all_reduce_sum(h)
        advance(p, h if summed is None else summed)


SHARD_SAMPLED_ROUNDS = 6


def dct_threshold_select_shard_workspace_bytes() -> int:
    return lib().dct_threshold_select_shard_workspace_bytes()


def dct_threshold_select_shard_sampled_workspace_bytes(n_local: int) -> int:
    return lib().dct_threshold_select_shard_sampled_workspace_bytes(n_local)


def dct_threshold_select_sharded(grad, residual, n_local, k_global, tau_out, result, workspace, group=None,
                                 hist=None, stream=None, n_global=None) -> bool:
    """The k_global-th largest |grad + residual| of a vector whose shards lie on the ranks of ``group`` (the default
    process group if None; a single process without a group selects over its own shard alone).  Every rank calls
    this with its own shard; all get the same tau_out / result.  Three rounds with one all-reduce of 2048 int64
    counts each; if ``n_global`` (the total size over the ranks) is given, the vector is large enough and the
    workspace holds dct_threshold_select_shard_sampled_workspace_bytes(n_local), the sampled variant runs instead: six
    rounds, but one streaming pass over the shard instead of three.  Returns True if the sampled variant ran."""
    import torch.distributed as dist
    if n_local:
        _need(grad, torch.float32, "grad")
    if residual is not None:
        _need(residual, torch.float32, "residual")
    _need(tau_out, torch.float32, "tau_out")
    _need(result, torch.int64, "result")
    _need(workspace, torch.uint8, "workspace")
    if hist is None:
        hist = torch.empty(SHARD_BINS, dtype=torch.int64, device=tau_out.device)
    _need(hist, torch.int64, "hist")
    L, s = lib(), _stream(stream)
    multi = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1

    def all_reduce_sum(h):
        if multi:
            dist.all_reduce(h, op=dist.ReduceOp.SUM, group=group)
        return None

    g_ptr = _p(grad) if n_local else None
    sampled = False
    if n_global is not None and workspace.numel() >= L.dct_threshold_select_shard_sampled_workspace_bytes(n_local):
        st = L.dct_threshold_select_shard_sampled_begin(k_global, n_global, n_local, _p(workspace), workspace.numel(), s)
        if st == DCT_OK:
            sampled = True
        elif st != DCT_ERR_UNSUPPORTED:
            _check("dct_threshold_select_shard_sampled_begin", st)
    if sampled:
        def local_counts(p):
            _check("dct_threshold_select_shard_sampled_pass",
                   L.dct_threshold_select_shard_sampled_pass(g_ptr, _p(residual), n_local, p, _p(workspace), _p(hist), s))
            return hist

        def act(p, h):
            _check("dct_threshold_select_shard_sampled_advance",
                   L.dct_threshold_select_shard_sampled_advance(_p(h), p, _p(workspace), _p(tau_out), _p(result), s))

        sharded_select_rounds(local_counts, act, all_reduce_sum, rounds=SHARD_SAMPLED_ROUNDS)
        return True

    _check("dct_threshold_select_shard_begin",
           L.dct_threshold_select_shard_begin(k_global, _p(workspace), workspace.numel(), s))

    def local_histogram(p):
        _check("dct_threshold_select_shard_pass",
               L.dct_threshold_select_shard_pass(g_ptr, _p(residual), n_local, p, _p(workspace), _p(hist), s))
        return hist

    def advance(p, h):
        _check("dct_threshold_select_shard_advance",
               L.dct_threshold_select_shard_advance(_p(h), p, _p(workspace), _p(tau_out), _p(result), s))

    sharded_select_rounds(local_histogram, advance, all_reduce_sum)
    return False
