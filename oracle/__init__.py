"""CPU oracle for the DCT compression path (test infrastructure, not product code).

Thin ctypes front end of ``dct_oracle.cpp``: it marshals numpy arrays and adds
no arithmetic of its own.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA path never does.

fp32 data are ``numpy.float32`` arrays; bf16 data are ``numpy.uint16`` arrays
holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import NamedTuple, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dct_oracle.cpp")
_LIB = os.path.join(_HERE, "libdct_oracle.so")

_c_u64 = ctypes.c_uint64
_c_u32 = ctypes.c_uint32
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math: denormals and RNE are kept)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-fno-fast-math",
             "-ffp-contract=off", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for name in ("oracle_dp_select", "oracle_dp_compress", "oracle_mp_fwd_f32",
                     "oracle_mp_fwd_bf16", "oracle_mp_bwd_f32", "oracle_mp_bwd_bf16",
                     "oracle_dp_decompress", "oracle_mp_unpack_f32", "oracle_mp_unpack_bf16",
                     "oracle_dp_select_multi", "oracle_mp_threshold_mean_f32", "oracle_mp_threshold_mean_bf16",
                     "oracle_dp_drift_flag"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(a: np.ndarray, dtype, name: str) -> np.ndarray:
    if a.dtype != dtype or not a.flags["C_CONTIGUOUS"]:
        raise TypeError(f"{name}: need C-contiguous {np.dtype(dtype).name}, got {a.dtype}")
    return a


class SelectResult(NamedTuple):
    tau: np.float32
    n_gt: int
    n_eq: int


class CompressResult(NamedTuple):
    idx: np.ndarray      # int32[count], ascending
    val: np.ndarray      # float32[count]
    count: int           # survivors written (<= capacity)
    needed: int          # survivors found


def dp_select(grad: np.ndarray, residual: Optional[np.ndarray], k: int,
              full_sort: bool = False) -> SelectResult:
    """Algorithm 1, threshold steps: k-th largest |grad + residual| and tie counts."""
    lib = _load()
    _check(grad, np.float32, "grad")
    if residual is not None:
        _check(residual, np.float32, "residual")
        assert residual.size == grad.size
    tau = ctypes.c_float()
    n_gt, n_eq = _c_u64(), _c_u64()
    rc = lib.oracle_dp_select(_ptr(grad), _ptr(residual), _c_u64(grad.size), _c_u64(k),
                              ctypes.c_int(1 if full_sort else 0),
                              ctypes.byref(tau), ctypes.byref(n_gt), ctypes.byref(n_eq))
    if rc:
        raise ValueError(f"oracle_dp_select: invalid argument (rc={rc})")
    return SelectResult(np.float32(tau.value), n_gt.value, n_eq.value)


def dp_compress(grad: np.ndarray, residual: np.ndarray, tau, tie_budget: Optional[int],
                capacity: int) -> CompressResult:
    """Algorithm 1, mask / compressed gradient / error steps.  ``residual`` is updated in place."""
    lib = _load()
    _check(grad, np.float32, "grad")
    _check(residual, np.float32, "residual")
    assert residual.size == grad.size
    idx = np.empty(capacity, dtype=np.int32)
    val = np.empty(capacity, dtype=np.float32)
    count, needed = _c_u64(), _c_u64()
    rc = lib.oracle_dp_compress(_ptr(grad), _ptr(residual), _c_u64(grad.size),
                                ctypes.c_float(float(np.float32(tau))),
                                ctypes.c_int(0 if tie_budget is None else 1),
                                _c_u64(0 if tie_budget is None else tie_budget),
                                _ptr(idx), _ptr(val), _c_u64(capacity),
                                ctypes.byref(count), ctypes.byref(needed))
    if rc:
        raise ValueError(f"oracle_dp_compress: invalid argument (rc={rc})")
    c = count.value
    return CompressResult(idx[:c].copy(), val[:c].copy(), c, needed.value)


class MpFwdResult(NamedTuple):
    cols: np.ndarray     # int16[rows, k], ascending within a row: the mask M
    vals: np.ndarray     # [rows, k], dtype of x
    tau: np.ndarray      # [rows], dtype of x: the row thresholds tau_i


def mp_fwd(x: np.ndarray, k: int, d: Optional[int] = None) -> MpFwdResult:
    """Algorithm 2, forward pass.  ``x`` is [rows, ld]; the first ``d`` columns of each row count."""
    lib = _load()
    assert x.ndim == 2
    rows, ld = x.shape
    d = ld if d is None else d
    if x.dtype == np.float32:
        fn = lib.oracle_mp_fwd_f32
    elif x.dtype == np.uint16:
        fn = lib.oracle_mp_fwd_bf16
    else:
        raise TypeError("x: float32 or uint16 (bf16 bits)")
    _check(x, x.dtype, "x")
    cols = np.empty((rows, k), dtype=np.int16)
    vals = np.empty((rows, k), dtype=x.dtype)
    tau = np.empty(rows, dtype=x.dtype)
    rc = fn(_ptr(x), _c_u32(rows), _c_u32(d), _c_u32(ld), _c_u32(k),
            _ptr(cols), _ptr(vals), _ptr(tau))
    if rc:
        raise ValueError(f"oracle_mp_fwd: invalid argument (rc={rc})")
    return MpFwdResult(cols, vals, tau)


def mp_bwd(gx: np.ndarray, cols: np.ndarray, d: Optional[int] = None) -> np.ndarray:
    """Algorithm 2, backward pass: gather ``gx`` through the forward mask ``cols``."""
    lib = _load()
    assert gx.ndim == 2 and cols.ndim == 2 and gx.shape[0] == cols.shape[0]
    rows, ld = gx.shape
    d = ld if d is None else d
    k = cols.shape[1]
    if gx.dtype == np.float32:
        fn = lib.oracle_mp_bwd_f32
    elif gx.dtype == np.uint16:
        fn = lib.oracle_mp_bwd_bf16
    else:
        raise TypeError("gx: float32 or uint16 (bf16 bits)")
    _check(gx, gx.dtype, "gx")
    _check(cols, np.int16, "cols")
    gvals = np.empty((rows, k), dtype=gx.dtype)
    rc = fn(_ptr(gx), _c_u32(rows), _c_u32(d), _c_u32(ld), _c_u32(k), _ptr(cols), _ptr(gvals))
    if rc:
        raise ValueError(f"oracle_mp_bwd: invalid argument (rc={rc})")
    return gvals


def dp_decompress(idx: np.ndarray, val: np.ndarray, dense: np.ndarray, accumulate: bool) -> None:
    """Receiving end of Algorithm 1's send: scatter (idx, val) into ``dense`` (in place); with
    ``accumulate`` the values are added to what is there, otherwise ``dense`` is cleared first."""
    lib = _load()
    _check(idx, np.int32, "idx")
    _check(val, np.float32, "val")
    _check(dense, np.float32, "dense")
    assert idx.size == val.size
    rc = lib.oracle_dp_decompress(_ptr(idx), _ptr(val), _c_u64(idx.size), _ptr(dense), _c_u64(dense.size),
                                  ctypes.c_int(1 if accumulate else 0))
    if rc:
        raise ValueError(f"oracle_dp_decompress: invalid argument (rc={rc})")


def mp_unpack(cols: np.ndarray, vals: np.ndarray, d: int, ld: Optional[int] = None) -> np.ndarray:
    """Receiving end of Algorithm 2's sends: the dense [rows, ld] matrix that holds ``vals`` at the mask
    columns and zero at the other columns below d (columns d..ld-1 are returned as zero)."""
    lib = _load()
    assert cols.ndim == 2 and vals.shape == cols.shape
    rows, k = cols.shape
    ld = d if ld is None else ld
    if vals.dtype == np.float32:
        fn = lib.oracle_mp_unpack_f32
    elif vals.dtype == np.uint16:
        fn = lib.oracle_mp_unpack_bf16
    else:
        raise TypeError("vals: float32 or uint16 (bf16 bits)")
    _check(cols, np.int16, "cols")
    _check(vals, vals.dtype, "vals")
    dense = np.zeros((rows, ld), dtype=vals.dtype)
    rc = fn(_ptr(cols), _ptr(vals), _c_u32(rows), _c_u32(d), _c_u32(ld), _c_u32(k), _ptr(dense))
    if rc:
        raise ValueError(f"oracle_mp_unpack: invalid argument (rc={rc})")
    return dense


class SelectMultiResult(NamedTuple):
    tau: np.ndarray        # float32 [m]
    n_gt: np.ndarray       # uint64 [m]
    n_eq: np.ndarray       # uint64 [m]


def dp_select_multi(grad: np.ndarray, residual: Optional[np.ndarray], ks) -> SelectMultiResult:
    """Top-k thresholds of one vector at several survivor targets (Sec. 2.1, threshold plot)."""
    lib = _load()
    _check(grad, np.float32, "grad")
    if residual is not None:
        _check(residual, np.float32, "residual")
    m = len(ks)
    ks_a = np.asarray(ks, dtype=np.uint64)
    tau = np.zeros(m, dtype=np.float32)
    n_gt = np.zeros(m, dtype=np.uint64)
    n_eq = np.zeros(m, dtype=np.uint64)
    rc = lib.oracle_dp_select_multi(_ptr(grad), _ptr(residual), _c_u64(grad.size), _ptr(ks_a), _c_u32(m),
                                    _ptr(tau), _ptr(n_gt), _ptr(n_eq))
    if rc != 0:
        raise ValueError(f"oracle_dp_select_multi: bad arguments ({rc})")
    return SelectMultiResult(tau, n_gt, n_eq)


class ThresholdMeanResult(NamedTuple):
    mean: np.ndarray       # float64 [m]
    tau: np.ndarray        # [m, rows], dtype of x


def mp_threshold_mean(x: np.ndarray, ks, d: Optional[int] = None) -> ThresholdMeanResult:
    """(1/B) sum_i tau_i at several sparsity levels, nothing sparsified (Sec. 2.2, threshold plot)."""
    lib = _load()
    rows, ld = x.shape
    d = ld if d is None else d
    m = len(ks)
    ks_a = np.asarray(ks, dtype=np.uint32)
    mean = np.zeros(m, dtype=np.float64)
    tau = np.zeros((m, rows), dtype=x.dtype)
    if x.dtype == np.float32:
        fn = lib.oracle_mp_threshold_mean_f32
    elif x.dtype == np.uint16:
        fn = lib.oracle_mp_threshold_mean_bf16
    else:
        raise TypeError("x: float32, or uint16 holding bf16 bit patterns")
    _check(x, x.dtype, "x")
    rc = fn(_ptr(x), _c_u32(rows), _c_u32(d), _c_u32(ld), _ptr(ks_a), _c_u32(m), _ptr(mean), _ptr(tau))
    if rc != 0:
        raise ValueError(f"oracle_mp_threshold_mean: bad arguments ({rc})")
    return ThresholdMeanResult(mean, tau)


def dp_drift_flag(needed: int, k: int, ratio_num: int, ratio_den: int) -> int:
    """1: survivors above k * ratio; 2: below k / ratio; 0: inside (ratio = ratio_num / ratio_den >= 1)."""
    lib = _load()
    return lib.oracle_dp_drift_flag(_c_u64(needed), _c_u64(k), _c_u32(ratio_num), _c_u32(ratio_den))
