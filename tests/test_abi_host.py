"""Host-side checks that need no GPU: the library builds and loads, exports every symbol the
header declares, and refuses bad arguments before touching the device."""
import ctypes
import os
import re

import pytest
import torch

from paper_2010_08899_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "dct.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"DCT_API\s+[\w\s\*]+?\b(dct_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    declared = _declared_symbols()
    assert len(declared) >= 10
    assert sorted(B.EXPORTED_SYMBOLS) == declared
    L = B.lib()
    for name in declared:
        assert getattr(L, name) is not None


def test_status_strings():
    L = B.lib()
    names = [L.dct_status_string(i).decode() for i in range(8)]
    assert names[0] == "DCT_OK" and names[5] == "DCT_ERR_CAPACITY" and len(set(names)) == 8
    assert L.dct_status_string(99).decode() == "DCT_ERR_UNKNOWN"


def test_workspace_sizes():
    assert B.dct_dp_compress_workspace_bytes(0) == 0
    assert B.dct_dp_compress_workspace_bytes(1 << 31) == 0          # beyond int32 indices
    small, big = B.dct_dp_compress_workspace_bytes(1), B.dct_dp_compress_workspace_bytes((1 << 31) - 1)
    assert 0 < small <= 1024 and small % 256 == 0
    assert big % 256 == 0 and big < 64 << 20                         # a few MiB even for the largest vector
    assert B.dct_threshold_select_workspace_bytes(1 << 30) > 0


def test_invalid_arguments_are_refused_on_the_host():
    """Null pointers, bad sizes and bad alignment come back as error codes with no launch
    (this runs on machines with no GPU at all)."""
    L = B.lib()
    buf = (ctypes.c_char * 4096)()
    p = (ctypes.addressof(buf) + 255) & ~255                          # a 256-aligned fake pointer
    ws = B.dct_dp_compress_workspace_bytes(1000)
    n, k = 1000, 10
    sel = L.dct_threshold_select
    assert sel(None, None, n, k, p, p, p, 1 << 20, None) == B.DCT_ERR_INVALID_ARG
    assert sel(p, None, 0, k, p, p, p, 1 << 20, None) == B.DCT_ERR_INVALID_ARG
    assert sel(p, None, n, 0, p, p, p, 1 << 20, None) == B.DCT_ERR_INVALID_ARG
    assert sel(p, None, n, n + 1, p, p, p, 1 << 20, None) == B.DCT_ERR_INVALID_ARG
    assert sel(p, None, 1 << 31, k, p, p, p, 1 << 20, None) == B.DCT_ERR_INVALID_ARG
    assert sel(p, None, n, k, p, p, p, 16, None) == B.DCT_ERR_WORKSPACE
    assert sel(p, None, n, k, p, p, p + 8, 1 << 20, None) == B.DCT_ERR_WORKSPACE
    assert sel(p + 2, None, n, k, p, p, p, 1 << 20, None) == B.DCT_ERR_INVALID_ARG
    cmp_ = L.dct_dp_compress
    assert cmp_(None, p, n, p, None, p, p, 10, p, p, ws, None) == B.DCT_ERR_INVALID_ARG
    assert cmp_(p, p, n, p, None, p, p, 10, p, p, ws, None) == B.DCT_ERR_INVALID_ARG          # grad aliases residual
    assert cmp_(p, p + 2000, n, p, None, p, p, 10, p, p, ws, None) == B.DCT_ERR_INVALID_ARG   # partial overlap
    assert cmp_(p, p + 4096, n, p, None, None, None, 10, p, p, ws, None) == B.DCT_ERR_INVALID_ARG
    assert cmp_(p, p + 4096, n, p, None, p, p, 10, p, p, ws - 1, None) == B.DCT_ERR_WORKSPACE
    assert cmp_(p, p + 4096, n, p, None, p, p, 10, p, None, ws, None) == B.DCT_ERR_WORKSPACE
    fwd = L.dct_mp_topk_pack_fwd
    assert fwd(None, 0, 4, 8, 8, 2, p, p, None, None, None, None) == B.DCT_ERR_INVALID_ARG
    assert fwd(p, 0, 4, 8, 8, 0, p, p, None, None, None, None) == B.DCT_ERR_INVALID_ARG
    assert fwd(p, 0, 4, 8, 8, 9, p, p, None, None, None, None) == B.DCT_ERR_INVALID_ARG
    assert fwd(p, 0, 4, 8, 7, 2, p, p, None, None, None, None) == B.DCT_ERR_INVALID_ARG       # ld < d
    assert fwd(p, 0, 4, 32769, 32769, 2, p, p, None, None, None, None) == B.DCT_ERR_INVALID_ARG
    assert fwd(p, 5, 4, 8, 8, 2, p, p, None, None, None, None) == B.DCT_ERR_UNSUPPORTED       # unknown dtype
    assert fwd(p, 0, 0, 8, 8, 2, p, p, None, None, None, None) == B.DCT_ERR_INVALID_ARG
    bwd = L.dct_mp_pack_bwd
    assert bwd(p, 1, 4, 8, 8, 2, None, p, None, None) == B.DCT_ERR_INVALID_ARG
    assert bwd(p + 1, 1, 4, 8, 8, 2, p, p, None, None) == B.DCT_ERR_INVALID_ARG               # bf16 needs 2-byte alignment


def test_binding_rejects_wrong_tensors():
    g = torch.zeros(8)
    with pytest.raises(ValueError):
        B.dct_dp_compress(g, g, 8, g, None, g.int(), g, 8, torch.zeros(5, dtype=torch.int64),
                          torch.zeros(512, dtype=torch.uint8))               # host tensors where device ones are due
    with pytest.raises(TypeError):
        B._dtype_code(torch.zeros(2, dtype=torch.float16))


def test_k_from_sparsity_matches_the_configs():
    # k = n - floor(n * eta) with eta the fraction dropped, in exact integer arithmetic
    assert B.k_from_sparsity(4096, 95, 100) == 205
    assert B.k_from_sparsity(1024, 15, 16) == 64
    assert B.k_from_sparsity(1 << 20, 1023, 1024) == 1024
    assert B.k_from_density(64 << 20, 1, 1000) == 67_109
    assert B.k_from_density(1 << 30, 1, 10_000) == 107_375
    assert B.k_from_sparsity(10, 1, 1) == 0 and B.k_from_sparsity(10, 0, 1) == 10
    with pytest.raises(ValueError):
        B.k_from_sparsity(10, 3, 2)
