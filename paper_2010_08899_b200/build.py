"""Build the C-ABI shared library with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import concurrent.futures
import os
import shutil
import subprocess
import sys
import tempfile

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libdct_b200.so")
SOURCES = ["mp_pack.cu", "mp_pack_span.cu", "mp_pack_f32_wide.cu", "mp_pack_f32.cu", "mp_pack_narrow.cu", "dp_compress.cu", "threshold_select.cu", "threshold_select_batched.cu", "threshold_select_sharded.cu", "decompress.cu", "diagnostics.cu",
           "dp_select_compress.cu", "abi.cu"]          # the slowest to compile first
HEADERS = [os.path.join(CSRC, h) for h in ("common.cuh", "row_select.cuh", "mp_warp.cuh", "dp_chain.cuh")] + \
          [os.path.join(ROOT, "include", "dct.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--ftz=false", "--prec-div=true", "--prec-sqrt=true", "--fmad=false",
    "-Xcompiler", "-fPIC,-fvisibility=hidden", "-cudart", "static",
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every kernel into one shared library next to this file and return its path.
    The translation units are compiled side by side (one nvcc each), then linked."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = tempfile.mkdtemp(prefix="dct_build_")
    try:
        common = [nvcc, *NVCC_FLAGS, "-I", os.path.join(ROOT, "include"), "-I", CSRC]
        if verbose:
            common += ["-Xptxas", "-v"]

        def compile_one(src: str) -> str:
            obj = os.path.join(objdir, os.path.splitext(src)[0] + ".o")
            subprocess.check_call(common + ["-c", os.path.join(CSRC, src), "-o", obj])
            return obj

        with concurrent.futures.ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
            objects = list(pool.map(compile_one, SOURCES))
        tmp = LIB + f".{os.getpid()}.tmp"
        subprocess.check_call([nvcc, "-shared", *NVCC_FLAGS, *objects, "-o", tmp])
        os.replace(tmp, LIB)
    finally:
        shutil.rmtree(objdir, ignore_errors=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
