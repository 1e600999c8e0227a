"""Build ``librkv.so`` in-tree with nvcc for sm_100a.

    python -m paper_2509_14279_b200.build [--force] [--verbose] [--debug-bounds]

The library is plain CUDA C++ behind a C ABI (``include/rkv.h``); it does not
link against torch.  ``-fmad=false`` forbids fused multiply-add contraction:
the generator and the comparison rule are defined operation by operation.

``--debug-bounds`` builds ``librkv_dbg.so`` instead: the same sources with
``-DRKV_DEBUG_BOUNDS``, where the verification kernel range-checks every index into
global memory and into its shared-memory tables, records the first violation in the
workspace header and skips the access (status RKV_ERR_BOUNDS; nothing traps).  Select it
with ``RKV_LIB=.../librkv_dbg.so``.
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "librkv.so")
LIB_DBG = os.path.join(PKG, "librkv_dbg.so")
SOURCES = ["rkv_api.cu", "rkv_gen.cu", "rkv_verify.cu", "rkv_screen.cu", "rkv_cross.cu"]
HEADERS = ["rkv_internal.h", "rkv_philox.cuh"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo", "-fmad=false",
    "-Xcompiler", "-fPIC", "-shared",
]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(ROOT, "include", "rkv.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    lib = LIB_DBG if debug_bounds else LIB
    if not (force or _stale(lib)):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if not os.path.exists(nvcc):
        nvcc = "nvcc"
    tmp = lib + f".{os.getpid()}.tmp"
    cmd = [nvcc, *NVCC_FLAGS, f"-I{os.path.join(ROOT, 'include')}", f"-I{CSRC}"]
    if debug_bounds:
        cmd += ["-DRKV_DEBUG_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", tmp, *[os.path.join(CSRC, s) for s in SOURCES]]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv,
                debug_bounds="--debug-bounds" in sys.argv))
