"""Builds libzipcache.so (sm_100a) in-tree with nvcc.  No JIT cache is involved: the
shared object sits next to this file so that it travels with the source tree."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libzipcache.so")
LIB_DEBUG = os.path.join(HERE, "libzipcache_debug.so")   # bounds-checked build (-DZC_DEBUG)
SOURCES = ["zc_host.cu", "zc_scores.cu", "zc_compress.cu", "zc_decode.cu", "zc_order.cu",
           "zc_export.cu", "zc_attention.cu"]
HEADERS = ["zc_internal.h", "zc_layout.cuh", "zc_mma.cuh", "zc_order.h", "zc_quant.cuh", "zc_tc.cuh"]


def _nvcc() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return cand


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(ROOT, "include", "zipcache.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """debug=True builds libzipcache_debug.so: the same sources with -DZC_DEBUG, whose kernels
    check the indices they address with and report a failed check through zc_device_status."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not _stale(lib):
        return lib
    cmd = [_nvcc(), "-shared", "-Xcompiler", "-fPIC", "-O3", "-std=c++17", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", lib] + (["-DZC_DEBUG"] if debug else []) + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
