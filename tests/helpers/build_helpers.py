"""Builds the test-support kernels (tests/helpers/*.cu) into libzctest.so next to this file."""
import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(HERE, "libzctest.so")
SRC = os.path.join(HERE, "zc_test_kernels.cu")
ROOT = os.path.dirname(os.path.dirname(HERE))
CSRC = os.path.join(ROOT, "paper_2405_14256_b200", "csrc")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= max(
            os.path.getmtime(SRC), os.path.getmtime(os.path.join(CSRC, "zc_quant.cuh"))):
        return LIB
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    res = subprocess.run([nvcc, "-shared", "-Xcompiler", "-fPIC", "-O2", "-std=c++17", "-lineinfo",
                          "-gencode", "arch=compute_100a,code=sm_100a", "-I", os.path.join(ROOT, "include"),
                          "-I", CSRC, "-o", LIB, SRC],
                         capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
