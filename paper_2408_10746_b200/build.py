"""Builds the CUDA library in-tree:  python -m paper_2408_10746_b200.build

nvcc cross-compiles for sm_100a without a GPU.  The result,
paper_2408_10746_b200/libpac_b200.so, exports the C ABI declared in include/pac.h.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libpac_b200.so")
SOURCES = [os.path.join(HERE, "csrc", "pac_api.cu")]
HEADERS = [os.path.join(HERE, "csrc", f) for f in ("pac_common.cuh", "pac_simt.cuh", "pac_tensor.cuh", "pac_mid.cuh", "pac_fused_fwd.cuh", "pac_gemm.cuh", "pac_quant.cuh")] + \
          [os.path.join(ROOT, "include", "pac.h")]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS if os.path.exists(p))


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(HERE, "csrc"), "-o", LIB] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
