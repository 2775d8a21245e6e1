"""Builds libskim.so (the CUDA kernels and their C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libskim.so")
LIB_CHECKED = os.path.join(HERE, "libskim_checked.so")   # the same sources with -DSKIM_CHECK_BOUNDS
SOURCES = ["skim_api.cu", "skim_cluster.cu", "skim_cluster16.cu", "skim_lloyd.cu", "skim_allocate.cu", "skim_quantize.cu", "skim_unpack.cu", "skim_scale.cu", "skim_lfull.cu", "skim_exact.cu"]


def _stale(lib=LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "skim.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Builds libskim.so; checked=True builds libskim_checked.so instead, in which every computed index
    into shared memory, a row record or a scratch list is range-checked (a violation sets
    SKIM_STATUS_BOUNDS in the status word and skips the access).  Load it by setting SKIM_LIB."""
    lib = LIB_CHECKED if checked else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", lib] + [os.path.join(CSRC, s) for s in SOURCES]
    if checked:
        cmd.insert(1, "-DSKIM_CHECK_BOUNDS")
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
