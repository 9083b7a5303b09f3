"""Compile the CUDA library in-tree for sm_100a with nvcc."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libbmgd.so")
TRACE_LIB_PATH = os.path.join(_PKG, "libbmgd_trace.so")  # the same sources with -DBMGD_TRACE (phase clock stamps)

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC",
]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    root = os.path.dirname(_PKG)
    return _sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(root, "include", "*.h"))


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(f) > t for f in _deps())


def find_nvcc():
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    return None


def build(force: bool = False, verbose: bool = False, trace: bool = False) -> str:
    """Build libbmgd.so next to this file if it is missing or older than its sources.

    trace=True builds libbmgd_trace.so instead: the same sources compiled with -DBMGD_TRACE, in which thread 0 of
    every CTA stamps the clock at the phase boundaries of its first steps (read by paper_2312_08728_b200.trace)."""
    out = TRACE_LIB_PATH if trace else LIB_PATH
    if not force and not is_stale(out):
        return out
    nvcc = find_nvcc()
    if nvcc is None:
        raise RuntimeError("nvcc not found: cannot build the BMGD CUDA library")
    tmp = out + f".{os.getpid()}.tmp"
    cmd = ([nvcc] + NVCC_FLAGS + (["-DBMGD_TRACE"] if trace else []) + (["-Xptxas", "-v"] if verbose else [])
           + ["-o", tmp] + _sources() + ["-lcudart"])
    subprocess.check_call(cmd, cwd=CSRC)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv, trace="--trace" in sys.argv))
