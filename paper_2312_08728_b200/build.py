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

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]
BUILD_DIR = os.path.join(_PKG, "_build")  # object files (kept out of the history)


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
    # the tables of step kernels are translation units of their own: compile all of them side by side, then link
    flags = NVCC_FLAGS + (["-DBMGD_TRACE"] if trace else []) + (["-Xptxas", "-v"] if verbose else [])
    objdir = os.path.join(BUILD_DIR, "trace" if trace else "lib")
    os.makedirs(objdir, exist_ok=True)
    jobs = []
    for src in _sources():
        obj = os.path.join(objdir, os.path.splitext(os.path.basename(src))[0] + ".o")
        jobs.append((obj, subprocess.Popen([nvcc] + flags + ["-c", "-o", obj, src], cwd=CSRC)))
    failed = [obj for obj, proc in jobs if proc.wait() != 0]
    if failed:
        raise RuntimeError("nvcc failed for " + ", ".join(os.path.basename(o) for o in failed))
    tmp = out + f".{os.getpid()}.tmp"
    subprocess.check_call([nvcc, "-shared"] + NVCC_FLAGS[:2] + ["-o", tmp] + [obj for obj, _ in jobs] + ["-lcudart"], cwd=CSRC)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv, trace="--trace" in sys.argv))
