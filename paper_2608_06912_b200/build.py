"""Builds the CUDA library (sm_100a) in-tree with nvcc.  No torch involved."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
# LAPSUM_B200_CHECK_BUILD=1 selects the check build (every computed store index compared with its limit, see
# LAPSUM_IN_BOUNDS in csrc/common.cuh): a separate library, built with build(check_bounds=True)
CHECK = os.environ.get("LAPSUM_B200_CHECK_BUILD", "0") not in ("", "0")
LIB = os.path.join(HERE, "liblapsum_b200_check.so" if CHECK else "liblapsum_b200.so")
SOURCES = ["lapsum_api.cu"]
HEADERS = ["common.cuh", "solve.cuh", "radix_sort.cuh", "row_block.cuh", "global_path.cuh", "bracket_select.cuh",
           os.path.join("..", "..", "include", "lapsum.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    files = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.getmtime(f) > t for f in files if os.path.exists(f))


def build(force: bool = False, verbose: bool = False, check_bounds: bool | None = None) -> str:
    """Compile the library; check_bounds=True builds the check variant (liblapsum_b200_check.so) instead, None follows
    the LAPSUM_B200_CHECK_BUILD environment variable."""
    check = CHECK if check_bounds is None else bool(check_bounds)
    lib = os.path.join(HERE, "liblapsum_b200_check.so" if check else "liblapsum_b200.so")
    if not force and lib == LIB and not stale():
        return LIB
    tmp = lib + f".{os.getpid()}.tmp"
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-rdc=true", "-o", tmp]
    if check:
        cmd += ["-DLAPSUM_CHECK_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    cmd += ["-lcudadevrt"]  # device-side launch of the full-sort fallback
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, check_bounds=True if "--check-bounds" in sys.argv else None))
