"""Builds libdecode_attn.so (sm_100a) in-tree with nvcc.  No JIT cache, no torch extension."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libdecode_attn.so")
SOURCES = ["decode_attn.cu"]
HEADERS = ["da_ptx.cuh", "da_kernels.cuh", "da_prefix.cuh", os.path.join("..", "..", "include", "decode_attn.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the CUDA library for sm_100a if it is missing or older than its sources."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


DIAG_LIB = os.path.join(_HERE, "libdecode_attn_diag.so")
DIAG_FLAGS = ["-DDA_TIMELINE", "-DDA_DIAG", "-DDA_BOUNDS_CHECK"]


def build_diag(force: bool = False) -> str:
    """The diagnostic variant of the library, from the same sources: -DDA_TIMELINE (the kernels keep
    global-timer stamps of their phases), -DDA_DIAG (the limit of the kernels' bounded waits becomes
    an option, and one tile's copies can be withheld so that a wait runs out) and -DDA_BOUNDS_CHECK
    (every index into the kernels' own arrays is checked into the status record).  Used by
    ``timeline.py`` and the diagnostic tests; the normal library carries none of it."""
    if not force and os.path.exists(DIAG_LIB):
        t = os.path.getmtime(DIAG_LIB)
        if not any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS):
            return DIAG_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = DIAG_LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17"] + DIAG_FLAGS + [
           "-shared", "-Xcompiler", "-fPIC", "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, DIAG_LIB)
    return DIAG_LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
