"""Builds and runs the tcgen05.mma issue-cost probe (csrc/mma_issue_probe.cu): a diagnostic that times
back-to-back tensor-core instructions of several shapes on one SM.

    python -m paper_2512_10977_b200.mma_probe
"""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))


def build() -> str:
    exe = os.path.join(_HERE, "mma_issue_probe")
    src = os.path.join(_HERE, "csrc", "mma_issue_probe.cu")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-o", exe, src], check=True)
    return exe


if __name__ == "__main__":
    sys.exit(subprocess.run([build()]).returncode)
