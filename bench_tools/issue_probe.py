"""Builds and runs the issue-cost probe: scheduler cycles per warp instruction of the classes the kernels are
made of, alone and in the kernels' mixes.

    python -m bench_tools.issue_probe [GROUP [WARPS_PER_SCHEDULER]]

The probe (``bench_tools/issue_probe.cu``) is a stand-alone CUDA program; it needs a GPU.  With a group key
(first column of its output) it launches only that group, which is what a profiler capture of one kernel wants.
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
SOURCE = HERE / "issue_probe.cu"
EXE = HERE / "_build" / "issue_probe"


def build(force: bool = False) -> Path:
    if not force and EXE.exists() and EXE.stat().st_mtime >= SOURCE.stat().st_mtime:
        return EXE
    EXE.parent.mkdir(parents=True, exist_ok=True)
    nvcc = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    tmp = EXE.with_suffix(f".{os.getpid()}.tmp")
    subprocess.run([nvcc if Path(nvcc).exists() else "nvcc", "-std=c++17", "-O3", "-gencode",
                    "arch=compute_100a,code=sm_100a", "-lineinfo", "-cudart", "static", "-o", str(tmp), str(SOURCE)],
                   check=True)
    os.replace(tmp, EXE)
    return EXE


def main() -> int:
    return subprocess.run([str(build()), *sys.argv[1:]]).returncode


if __name__ == "__main__":
    sys.exit(main())
