"""Builds and runs the read-bandwidth test (``bench_tools/read_bandwidth.cu``, a stand-alone CUDA program).

    python -m bench_tools.read_bandwidth [ELEMENTS]
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
SOURCE = HERE / "read_bandwidth.cu"
EXE = HERE / "_build" / "read_bandwidth"


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
