"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "lib" / "libdq_b200.so"
SOURCES = [CSRC / "dq_b200.cu"]
PROBE_SOURCE = CSRC / "issue_probe.cu"          # stand-alone program, see issue_probe.py
PROBE = PKG / "lib" / "dq_issue_probe"
DEPS = sorted(f for f in CSRC.glob("*.cu*") if f != PROBE_SOURCE) + [ROOT / "include" / "dq.h"]

NVCC_FLAGS = [
    "-std=c++17", "-O3",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo",
    "--fmad=false",          # every fused multiply-add in the kernels is written explicitly
    "-Xcompiler", "-fPIC",
    "-cudart", "static",
    "-shared",
]


def nvcc_path() -> str:
    cand = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return cand if Path(cand).exists() else "nvcc"


def stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    return any(d.stat().st_mtime > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not stale():
        return LIB
    LIB.parent.mkdir(parents=True, exist_ok=True)
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
    cmd = [nvcc_path(), *NVCC_FLAGS, f"-I{ROOT / 'include'}", f"-I{CSRC}", "-o", str(tmp)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [str(s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


def build_probe(force: bool = False) -> Path:
    """Compiles the issue-cost probe (a stand-alone executable that uses no library code)."""
    if not force and PROBE.exists() and PROBE.stat().st_mtime >= PROBE_SOURCE.stat().st_mtime:
        return PROBE
    PROBE.parent.mkdir(parents=True, exist_ok=True)
    tmp = PROBE.with_suffix(f".{os.getpid()}.tmp")
    subprocess.run([nvcc_path(), "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
                    "-cudart", "static", "-o", str(tmp), str(PROBE_SOURCE)], check=True)
    os.replace(tmp, PROBE)
    return PROBE


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_probe(force="--force" in sys.argv))
