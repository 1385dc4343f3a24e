"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU).

The kernels are templates with many instantiations; they are spread over translation units (one per encoder
mode and dither width, one per decoder variant) that are compiled in parallel and linked into one shared library.
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "lib" / "libdq_b200.so"
OBJ = PKG / "lib" / "obj"
DEPS = sorted(CSRC.glob("*.cu*")) + sorted(CSRC.glob("*.h")) + [ROOT / "include" / "dq.h"]

NVCC_FLAGS = [
    "-std=c++17", "-O3",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo",
    "--fmad=false",          # every fused multiply-add in the kernels is written explicitly
    "-Xcompiler", "-fPIC",
]

# (object name, source, extra defines)
UNITS = [("dq_b200", "dq_b200.cu", [])]
UNITS += [(f"enc_m{m}_d{d}", "dq_encode_inst.cu", [f"-DDQ_INST_MODE={m}", f"-DDQ_INST_DITH={d}"])
          for m in (0, 1, 2, 3) for d in (32, 16)]
UNITS += [(f"dec_d{d}_r{r}", "dq_decode_inst.cu", [f"-DDQ_INST_DITH={d}", f"-DDQ_INST_RUN={r}"])
          for d, r in ((32, 0), (32, 1), (32, 2), (16, 0), (16, 1), (16, 2), (0, 0))]


def nvcc_path() -> str:
    cand = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return cand if Path(cand).exists() else "nvcc"


def source_hash() -> str:
    """Content hash of everything the library is built from (sources, headers, flags)."""
    h = hashlib.sha256()
    for f in DEPS:
        h.update(f.name.encode())
        h.update(f.read_bytes())
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()[:16]


def stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    return any(d.stat().st_mtime > t for d in DEPS)


def _compile(unit, verbose: bool, obj_dir: Path = OBJ, extra_flags=()) -> Path:
    name, src, defs = unit
    obj = obj_dir / f"{name}.o"
    cmd = [nvcc_path(), *NVCC_FLAGS, *defs, *extra_flags, f"-I{ROOT / 'include'}", f"-I{CSRC}", "-c", "-o", str(obj),
           str(CSRC / src)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    subprocess.run(cmd, check=True)
    return obj


def build(force: bool = False, verbose: bool = False, out: Path | None = None, extra_flags=()) -> Path:
    """Compiles every translation unit and links the shared library.  `out` / `extra_flags` build a variant
    (other tile or occupancy constants, see the DQ_* macros in csrc/) beside the default library."""
    if out is not None:
        return _build_to(Path(out), list(extra_flags), verbose)
    if not force and not stale():
        return LIB
    return _build_to(LIB, [], verbose)


def _build_to(lib: Path, extra_flags, verbose: bool) -> Path:
    global OBJ
    obj_dir = OBJ if lib == LIB else lib.parent / (lib.stem + "_obj")
    obj_dir.mkdir(parents=True, exist_ok=True)
    jobs = int(os.environ.get("DQ_BUILD_JOBS", "0")) or min(len(UNITS), os.cpu_count() or 1)
    with ThreadPoolExecutor(max_workers=jobs) as pool:
        objs = list(pool.map(lambda u: _compile(u, verbose, obj_dir, extra_flags), UNITS))
    tmp = lib.with_suffix(f".{os.getpid()}.tmp")
    subprocess.run([nvcc_path(), "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                    "-o", str(tmp), *[str(o) for o in objs]], check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
