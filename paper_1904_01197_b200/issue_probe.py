"""Runs the issue-cost probe: scheduler cycles per warp instruction of the classes the kernels are made of.

    python -m paper_1904_01197_b200.issue_probe

The probe (``csrc/issue_probe.cu``) is a stand-alone CUDA program; it needs a GPU.  Its table is what the
decode kernel's issue ceiling in ``bench.py`` rests on: integer, logic and shift instructions cost two scheduler
cycles, fp32 adds and multiply-adds about one, a 32x32->64 multiply 4.4 (with one logic instruction hidden
behind it), and the classes do not overlap.
"""
from __future__ import annotations

import subprocess
import sys

from . import build


def main() -> int:
    exe = build.build_probe()
    return subprocess.run([str(exe)]).returncode


if __name__ == "__main__":
    sys.exit(main())
