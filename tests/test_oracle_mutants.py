"""Do the pins notice a mistake?  Each case plants one plausible error in a copy of the oracle's C source
(a dropped term, a wrong sign, index or constant), builds it, and runs the pin files against it in a
subprocess: at least one pin must fail.  The mistakes live in the oracle only, on the CPU."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
SRC = (ROOT / "oracle" / "dq_oracle.c").read_text()
PIN_FILES = ["tests/test_oracle_pins.py", "tests/test_oracle_dither16.py", "tests/test_oracle_running_mean.py",
             "tests/test_oracle_ternary.py"]

MUTANTS = [
    ("philox multipliers swapped", "(uint64_t)0xD2511F53u * (uint64_t)c0", "(uint64_t)0xCD9E8D57u * (uint64_t)c0"),
    ("philox nine rounds", "round < 10", "round < 9"),
    ("counter words permuted", "ctr[1] = worker;\n    ctr[2] = (uint32_t)(step & 0xFFFFFFFFu);\n    ctr[3] = (uint32_t)(step >> 32);\n    key[0] = (uint32_t)(seed & 0xFFFFFFFFu);\n    key[1] = (uint32_t)(seed >> 32);\n    dqo_philox4x32_10(ctr, key, out);\n    return out[i & 3u];",
     "ctr[2] = worker;\n    ctr[1] = (uint32_t)(step & 0xFFFFFFFFu);\n    ctr[3] = (uint32_t)(step >> 32);\n    key[0] = (uint32_t)(seed & 0xFFFFFFFFu);\n    key[1] = (uint32_t)(seed >> 32);\n    dqo_philox4x32_10(ctr, key, out);\n    return out[i & 3u];"),
    ("dither uses the wrong bits", "((x >> 10) << 1) | 1u", "((x >> 9) << 1) | 1u"),
    ("dither not centred", "(float)odd * 0x1p-23f - 0.5f", "(float)odd * 0x1p-23f - 0.25f"),
    ("encoder forgets the dither", "float v = fmaf(g[i], a, delta);\n            float w = v + s;", "float v = fmaf(g[i], a, 0.0f * delta);\n            float w = v + s;"),
    ("decoder adds the dither", "float d = ((float)k - s) - delta;", "float d = ((float)k - s) + delta;"),
    ("scale is not the maximum", "if (a > kappa) kappa = a;", "if (a > kappa && i < len / 2) kappa = a;"),
    ("straddling code misplaced", "words[w + 1] |= code[i] >> (32u - sh);", "words[w + 1] |= code[i] >> (31u - sh);"),
    ("coset of a negative index", "int32_t m = ((q1 % K) + K) % K;", "int32_t m = (q1 % K + K - 1) % K;"),
    ("nested decoder sign of the dither", "float r1 = (float)m - delta;", "float r1 = (float)m + delta;"),
    ("coarse cell resolved the wrong way", "int32_t qhat = (int32_t)m - K * jj;", "int32_t qhat = (int32_t)m + K * jj;"),
    ("side information not normalised by the sender's scale", "float r = fmaf(-y, a, r1);", "float r = fmaf(-y, 1.0f, r1);"),
    ("shrinkage term", "(1.0f - alpha * alpha) * y", "(1.0f - alpha) * y"),
    ("mean divides by the wrong count", "out_avg[i] = acc / (float)W;", "out_avg[i] = acc / (float)(W + 1u);"),
    ("half-words swapped in the 16-bit stream", "return (i & 1u) ? (word >> 16) : (word & 0xFFFFu);", "return (i & 1u) ? (word & 0xFFFFu) : (word >> 16);"),
    ("16-bit grid off centre", "(float)(2u * h + 1u) * 0x1p-17f - 0.5f", "(float)(2u * h) * 0x1p-17f - 0.5f"),
    ("running mean counts one worker too many", "acc * (1.0f / (float)w)", "acc * (1.0f / (float)(w + 1u))"),
    ("ternary digit weights", "weight *= 3u;", "weight *= 4u;"),
    ("ternary digits read in the wrong order", "q < (uint32_t)(i % 5u); ++q)", "q < 4u - (uint32_t)(i % 5u); ++q)"),
    ("ternary container drops the last partial byte", "return (n + 4u) / 5u;", "return n / 5u;"),
    ("scalar quantizer truncates", "return Delta * nearbyint(v / Delta);", "return Delta * floor(v / Delta);"),
    ("nested scalar decoder drops the coarse term", "return y + alpha * (r - dqo_Q(r, Delta2));", "return y + alpha * r;"),
]


def _run_pins(src_path, lib_path):
    env = dict(os.environ, DQ_ORACLE_SOURCE=str(src_path), DQ_ORACLE_LIBRARY=str(lib_path))
    return subprocess.run([sys.executable, "-m", "pytest", *PIN_FILES, "-x", "-q", "-p", "no:cacheprovider"],
                          cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)


def test_every_mutation_site_exists_once():
    for name, old, new in MUTANTS:
        assert SRC.count(old) == 1, f"{name}: pattern occurs {SRC.count(old)} times"
        assert old != new


@pytest.mark.parametrize("idx", range(len(MUTANTS)), ids=[m[0].replace(" ", "_") for m in MUTANTS])
def test_pins_catch_planted_mistake(tmp_path, idx):
    name, old, new = MUTANTS[idx]
    src = tmp_path / "dq_oracle_mutant.c"
    src.write_text(SRC.replace(old, new))
    out = _run_pins(src, tmp_path / "libmutant.so")
    assert out.returncode != 0, f"no pin noticed: {name}"
    assert "failed" in out.stdout or "error" in out.stdout.lower(), out.stdout[-500:]


def test_unmodified_copy_passes(tmp_path):
    src = tmp_path / "dq_oracle_copy.c"
    src.write_text(SRC)
    out = _run_pins(src, tmp_path / "libcopy.so")
    assert out.returncode == 0, out.stdout[-2000:]
