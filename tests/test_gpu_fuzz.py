"""GPU parity on seeded random configurations: combinations the hand-picked cases do not enumerate (odd bucket sizes
with mixed kinds and widths per worker, non-power-of-two coarse ratios with shrinkage, both dither streams, ragged
lengths, wide value ranges).  Every case is reproducible from its index."""
import numpy as np
import pytest

from dq_workloads.generators import DQSG, NDQSG, WorkerSpec

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import assert_fp32_close  # noqa: E402
from test_gpu_parity import _check_encode, _roundtrip_decode, dq, oracle  # noqa: E402,F401

BUCKETS = [32, 64, 96, 160, 256, 480, 512, 1024, 1504, 2048, 4096, 8192, 12288]


def _random_spec(rng, dither_bits):
    bits = int(rng.integers(1, 9))
    seed = int(rng.integers(0, 2 ** 63))
    if rng.random() < 0.45:
        lo = 2
        levels = int(rng.integers(lo, (1 << bits) + 1))
        return WorkerSpec(DQSG, bits, levels, seed=seed, dither_bits=dither_bits)
    K = int(rng.integers(2, (1 << bits) + 1))
    M1 = float(rng.choice([1.0, 1.5, 2.0, 3.0, 4.0, 7.5, 16.0, 100.0]))
    alpha = float(rng.choice([1.0, 1.0, 0.9, 0.75, 0.5]))
    return WorkerSpec(NDQSG, bits, 0, K, M1, alpha, seed, dither_bits=dither_bits)


@pytest.mark.parametrize("case", range(24))
def test_random_configuration(dq, oracle, case):
    rng = np.random.default_rng(77_000 + case)
    bucket = int(rng.choice(BUCKETS))
    n = int(rng.integers(1, 9)) * bucket + int(rng.integers(0, bucket)) + (0 if case % 4 else 8192 * 3)
    W = int(rng.integers(1, 7))
    dither_bits = 16 if case % 3 == 2 else 32                     # one stream per call
    step = int(rng.integers(0, 2 ** 40))
    scale = float(rng.choice([1e-6, 1e-3, 1.0, 300.0]))
    side = (rng.standard_normal(n) * scale).astype(np.float32)
    grads = [(side + rng.standard_normal(n) * scale * float(rng.choice([0.01, 0.2, 1.0]))).astype(np.float32)
             for _ in range(W)]
    specs = [_random_spec(rng, dither_bits) for _ in range(W)]
    for w in range(W):                                             # encoder parity, worker by worker
        _check_encode(dq, oracle, grads[w], specs[w], worker=w, step=step, bucket=bucket)
    got, ref = _roundtrip_decode(dq, oracle, W, n, bucket, specs, grads, side, step)
    assert_fp32_close(got, ref, f"case {case}: bucket={bucket} n={n} W={W} specs={specs}")
    assert dq.device_error_flags() == 0
