"""GPU parity for the 16-bit dither stream (eight elements per Philox block): same comparisons as for the
default stream, against the oracle's own 16-bit stream."""
import dataclasses

import numpy as np
import pytest

import dq_workloads as wl
from dq_workloads.generators import DQSG, NDQSG, WorkerSpec

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import assert_fp32_close  # noqa: E402
from test_gpu_parity import _check_encode, _roundtrip_decode, _specs_for_bits, dq, oracle  # noqa: E402,F401
from test_gpu_fullsize import _run_full_size  # noqa: E402


def _d16(spec):
    return dataclasses.replace(spec, dither_bits=16)


@pytest.mark.parametrize("bits", range(1, 9))
def test_encode_bit_exact_all_widths_16_bit_dither(dq, oracle, bits):
    rng = np.random.default_rng(900 + bits)
    for bucket in (64, 2048):
        n = 9 * 8192 + 5 * bucket + 77
        g = (rng.standard_normal(n) * 0.02).astype(np.float32)
        for spec in _specs_for_bits(bits):
            _check_encode(dq, oracle, g, _d16(spec), worker=5, step=(1 << 32) + 9, bucket=bucket)


@pytest.mark.parametrize("bits", range(1, 9))
def test_decode_aggregate_all_widths_16_bit_dither(dq, oracle, bits):
    rng = np.random.default_rng(950 + bits)
    bucket, W = 256, 3
    n = 11 * bucket + 45
    side = (rng.standard_normal(n) * 0.02).astype(np.float32)
    grads = [(side + rng.standard_normal(n) * 0.004).astype(np.float32) for _ in range(W)]
    all_specs = [_d16(s) for s in _specs_for_bits(bits)]
    for variant in range(3):
        specs = [all_specs[(variant + w) % len(all_specs)] for w in range(W)]
        got, ref = _roundtrip_decode(dq, oracle, W, n, bucket, specs, grads, side, step=13)
        assert assert_fp32_close(got, ref, f"bits={bits} variant={variant}")


def test_streams_differ_and_must_match_between_encoder_and_decoder(dq, oracle):
    rng = np.random.default_rng(990)
    n, bucket = 40_000, 2048
    g = rng.standard_normal(n).astype(np.float32)
    s32 = WorkerSpec(DQSG, 2, 3, seed=77)
    pk32, *_ = _check_encode(dq, oracle, g, s32, 0, 1, bucket)
    pk16, *_ = _check_encode(dq, oracle, g, _d16(s32), 0, 1, bucket)
    assert not torch.equal(pk32, pk16)


def test_full_size_ndqsg_resnet50_16_bit_dither(dq, oracle):
    cfg = wl.with_dither_bits(wl.ndqsg_resnet50(), 16)
    assert all(s.dither_bits == 16 for s in cfg.workers)
    assert _run_full_size(dq, oracle, cfg, seed=16)


def test_full_size_dqsg_resnet18_16_bit_dither(dq, oracle):
    cfg = wl.with_dither_bits(wl.dqsg_resnet18(bits=2), 16)
    assert _run_full_size(dq, oracle, cfg, seed=17)
