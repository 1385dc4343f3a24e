"""Shared helpers of the GPU parity tests: run one workload through the CUDA library and through the
oracle, on the same seeded inputs."""
from __future__ import annotations

import numpy as np

import dq_workloads as wl
from dq_workloads.generators import DQSG, NDQSG, WorkerSpec


def spec_params(dq, spec: WorkerSpec, bucket: int):
    return dq.binding.make_params(bucket, spec.bits, spec.levels, spec.coarse_K, spec.fine_M, spec.alpha,
                                  spec.dither_bits)


def gpu_encode(dq, torch, g_dev, spec: WorkerSpec, worker: int, step: int, bucket: int):
    p = spec_params(dq, spec, bucket)
    fn = dq.dqsg_encode if spec.kind == DQSG else dq.ndqsg_encode
    packed, scale = fn(g_dev, spec.seed, worker, step, p)
    n = g_dev.numel()
    return packed[:dq.packed_words(n, spec.bits)], scale[:dq.num_buckets(n, bucket)]


def oracle_encode(oracle, g: np.ndarray, spec: WorkerSpec, worker: int, step: int, bucket: int, i0: int = 0,
                  threads: int = 4):
    if spec.kind == DQSG:
        return oracle.dqsg_encode(g, spec.seed, worker, step, bucket, spec.bits, spec.levels, i0=i0,
                                  threads=threads, dither_bits=spec.dither_bits)
    return oracle.ndqsg_encode(g, spec.seed, worker, step, bucket, spec.bits, spec.coarse_K, spec.fine_M,
                               spec.alpha, i0=i0, threads=threads, dither_bits=spec.dither_bits)


def oracle_msg(oracle, packed, scale, spec: WorkerSpec, worker: int, bucket: int):
    return oracle.Msg(packed, scale, spec.seed, worker, spec.kind, bucket, spec.bits, spec.levels,
                      spec.coarse_K, spec.fine_M, spec.alpha, spec.dither_bits)


def gpu_msg(dq, packed_dev, scale_dev, spec: WorkerSpec, worker: int, bucket: int):
    return dq.Message(packed_dev, scale_dev, spec.seed, worker, spec.kind, spec_params(dq, spec, bucket))


def words_np(t) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint32)


def assert_fp32_close(got: np.ndarray, ref: np.ndarray, what: str = ""):
    """|got - ref| <= max(1e-6 |ref|, 2 ulp(ref)): the stated tolerance for reconstructed / averaged values."""
    got = np.asarray(got, dtype=np.float32)
    ref = np.asarray(ref, dtype=np.float32)
    assert got.shape == ref.shape, what
    tol = np.maximum(1e-6 * np.abs(ref.astype(np.float64)), 2.0 * np.spacing(np.abs(ref)).astype(np.float64))
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    bad = err > tol
    assert not bad.any(), f"{what}: {int(bad.sum())} of {bad.size} outside tolerance, worst {err.max()} at {int(err.argmax())}"
    return bool(np.array_equal(got.view(np.uint32), ref.view(np.uint32)))


def host_output(torch, numel: int, dtype):
    """A pinned host buffer for a *_host entry point's output, with guard words around it while a GPU test runs."""
    import conftest
    if conftest.CURRENT_GUARD is not None:
        return conftest.CURRENT_GUARD.host_output(numel, dtype)
    return torch.empty(numel, dtype=dtype).pin_memory()
