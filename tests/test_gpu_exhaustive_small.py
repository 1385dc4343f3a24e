"""Every small length, every code width, both quantizers: the edge cases of the tiling (ragged last row, ragged
last bucket, last unit, buffers that end a few bytes after the last word) in one sweep, with guard words around
every output (the autouse fixture of conftest.py).  Lengths: every n up to four buckets and five elements for
buckets of 32 and 96 elements; for buckets of 2048 every n up to 70 and every n within 35 elements of the first
four bucket boundaries."""
import numpy as np
import pytest

from dq_workloads.generators import DQSG, NDQSG, WorkerSpec, worker_seed

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import assert_fp32_close, gpu_msg, oracle_encode, oracle_msg, spec_params, words_np  # noqa: E402
from test_gpu_parity import dq, oracle  # noqa: E402,F401


def _lengths(bucket):
    if bucket <= 96:
        return list(range(1, 4 * bucket + 6))
    ns = set(range(1, 71))
    for k in range(1, 5):
        ns.update(range(k * bucket - 35, k * bucket + 36))
    return sorted(ns)


@pytest.mark.parametrize("kind", [DQSG, NDQSG])
@pytest.mark.parametrize("bits", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("bucket", [32, 96, 2048])
def test_every_small_length(dq, oracle, guarded_outputs, bucket, bits, kind):
    rng = np.random.default_rng(1000 * bucket + 10 * bits + kind)
    nmax = max(_lengths(bucket))
    base = (0.02 * rng.standard_normal(nmax)).astype(np.float32)
    noise = (0.004 * rng.standard_normal(nmax)).astype(np.float32)
    first = WorkerSpec(DQSG, 3, 5, seed=worker_seed(11, 0))
    if kind == DQSG:
        sp = WorkerSpec(DQSG, bits, 0, seed=worker_seed(11, 1))
    else:
        K = (1 << bits) if bits % 2 else max(2, (1 << bits) - 1)          # powers of two and other ratios
        sp = WorkerSpec(NDQSG, bits, 0, K, 4.0, 1.0, worker_seed(11, 1))
    step = 3
    for n in _lengths(bucket):
        g0, g1 = base[:n], (base[:n] + noise[:n])
        o0 = oracle_encode(oracle, g0, first, 0, step, bucket, threads=1)
        o1 = oracle_encode(oracle, g1, sp, 1, step, bucket, threads=1)
        p1 = spec_params(dq, sp, bucket)
        fn = dq.dqsg_encode if kind == DQSG else dq.ndqsg_encode
        pk, sc = fn(torch.from_numpy(g1).cuda(), sp.seed, 1, step, p1)
        assert np.array_equal(words_np(pk)[:o1[0].size], o1[0]), f"n={n}: packed words differ"
        assert np.array_equal(sc.cpu().numpy()[:o1[1].size], o1[1]), f"n={n}: scales differ"
        pk0 = torch.from_numpy(o0[0].view(np.int32).copy()).cuda()
        sc0 = torch.from_numpy(o0[1].copy()).cuda()
        gm = [gpu_msg(dq, pk0, sc0, first, 0, bucket), gpu_msg(dq, pk, sc, sp, 1, bucket)]
        om = [oracle_msg(oracle, o0[0], o0[1], first, 0, bucket), oracle_msg(oracle, o1[0], o1[1], sp, 1, bucket)]
        ref = oracle.decode_aggregate(om, n, step, side_info=g0.copy() if kind == NDQSG else None, threads=1)
        if kind == NDQSG:
            out = dq.ndqsg_decode_aggregate(gm, n, step, torch.from_numpy(g0.copy()).cuda())
        else:
            out = dq.dqsg_decode_aggregate(gm, n, step)
        assert_fp32_close(out.cpu().numpy()[:n], ref, f"n={n}")
        guarded_outputs.check()                      # per length, so that a stray write names its n
    assert dq.device_error_flags() == 0
