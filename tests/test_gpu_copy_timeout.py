"""The bounded wait of the tile pipeline: a copy that never lands must end in an error flag, not in a hang.

DQ_FLAG_TEST_DROP_COPY makes one warp of the encoder announce the copy of its last work unit without issuing it.
Nothing is broken on the device: the wait gives up after its 20 ms bound, the kernel runs to its end, and the host
reads DQ_ERR_COPY_TIMEOUT; every other unit of the message is still bit-identical to the oracle's."""
import time

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from test_gpu_parity import dq, oracle  # noqa: E402,F401


@pytest.mark.parametrize("bucket", [512, 2048])
def test_a_copy_that_never_lands_sets_the_error_flag_and_the_kernel_ends(dq, oracle, bucket):
    n = 2 * 3 * 148 * 8 * max(1024, bucket) + 12345          # every warp of the persistent grid has two units or more
    rng = np.random.default_rng(bucket)
    g = (0.01 * rng.standard_normal(n)).astype(np.float32)
    gd = torch.from_numpy(g).cuda()
    assert dq.device_error_flags() == 0
    p = dq.binding.make_params(bucket, 2, 3, flags=dq.binding.DQ_FLAG_TEST_DROP_COPY)
    t0 = time.perf_counter()
    pk, sc = dq.dqsg_encode(gd, 5, 1, 2, p)
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    assert elapsed < 5.0, "the wait must give up after its bound"
    assert dq.device_error_flags() == dq.DQ_ERR_COPY_TIMEOUT
    assert dq.device_error_flags() == 0                      # reading clears the word
    # exactly one work unit (at most max(1024, bucket) elements) may differ from the oracle's message
    opk, osc = oracle.dqsg_encode(g, 5, 1, 2, bucket, 2, 3, threads=8)
    got = pk.cpu().numpy().view(np.uint32)[:opk.size]
    bad = np.nonzero(got != opk)[0]
    unit_words = max(1024, bucket) * 2 // 32
    assert bad.size == 0 or bad.max() // unit_words == bad.min() // unit_words
    bad_sc = np.nonzero(sc.cpu().numpy()[:osc.size].view(np.uint32) != osc.view(np.uint32))[0]
    unit_buckets = max(1024, bucket) // bucket
    assert bad_sc.size == 0 or bad_sc.max() // unit_buckets == bad_sc.min() // unit_buckets
    if bad.size and bad_sc.size:
        assert bad.min() // unit_words == bad_sc.min() // unit_buckets
    # and a normal call afterwards is clean
    p0 = dq.binding.make_params(bucket, 2, 3)
    pk2, sc2 = dq.dqsg_encode(gd, 5, 1, 2, p0)
    torch.cuda.synchronize()
    assert np.array_equal(pk2.cpu().numpy().view(np.uint32)[:opk.size], opk)
    assert dq.device_error_flags() == 0
