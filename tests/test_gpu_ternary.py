"""GPU parity for the radix-3 container (five ternary codes per byte): container bytes and the stream that comes
back are bit-exact against the oracle, on sizes that span many units and every ragged tail."""
import numpy as np
import pytest

from dq_workloads.generators import DQSG, WorkerSpec

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import assert_fp32_close, gpu_encode, gpu_msg, oracle_encode, oracle_msg, words_np  # noqa: E402
from test_gpu_parity import dq, oracle  # noqa: E402,F401


def _stream_dev(words: np.ndarray):
    return torch.from_numpy(words.view(np.int32).copy()).cuda()


@pytest.mark.parametrize("n", [1, 4, 5, 6, 15, 16, 17, 79, 80, 81, 159, 160, 161, 20479, 20480, 20481,
                               80 * 256 * 3 + 41, 1_000_003])
def test_pack_and_unpack_bit_exact(dq, oracle, n):
    rng = np.random.default_rng(n)
    codes = rng.integers(0, 3, size=n, dtype=np.uint32)
    words = oracle.pack(codes, 2)
    ref = oracle.ternary_pack(codes)
    assert dq.ternary_bytes(n) == ref.size == oracle.ternary_bytes(n)
    # the output buffers start out as all ones: every byte and every pad bit must be written
    out = torch.full((ref.size + 16,), 0xFF, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dq.ternary_pack(_stream_dev(words), n, out, status)
    got = out.cpu().numpy()
    assert np.array_equal(got[:ref.size], ref)
    assert (got[ref.size:] == 0xFF).all()                      # nothing written past the container
    assert int(status.item()) == 0
    back = torch.full((words.size + 4,), -1, dtype=torch.int32, device="cuda")
    dq.ternary_unpack(out, n, back)
    b = words_np(back)
    assert np.array_equal(b[:words.size], words)               # pad bits of the last word are 0 again
    assert (b[words.size:] == 0xFFFFFFFF).all()
    assert np.array_equal(b[:words.size], oracle.ternary_unpack_stream(ref, n))


def test_code_three_is_flagged_and_stored_as_two(dq, oracle):
    n = 5000
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 4, size=n, dtype=np.uint32)        # not a three-level message
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = dq.ternary_pack(_stream_dev(oracle.pack(codes, 2)), n, None, status)
    assert np.array_equal(out.cpu().numpy()[:oracle.ternary_bytes(n)], oracle.ternary_pack(codes))
    assert int(status.item()) == dq.DQ_WARN_CODE_RANGE
    back = words_np(dq.ternary_unpack(out, n))[:oracle.packed_words(n, 2)]
    assert np.array_equal(oracle.unpack(back, n, 2), np.minimum(codes, 2))


def test_garbage_past_the_end_of_the_stream_is_ignored(dq, oracle):
    n = 80 * 7 + 13                                            # the last word holds 13 codes, then pad bits
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 3, size=n, dtype=np.uint32)
    words = oracle.pack(codes, 2)
    dirty = words.copy()
    dirty[-1] |= np.uint32(0xFFFFFFFF) << np.uint32(2 * (n % 16))
    got = dq.ternary_pack(_stream_dev(dirty), n).cpu().numpy()[:oracle.ternary_bytes(n)]
    assert np.array_equal(got, oracle.ternary_pack(codes))


def test_three_level_messages_through_the_container_decode_identically(dq, oracle):
    # encode (L = 3) -> container -> back -> fused decode-and-average: the same mean as without the container,
    # and as the oracle's.
    rng = np.random.default_rng(11)
    W, bucket, step = 3, 512, 21
    n = 37 * bucket + 123
    specs = [WorkerSpec(DQSG, 2, 3, seed=500 + w) for w in range(W)]
    grads = [(rng.standard_normal(n) * 0.01).astype(np.float32) for _ in range(W)]
    direct, via, omsgs, keep = [], [], [], []
    total_container = 0
    for w, (g, s) in enumerate(zip(grads, specs)):
        pk, sc = gpu_encode(dq, torch, torch.from_numpy(g).cuda(), s, w, step, bucket)
        opk, osc = oracle_encode(oracle, g, s, w, step, bucket)
        data = dq.ternary_pack(pk, n)
        assert np.array_equal(data.cpu().numpy()[:oracle.ternary_bytes(n)], oracle.ternary_pack_stream(opk, n))
        total_container += dq.ternary_bytes(n)
        pk2 = dq.ternary_unpack(data, n)
        assert torch.equal(pk2[:pk.numel()], pk)
        keep += [pk, sc, pk2]
        direct.append(gpu_msg(dq, pk, sc, s, w, bucket))
        via.append(gpu_msg(dq, pk2, sc, s, w, bucket))
        omsgs.append(oracle_msg(oracle, opk, osc, s, w, bucket))
    assert total_container * 8 <= 1.6 * W * n + 8 * W
    a = dq.dqsg_decode_aggregate(direct, n, step)[:n].cpu().numpy()
    b = dq.dqsg_decode_aggregate(via, n, step)[:n].cpu().numpy()
    assert np.array_equal(a, b)
    assert_fp32_close(b, oracle.decode_aggregate(omsgs, n, step), "mean through the container")
    assert dq.device_error_flags() == 0


def test_rejects_bad_arguments(dq):
    ok = torch.zeros(64, dtype=torch.int32, device="cuda")
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(dq.DqError) as e:
        dq.ternary_pack(ok, 100, out[1:])                      # misaligned container
    assert e.value.status == 3
    with pytest.raises(dq.DqError) as e:
        dq.ternary_unpack(out[1:], 100, ok)
    assert e.value.status == 3
    assert dq.lib().dq_ternary_pack(None, 100, out.data_ptr(), None, None) == 1
    assert dq.lib().dq_ternary_unpack(out.data_ptr(), 100, None, None) == 1
    assert dq.lib().dq_ternary_pack(None, 0, None, None, None) == 0     # n = 0 is a no-op
