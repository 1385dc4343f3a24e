"""GPU parity on seeded random configurations: combinations the hand-picked cases do not enumerate (odd bucket sizes
with mixed kinds and widths per worker, non-power-of-two coarse ratios with shrinkage, both dither streams, ragged
lengths, wide value ranges).  Every case is reproducible from its index."""
import numpy as np
import pytest

from dq_workloads.generators import DQSG, NDQSG, WorkerSpec

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import assert_fp32_close, host_output  # noqa: E402
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


@pytest.mark.parametrize("case", range(48))
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


@pytest.mark.parametrize("case", range(10))
def test_random_running_mean_configuration(dq, oracle, case):
    # Algorithm 2's server loop: the first message is DQSG, the rest are drawn at random
    from test_gpu_running_mean import _run
    rng = np.random.default_rng(78_000 + case)
    bucket = int(rng.choice(BUCKETS))
    n = int(rng.integers(1, 6)) * bucket + int(rng.integers(0, bucket)) + (0 if case % 3 else 8192 * 2)
    W = int(rng.integers(2, 7))
    dither_bits = 16 if case % 2 else 32
    step = int(rng.integers(0, 2 ** 40))
    c = rng.standard_normal(n).astype(np.float32)
    grads = [(c + 0.2 * rng.standard_normal(n)).astype(np.float32) for _ in range(W)]
    first = WorkerSpec(DQSG, 3, int(rng.integers(2, 9)), seed=int(rng.integers(0, 2 ** 63)), dither_bits=dither_bits)
    specs = [first] + [_random_spec(rng, dither_bits) for _ in range(W - 1)]
    got, ref = _run(dq, oracle, specs, grads, n, bucket, step)
    assert_fp32_close(got, ref, f"case {case}: bucket={bucket} n={n} specs={specs}")


@pytest.mark.parametrize("case", range(6))
def test_random_host_buffer_round_trip(dq, oracle, case):
    # the host-buffer entry points on random configurations: same bits and the same mean as the oracle
    from dq_testlib import oracle_encode, oracle_msg, spec_params
    rng = np.random.default_rng(79_000 + case)
    bucket = int(rng.choice(BUCKETS))
    n = int(rng.integers(1, 6)) * bucket + int(rng.integers(0, bucket))
    W = int(rng.integers(1, 5))
    dither_bits = 16 if case % 2 else 32
    step = int(rng.integers(0, 2 ** 40))
    side = rng.standard_normal(n).astype(np.float32)
    grads = [(side + 0.1 * rng.standard_normal(n)).astype(np.float32) for _ in range(W)]
    specs = [_random_spec(rng, dither_bits) for _ in range(W)]
    host_msgs, omsgs = [], []
    for w, (g, sp) in enumerate(zip(grads, specs)):
        p = spec_params(dq, sp, bucket)
        pk = host_output(torch, max(1, dq.packed_words(n, sp.bits)), torch.int32)
        sc = host_output(torch, max(1, dq.num_buckets(n, bucket)), torch.float32)
        ws = torch.empty(dq.encode_workspace_bytes(n, p), dtype=torch.uint8, device="cuda")
        fn = dq.dqsg_encode_host if sp.kind == DQSG else dq.ndqsg_encode_host
        fn(torch.from_numpy(g).pin_memory(), sp.seed, w, step, p, pk, sc, ws)
        opk, osc = oracle_encode(oracle, g, sp, w, step, bucket)
        assert np.array_equal(pk.numpy().view(np.uint32)[:opk.size], opk), f"case {case}: worker {w} {sp}"
        assert np.array_equal(sc.numpy()[:osc.size].view(np.uint32), osc.view(np.uint32))
        host_msgs.append(dq.Message(pk, sc, sp.seed, w, sp.kind, p))
        omsgs.append(oracle_msg(oracle, opk, osc, sp, w, bucket))
    any_nd = any(s.kind == NDQSG for s in specs)
    out = host_output(torch, n, torch.float32)
    ws = torch.empty(dq.decode_workspace_bytes(host_msgs, n, any_nd), dtype=torch.uint8, device="cuda")
    dq.ndqsg_decode_aggregate_host(host_msgs, n, step, torch.from_numpy(side).pin_memory() if any_nd else None, out, ws)
    ref = oracle.decode_aggregate(omsgs, n, step, side_info=side if any_nd else None, threads=4)
    assert_fp32_close(out.numpy(), ref, f"case {case}")
    assert dq.device_error_flags() == 0


@pytest.mark.parametrize("case", range(15))
def test_random_decode_with_several_draws_per_cta(dq, oracle, case):
    """Lengths up to three million elements, where every persistent decoder CTA draws several groups of units, in
    the three side-information modes (a given vector, the reconstruction of message 0, the running mean)."""
    from dq_testlib import gpu_msg, oracle_encode, oracle_msg
    rng = np.random.default_rng(910_000 + case)
    bucket = int(rng.choice(BUCKETS))
    n = int(rng.integers(1, 3_000_000))
    if case % 5 == 0:
        n = max(1024, (n // 1024) * 1024)                          # whole units now and then
    W = int(rng.integers(1, 10))
    dither_bits = 16 if case % 3 == 2 else 32
    step = int(rng.integers(0, 2 ** 40))
    mode = case % 3
    c = rng.standard_normal(n).astype(np.float32)
    grads = [(c + 0.2 * rng.standard_normal(n)).astype(np.float32) for _ in range(W)]
    specs = [_random_spec(rng, dither_bits) for _ in range(W)]
    if mode != 0:                                                  # Algorithm 2: the first message is DQSG
        specs[0] = WorkerSpec(DQSG, 3, int(rng.integers(2, 9)), seed=int(rng.integers(0, 2 ** 63)),
                              dither_bits=dither_bits)
    omsgs, gmsgs, keep = [], [], []
    for w, (sp, g) in enumerate(zip(specs, grads)):
        opk, osc = oracle_encode(oracle, g, sp, w, step, bucket)
        omsgs.append(oracle_msg(oracle, opk, osc, sp, w, bucket))
        pk = torch.from_numpy(np.concatenate([opk, np.zeros(4, np.uint32)]).view(np.int32)).cuda()
        sc = torch.from_numpy(osc.copy()).cuda()
        keep.append((pk, sc))
        gmsgs.append(gpu_msg(dq, pk, sc, sp, w, bucket))
    any_nd = any(s.kind == NDQSG for s in specs)
    if mode == 0:
        ref = oracle.decode_aggregate(omsgs, n, step, side_info=c if any_nd else None, threads=8)
        out = (dq.ndqsg_decode_aggregate(gmsgs, n, step, torch.from_numpy(c).cuda()) if any_nd
               else dq.dqsg_decode_aggregate(gmsgs, n, step))
    elif mode == 1:
        side = oracle.decode_aggregate(omsgs[:1], n, step, threads=8)
        ref = oracle.decode_aggregate(omsgs, n, step, side_info=side, threads=8)
        out = dq.ndqsg_decode_aggregate_side_first(gmsgs, n, step)
    else:
        ref = oracle.decode_aggregate(omsgs, n, step, running=True, threads=8)
        out = dq.ndqsg_decode_aggregate_running(gmsgs, n, step)
    torch.cuda.synchronize()
    assert_fp32_close(out[:n].cpu().numpy(), ref, f"case {case}: mode={mode} bucket={bucket} n={n} specs={specs}")
    assert dq.device_error_flags() == 0
