"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element, on the same
seeded inputs.  Packed words and scales must be bit-identical; reconstructed / averaged gradients must be
within max(1e-6 relative, 2 ulp) of the oracle's fp32 value."""
import numpy as np
import pytest

import dq_workloads as wl
from dq_workloads.generators import DQSG, NDQSG, WorkerSpec, default_levels, worker_seed

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def dq():
    from paper_1904_01197_b200 import build
    build.build()
    import paper_1904_01197_b200 as dq
    assert torch.cuda.is_available()
    return dq


@pytest.fixture(scope="module")
def oracle():
    import oracle
    oracle.build()
    return oracle


from dq_testlib import (assert_fp32_close, gpu_encode, gpu_msg, host_output, oracle_encode, oracle_msg,  # noqa: E402
                        spec_params, words_np)


def _specs_for_bits(bits):
    out = [WorkerSpec(DQSG, bits, default_levels(bits), seed=worker_seed(7, bits))]
    if bits >= 2:
        out.append(WorkerSpec(DQSG, bits, 1 << bits, seed=worker_seed(8, bits)))          # even level count
    out.append(WorkerSpec(NDQSG, bits, 0, 1 << bits, float(1 << bits), 1.0, worker_seed(9, bits)))
    if bits >= 2:
        K = (1 << bits) - 1                                                                # K not a power of two
        out.append(WorkerSpec(NDQSG, bits, 0, K, float(2 * K) + 0.5, 0.75, worker_seed(10, bits)))
    return out


def _check_encode(dq, oracle, g, spec, worker, step, bucket):
    gd = torch.from_numpy(g).cuda()
    pk, sc = gpu_encode(dq, torch, gd, spec, worker, step, bucket)
    torch.cuda.synchronize()
    opk, osc = oracle_encode(oracle, g, spec, worker, step, bucket)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), osc.view(np.uint32)), "scales differ"
    got = words_np(pk)
    if not np.array_equal(got, opk):
        bad = np.nonzero(got != opk)[0]
        raise AssertionError(f"packed words differ at {bad[:8]} ({bad.size} of {opk.size}); "
                             f"spec={spec} bucket={bucket} n={g.size}")
    return pk, sc, opk, osc


@pytest.mark.parametrize("bits", range(1, 9))
def test_encode_bit_exact_all_widths(dq, oracle, bits):
    rng = np.random.default_rng(100 + bits)
    bucket = 512
    n = 9 * bucket + 77                                   # several tiles, a partial bucket, a partial row
    g = (rng.standard_normal(n) * 0.02).astype(np.float32)
    for spec in _specs_for_bits(bits):
        _check_encode(dq, oracle, g, spec, worker=3, step=(1 << 33) + 5, bucket=bucket)


@pytest.mark.parametrize("bucket", [32, 64, 128, 256, 512, 1024, 2048, 4096, 8192, 96, 1504, 16384, 65536])
def test_encode_bit_exact_bucket_sizes(dq, oracle, bucket):
    rng = np.random.default_rng(200 + bucket)
    n = max(3 * bucket + 1000 + 13, 20_000)
    g = (rng.standard_normal(n) * rng.choice([1e-3, 1.0, 50.0])).astype(np.float32)
    for spec in (WorkerSpec(DQSG, 2, 3, seed=11), WorkerSpec(DQSG, 3, 5, seed=12),
                 WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, 13), WorkerSpec(NDQSG, 3, 0, 8, 16.0, 1.0, 14)):
        _check_encode(dq, oracle, g, spec, worker=1, step=9, bucket=bucket)


@pytest.mark.parametrize("bits", range(2, 9))
def test_encode_coarse_ratio_below_the_field_width(dq, oracle, bits):
    # every power of two K < 2^bits: the code is q1 mod K, not the low `bits` bits of q1
    rng = np.random.default_rng(250 + bits)
    n = 3 * 2048 + 8192 + 57
    g = (rng.standard_normal(n) * 0.3).astype(np.float32)
    for logk in range(1, bits):
        spec = WorkerSpec(NDQSG, bits, 0, 1 << logk, float(3 << logk), 1.0, 40 + logk)
        for bucket in (2048, 96):
            pk, sc, opk, osc = _check_encode(dq, oracle, g, spec, worker=2, step=5, bucket=bucket)
        assert oracle.unpack(opk, n, bits).max() < (1 << logk)


@pytest.mark.parametrize("n", [1, 3, 31, 32, 33, 100, 1023, 1024, 1025, 2048, 4097, 8191])
def test_encode_ragged_lengths(dq, oracle, n):
    rng = np.random.default_rng(300 + n)
    g = rng.standard_normal(n).astype(np.float32)
    for bucket in (32, 1024, 2048):
        for spec in (WorkerSpec(DQSG, 3, 7, seed=21), WorkerSpec(NDQSG, 3, 0, 5, 7.0, 1.0, 22)):
            _check_encode(dq, oracle, g, spec, worker=0, step=1, bucket=bucket)


def test_encode_degenerate_buckets(dq, oracle):
    n, bucket = 4 * 2048, 2048
    g = np.zeros(n, dtype=np.float32)
    g[2048 + 5] = 3.0e-38                                   # a tiny but nonzero bucket
    g[4096:6144] = -1.0                                     # constant bucket: every element sits on the top level
    g[6144] = 1e-42                                         # denormal scale: treated as a zero bucket
    for spec in (WorkerSpec(DQSG, 2, 3, seed=31), WorkerSpec(DQSG, 2, 4, seed=32),
                 WorkerSpec(NDQSG, 2, 0, 4, 4.0, 1.0, 33)):
        _check_encode(dq, oracle, g, spec, worker=2, step=0, bucket=bucket)


def test_empty_input_is_a_no_op(dq):
    p = dq.binding.make_params(512, 2)
    g = torch.zeros(4, device="cuda")
    pk = torch.full((4,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    sc = torch.full((4,), 7.0, device="cuda")
    L = dq.lib()
    assert L.dqsg_encode(g.data_ptr(), 0, 1, 0, 0, __import__("ctypes").byref(p), pk.data_ptr(), sc.data_ptr(), None) == 0
    torch.cuda.synchronize()
    assert (pk == 0x5A5A5A5A).all() and (sc == 7.0).all()


def _roundtrip_decode(dq, oracle, W, n, bucket, specs, grads, side, step):
    """Messages come from the oracle's encoder; both decoders see the same bits."""
    omsgs, gmsgs, keep = [], [], []
    for w in range(W):
        opk, osc = oracle_encode(oracle, grads[w], specs[w], w, step, bucket)
        omsgs.append(oracle_msg(oracle, opk, osc, specs[w], w, bucket))
        pk = torch.from_numpy(np.concatenate([opk, np.zeros(4, np.uint32)]).view(np.int32)).cuda()
        sc = torch.from_numpy(osc.copy()).cuda()
        keep.append((pk, sc))
        gmsgs.append(gpu_msg(dq, pk, sc, specs[w], w, bucket))
    any_nd = any(s.kind == NDQSG for s in specs)
    ref = oracle.decode_aggregate(omsgs, n, step, side_info=side if any_nd else None, threads=4)
    side_dev = torch.from_numpy(side).cuda() if any_nd else None
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    if any_nd:
        out = dq.ndqsg_decode_aggregate(gmsgs, n, step, side_dev, status_word=status)
    else:
        out = dq.dqsg_decode_aggregate(gmsgs, n, step)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    return out[:n].cpu().numpy(), ref


@pytest.mark.parametrize("bits", range(1, 9))
def test_decode_aggregate_all_widths(dq, oracle, bits):
    rng = np.random.default_rng(400 + bits)
    bucket, W = 256, 3
    n = 7 * bucket + 45
    side = (rng.standard_normal(n) * 0.02).astype(np.float32)
    grads = [(side + rng.standard_normal(n) * 0.004).astype(np.float32) for _ in range(W)]
    for variant in range(3):
        all_specs = _specs_for_bits(bits)
        specs = [all_specs[(variant + w) % len(all_specs)] for w in range(W)]
        got, ref = _roundtrip_decode(dq, oracle, W, n, bucket, specs, grads, side, step=77)
        assert_fp32_close(got, ref, f"bits={bits} variant={variant}")


@pytest.mark.parametrize("W", [1, 2, 3, 5, 8, 16, 33, 64])
def test_decode_aggregate_worker_counts(dq, oracle, W):
    rng = np.random.default_rng(500 + W)
    bucket = 1024
    n = 3 * bucket + 500
    side = rng.standard_normal(n).astype(np.float32)
    grads = [(side + 0.1 * rng.standard_normal(n)).astype(np.float32) for _ in range(W)]
    specs = [WorkerSpec(DQSG, 3, 5, seed=worker_seed(1, w)) if w % 3 == 0 else
             WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, worker_seed(1, w)) for w in range(W)]
    got, ref = _roundtrip_decode(dq, oracle, W, n, bucket, specs, grads, side, step=2)
    exact = assert_fp32_close(got, ref, f"W={W}")
    assert exact, "the prescribed operation order should make the average bit-identical"


@pytest.mark.parametrize("n", [1, 31, 32, 33, 1000, 4097])
def test_decode_ragged_lengths(dq, oracle, n):
    rng = np.random.default_rng(600 + n)
    side = rng.standard_normal(n).astype(np.float32)
    grads = [(side + 0.05 * rng.standard_normal(n)).astype(np.float32) for _ in range(2)]
    for bucket in (32, 2048):
        specs = [WorkerSpec(DQSG, 3, 7, seed=41), WorkerSpec(NDQSG, 3, 0, 6, 9.0, 0.9, 42)]
        got, ref = _roundtrip_decode(dq, oracle, 2, n, bucket, specs, grads, side, step=5)
        assert_fp32_close(got, ref, f"n={n} bucket={bucket}")


@pytest.mark.parametrize("units", [1, 3, 4, 5, 9, 147, 148, 149, 591, 592, 593, 597, 1187])
def test_decode_unit_counts(dq, oracle, units):
    """Lengths around the decoder's work distribution: a unit is 32 rows of 32 elements, warps take units in
    teams of four and a CTA per SM draws its teams' units from a counter, so the counts that matter are multiples
    of 4 and of (4 x number of SMs) and their neighbours; each with a whole last row, a ragged one and a short
    last unit."""
    rng = np.random.default_rng(650 + units)
    bucket = 2048
    for short in (0, 1, 1000):
        n = units * 1024 - short
        side = rng.standard_normal(n).astype(np.float32)
        grads = [(side + 0.05 * rng.standard_normal(n)).astype(np.float32) for _ in range(2)]
        specs = [WorkerSpec(DQSG, 3, 5, seed=43), WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, 44)]
        got, ref = _roundtrip_decode(dq, oracle, 2, n, bucket, specs, grads, side, step=9)
        assert assert_fp32_close(got, ref, f"units={units} n={n}")


def test_decode_with_a_wrong_step_matches_the_oracles_wrong_decode(dq, oracle):
    """A message whose header is corrupt (here: decoded at another step than it was encoded at) cannot be detected
    from the codes; the decoder must then compute exactly what the definition gives for that step, dither of the
    wrong stream and all, and must not flag the scales."""
    rng = np.random.default_rng(660)
    n, bucket, W, step = 9 * 2048 + 333, 2048, 3, 11
    side = rng.standard_normal(n).astype(np.float32)
    grads = [(side + 0.05 * rng.standard_normal(n)).astype(np.float32) for _ in range(W)]
    specs = [WorkerSpec(DQSG, 3, 5, seed=45), WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, 46),
             WorkerSpec(NDQSG, 3, 0, 6, 9.0, 0.9, 47)]
    omsgs, gmsgs, keep = [], [], []
    for w in range(W):
        opk, osc = oracle_encode(oracle, grads[w], specs[w], w, step, bucket)
        omsgs.append(oracle_msg(oracle, opk, osc, specs[w], w, bucket))
        pk = torch.from_numpy(np.concatenate([opk, np.zeros(4, np.uint32)]).view(np.int32)).cuda()
        sc = torch.from_numpy(osc.copy()).cuda()
        keep.append((pk, sc))
        gmsgs.append(gpu_msg(dq, pk, sc, specs[w], w, bucket))
    right = oracle.decode_aggregate(omsgs, n, step, side_info=side, threads=4)
    wrong = oracle.decode_aggregate(omsgs, n, step + 1, side_info=side, threads=4)
    assert np.abs(wrong - right).max() > 0.01                 # the other stream's dither is visible
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    out = dq.ndqsg_decode_aggregate(gmsgs, n, step + 1, torch.from_numpy(side).cuda(), status_word=status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    assert assert_fp32_close(out[:n].cpu().numpy(), wrong, "wrong step")


def test_decodes_and_encodes_on_two_streams_at_once(dq, oracle):
    """Launches of the library that run side by side on two streams share nothing but the error word: results are
    those of the same calls made one after the other."""
    rng = np.random.default_rng(670)
    n, bucket, step, W = 1_500_000 + 77, 2048, 4, 4
    jobs = []
    for j in range(2):
        side = rng.standard_normal(n).astype(np.float32)
        grads = [(side + 0.05 * rng.standard_normal(n)).astype(np.float32) for _ in range(W)]
        specs = [WorkerSpec(DQSG, 3, 5, seed=100 + j)] + [WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, 110 + 10 * j + w)
                                                         for w in range(1, W)]
        gdev = [torch.from_numpy(g).cuda() for g in grads]
        jobs.append((specs, gdev, torch.from_numpy(side).cuda()))
    def run(j, stream):
        specs, gdev, side = jobs[j]
        msgs = []
        for w, sp in enumerate(specs):
            p = spec_params(dq, sp, bucket)
            fn = dq.dqsg_encode if sp.kind == DQSG else dq.ndqsg_encode
            pk, sc = fn(gdev[w], sp.seed, w, step, p, stream=stream)
            msgs.append(gpu_msg(dq, pk, sc, sp, w, bucket))
        return msgs, dq.ndqsg_decode_aggregate(msgs, n, step, side, stream=stream)
    torch.cuda.synchronize()
    serial = [run(j, None) for j in range(2)]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for rep in range(3):
        both = [run(j, streams[j]) for j in range(2)]
        torch.cuda.synchronize()
        for j in range(2):
            for m_s, m_b in zip(serial[j][0], both[j][0]):
                assert torch.equal(m_s.packed, m_b.packed) and torch.equal(m_s.scale, m_b.scale)
            assert torch.equal(serial[j][1], both[j][1]), f"job {j}, repetition {rep}"
    assert dq.device_error_flags() == 0


def test_decode_dqsg_only_and_shrinkage(dq, oracle):
    rng = np.random.default_rng(700)
    n, bucket, W = 50_000, 2048, 4
    side = rng.standard_normal(n).astype(np.float32)
    grads = [(side + 0.2 * rng.standard_normal(n)).astype(np.float32) for _ in range(W)]
    specs = [WorkerSpec(DQSG, b, default_levels(b), seed=50 + b) for b in (1, 2, 3, 4)]
    got, ref = _roundtrip_decode(dq, oracle, W, n, bucket, specs, grads, side, step=3)
    assert assert_fp32_close(got, ref, "dqsg only")
    specs = [WorkerSpec(NDQSG, 3, 0, 8, 8.0, a, 60 + i) for i, a in enumerate((1.0, 0.9, 0.5, 0.99))]
    got, ref = _roundtrip_decode(dq, oracle, W, n, bucket, specs, grads, side, step=3)
    assert assert_fp32_close(got, ref, "shrinkage")


def test_nonfinite_scale_sets_the_status_word(dq, oracle):
    n, bucket = 4096, 1024
    g = np.linspace(-1, 1, n).astype(np.float32)
    spec = WorkerSpec(DQSG, 2, 3, seed=5)
    opk, osc = oracle_encode(oracle, g, spec, 0, 1, bucket)
    osc = osc.copy()
    osc[2] = np.inf
    pk = torch.from_numpy(opk.view(np.int32)).cuda()
    sc = torch.from_numpy(osc).cuda()
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    dq.ndqsg_decode_aggregate([gpu_msg(dq, pk, sc, spec, 0, bucket)], n, 1, None, status_word=status)
    torch.cuda.synchronize()
    assert int(status[0]) & dq.DQ_WARN_NONFINITE_SCALE


def test_end_to_end_tiny_config(dq, oracle):
    """Config 1: W=2, d=65536, bucket 512; 2-bit DQSG, and NDQSG with K=4 against y = c."""
    for kind in ("dqsg", "mixed", "ndqsg"):
        cfg = wl.tiny(kind=kind)
        side = cfg.side_info()
        omsgs, gmsgs, keep = [], [], []
        for w, spec in enumerate(cfg.workers):
            g = cfg.grad(w)
            pk, sc, opk, osc = _check_encode(dq, oracle, g, spec, w, cfg.step, cfg.bucket)
            keep.append((pk, sc))
            omsgs.append(oracle_msg(oracle, opk, osc, spec, w, cfg.bucket))
            gmsgs.append(gpu_msg(dq, pk.contiguous(), sc.contiguous(), spec, w, cfg.bucket))
        ref = oracle.decode_aggregate(omsgs, cfg.n, cfg.step, side_info=side)
        out = dq.ndqsg_decode_aggregate(gmsgs, cfg.n, cfg.step, torch.from_numpy(side).cuda())
        torch.cuda.synchronize()
        assert assert_fp32_close(out[:cfg.n].cpu().numpy(), ref, kind)
        # the average is close to the true mean gradient: error below the per-worker bound kappa*Delta/2
        true = np.mean([cfg.grad(w) for w in range(cfg.W)], axis=0)
        assert np.abs(ref - true).max() < 0.5
    assert dq.device_error_flags() == 0


def test_host_buffer_entry_points(dq, oracle):
    rng = np.random.default_rng(800)
    n, bucket = 100_000 + 17, 2048
    g = rng.standard_normal(n).astype(np.float32)
    spec = WorkerSpec(DQSG, 3, 5, seed=71)
    nspec = WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, 72)
    msgs, omsgs = [], []
    for w, sp in enumerate((spec, nspec)):
        p = dq.binding.make_params(bucket, sp.bits, sp.levels, sp.coarse_K, sp.fine_M, sp.alpha)
        ws = torch.empty(dq.encode_workspace_bytes(n, p), dtype=torch.uint8, device="cuda")
        gh = torch.from_numpy(g).pin_memory()
        pk = host_output(torch, dq.packed_words(n, sp.bits), torch.int32)
        sc = host_output(torch, dq.num_buckets(n, bucket), torch.float32)
        fn = dq.dqsg_encode_host if sp.kind == DQSG else dq.ndqsg_encode_host
        fn(gh, sp.seed, w, 4, p, pk, sc, ws)
        opk, osc = oracle_encode(oracle, g, sp, w, 4, bucket)
        assert np.array_equal(pk.numpy().view(np.uint32), opk) and np.array_equal(sc.numpy(), osc)
        msgs.append(dq.Message(pk, sc, sp.seed, w, sp.kind, p))
        omsgs.append(oracle_msg(oracle, opk, osc, sp, w, bucket))
    side = torch.from_numpy((g + 0.01 * rng.standard_normal(n)).astype(np.float32)).pin_memory()
    out = host_output(torch, n, torch.float32)
    ws = torch.empty(dq.decode_workspace_bytes(msgs, n, True), dtype=torch.uint8, device="cuda")
    dq.ndqsg_decode_aggregate_host(msgs, n, 4, side, out, ws)
    ref = oracle.decode_aggregate(omsgs, n, 4, side_info=side.numpy())
    assert assert_fp32_close(out.numpy(), ref, "host entry points")


def test_half_dithered_decode_matches_oracle(dq, oracle):
    """The receiver without the dither (Section 2.1): mean of kappa * Delta * q over the workers."""
    import dataclasses
    rng = np.random.default_rng(1234)
    n, bucket, W = 3 * 8192 + 777, 1024, 5
    specs = [WorkerSpec(DQSG, b, default_levels(b), seed=90 + b) for b in (1, 2, 3, 4, 8)]
    omsgs, gmsgs, keep = [], [], []
    for w, sp in enumerate(specs):
        g = rng.standard_normal(n).astype(np.float32)
        opk, osc = oracle_encode(oracle, g, sp, w, 6, bucket)
        omsgs.append(oracle_msg(oracle, opk, osc, dataclasses.replace(sp, dither_bits=0), w, bucket))
        pk = torch.from_numpy(np.concatenate([opk, np.zeros(4, np.uint32)]).view(np.int32)).cuda()
        sc = torch.from_numpy(osc.copy()).cuda()
        keep.append((pk, sc))
        gmsgs.append(gpu_msg(dq, pk, sc, sp, w, bucket))
    ref = oracle.decode_aggregate(omsgs, n, 6)
    out = dq.dqsg_decode_aggregate_half_dithered(gmsgs, n)
    torch.cuda.synchronize()
    assert assert_fp32_close(out[:n].cpu().numpy(), ref, "half-dithered")


@pytest.mark.parametrize("bits", [1, 2, 3, 5, 8])
def test_code_histogram_matches_oracle_counts(dq, oracle, bits):
    rng = np.random.default_rng(4321 + bits)
    n = 300_000 + 19
    g = rng.standard_normal(n).astype(np.float32)
    spec = WorkerSpec(DQSG, bits, default_levels(bits), seed=66)
    pk, sc, opk, osc = _check_encode(dq, oracle, g, spec, 0, 3, 2048)
    want = np.bincount(oracle.unpack(opk, n, bits), minlength=1 << bits)
    hist = dq.code_histogram(pk.contiguous(), n, bits)
    torch.cuda.synchronize()
    assert np.array_equal(hist.cpu().numpy(), want)
    H = dq.entropy_bits_per_element(hist)
    p = want[want > 0] / n
    assert abs(H + (p * np.log2(p)).sum()) < 1e-9
