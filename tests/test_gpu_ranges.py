"""GPU parity for bucket ranges: a gradient encoded / decoded in pieces gives the bits and values of the whole-vector
calls (and of the oracle run on the same range with its global offset)."""
import dataclasses

import numpy as np
import pytest

from dq_workloads.generators import DQSG, NDQSG, WorkerSpec

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import (assert_fp32_close, gpu_encode, gpu_msg, host_output, oracle_encode, oracle_msg,  # noqa: E402
                        spec_params, words_np)
from test_gpu_parity import dq, oracle  # noqa: E402,F401

SPECS = [WorkerSpec(DQSG, 2, 3, seed=601), WorkerSpec(DQSG, 3, 5, seed=602), WorkerSpec(DQSG, 1, 2, seed=603),
         WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, 604), WorkerSpec(NDQSG, 3, 0, 5, 7.0, 0.8, 605),
         WorkerSpec(NDQSG, 4, 0, 4, 6.0, 1.0, 606)]


def _encode_range(dq, g_dev, lo, hi, spec, worker, step, bucket):
    p = spec_params(dq, spec, bucket)
    fn = dq.dqsg_encode_range if spec.kind == DQSG else dq.ndqsg_encode_range
    pk, sc = fn(g_dev[lo:hi], lo, spec.seed, worker, step, p)
    n = hi - lo
    return pk[:dq.packed_words(n, spec.bits)], sc[:dq.num_buckets(n, bucket)]


def _cuts(n, bucket, rng, pieces):
    nb = -(-n // bucket)
    inner = sorted(set(int(b) for b in rng.integers(1, nb, size=pieces - 1))) if nb > 1 else []
    return [0] + [b * bucket for b in inner] + [n]


@pytest.mark.parametrize("dither_bits", [32, 16])
@pytest.mark.parametrize("bucket", [96, 512, 2048, 4096])
def test_ranges_concatenate_to_the_whole_message_and_mean(dq, oracle, bucket, dither_bits):
    rng = np.random.default_rng(bucket + dither_bits)
    n = 23 * bucket + bucket // 3 + 5
    step = (7 << 32) + 11
    side = rng.standard_normal(n).astype(np.float32)
    specs = [dataclasses.replace(s, dither_bits=dither_bits) for s in SPECS]
    grads = [(side + 0.15 * rng.standard_normal(n)).astype(np.float32) for _ in specs]
    cuts = _cuts(n, bucket, rng, 5)
    side_dev = torch.from_numpy(side).cuda()
    whole_msgs, keep = [], []
    range_msgs = {(lo, hi): [] for lo, hi in zip(cuts[:-1], cuts[1:])}
    for w, (g, sp) in enumerate(zip(grads, specs)):
        g_dev = torch.from_numpy(g).cuda()
        pk, sc = gpu_encode(dq, torch, g_dev, sp, w, step, bucket)
        whole_msgs.append(gpu_msg(dq, pk, sc, sp, w, bucket))
        parts_pk, parts_sc = [], []
        for lo, hi in zip(cuts[:-1], cuts[1:]):
            rpk, rsc = _encode_range(dq, g_dev, lo, hi, sp, w, step, bucket)
            opk, osc = oracle_encode(oracle, g[lo:hi], sp, w, step, bucket, i0=lo)
            assert np.array_equal(words_np(rpk), opk), f"worker {w} range {lo}:{hi}"
            assert np.array_equal(rsc.cpu().numpy().view(np.uint32), osc.view(np.uint32))
            parts_pk.append(words_np(rpk))
            parts_sc.append(rsc.cpu().numpy())
            range_msgs[(lo, hi)].append(gpu_msg(dq, rpk, rsc, sp, w, bucket))
            keep += [rpk, rsc]
        # a range starts at a word boundary of the stream: the pieces are the whole message cut at those words
        assert np.array_equal(np.concatenate(parts_pk), words_np(pk))
        assert np.array_equal(np.concatenate(parts_sc).view(np.uint32), sc.cpu().numpy().view(np.uint32))
        keep += [pk, sc, g_dev]
    whole = dq.ndqsg_decode_aggregate(whole_msgs, n, step, side_dev)[:n].cpu().numpy()
    pieces = []
    for (lo, hi), msgs in range_msgs.items():
        out = dq.ndqsg_decode_aggregate_range(msgs, hi - lo, lo, step, side_dev[lo:hi])
        pieces.append(out[:hi - lo].cpu().numpy())
    assert np.array_equal(np.concatenate(pieces).view(np.uint32), whole.view(np.uint32))
    assert dq.device_error_flags() == 0


def test_range_far_into_a_long_gradient(dq, oracle):
    # element indices beyond 2^32: the dither counters of the range must be those of the whole vector
    bucket, n, step = 2048, 5 * 2048 + 77, 3
    lo = (1 << 33) + 6 * bucket
    rng = np.random.default_rng(9)
    side = rng.standard_normal(n).astype(np.float32)
    specs = [WorkerSpec(DQSG, 3, 7, seed=701), WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, 702),
             WorkerSpec(NDQSG, 3, 0, 8, 8.0, 1.0, 703, dither_bits=32)]
    for dither_bits in (32, 16):
        gm, om, keep = [], [], []
        for w, sp0 in enumerate(specs):
            sp = dataclasses.replace(sp0, dither_bits=dither_bits)
            g = (side + 0.2 * rng.standard_normal(n)).astype(np.float32)
            g_dev = torch.from_numpy(g).cuda()
            p = spec_params(dq, sp, bucket)
            fn = dq.dqsg_encode_range if sp.kind == DQSG else dq.ndqsg_encode_range
            pk, sc = fn(g_dev, lo, sp.seed, w, step, p)
            opk, osc = oracle_encode(oracle, g, sp, w, step, bucket, i0=lo)
            assert np.array_equal(words_np(pk)[:opk.size], opk), f"worker {w}"
            assert np.array_equal(sc.cpu().numpy()[:osc.size].view(np.uint32), osc.view(np.uint32))
            gm.append(gpu_msg(dq, pk, sc, sp, w, bucket))
            om.append(oracle_msg(oracle, opk, osc, sp, w, bucket))
            keep += [pk, sc]
        out = dq.ndqsg_decode_aggregate_range(gm, n, lo, step, torch.from_numpy(side).cuda())[:n].cpu().numpy()
        ref = oracle.decode_aggregate(om, n, step, side_info=side, i0=lo)
        assert_fp32_close(out, ref, f"dither_bits={dither_bits}")


def test_a_range_must_start_at_a_bucket_boundary(dq):
    p = dq.binding.make_params(512, 2)
    g = torch.zeros(2048, device="cuda")
    with pytest.raises(dq.DqError) as e:
        dq.dqsg_encode_range(g, 100, 1, 0, 0, p)
    assert e.value.status == 1
    pk, sc = dq.dqsg_encode_range(g, 1024, 1, 0, 0, p)
    with pytest.raises(dq.DqError) as e:
        dq.ndqsg_decode_aggregate_range([dq.Message(pk, sc, 1, 0, dq.DQ_KIND_DQSG, p)], 2048, 256, 0, None)
    assert e.value.status == 1
    with pytest.raises(dq.DqError) as e:                       # beyond the supported length
        dq.dqsg_encode_range(g, (1 << 34), 1, 0, 0, p)
    assert e.value.status == 2


@pytest.mark.parametrize("bucket,bits_mix", [(2048, (3, 2, 2)), (96, (1, 5, 3))])
def test_host_buffer_decode_of_a_long_gradient(dq, oracle, bucket, bits_mix):
    # the host-buffer decode of a few million elements: same bits as the device entry point on the whole vector,
    # and as the oracle on sampled bucket ranges (encoded and decoded with their global offset)
    rng = np.random.default_rng(bucket)
    n = (1 << 21) + 37 * bucket + 19
    step = 12
    side = rng.standard_normal(n).astype(np.float32)
    specs = [WorkerSpec(DQSG, bits_mix[0], 0, seed=801), WorkerSpec(NDQSG, bits_mix[1], 0, 1 << bits_mix[1], 4.0, 1.0, 802),
             WorkerSpec(NDQSG, bits_mix[2], 0, (1 << bits_mix[2]) - 1 if bits_mix[2] > 1 else 2, 3.0, 0.9, 803)]
    dev_msgs, host_msgs, keep = [], [], []
    grads = []
    for w, sp in enumerate(specs):
        g = (side + 0.1 * rng.standard_normal(n)).astype(np.float32)
        grads.append(g)
        pk, sc = gpu_encode(dq, torch, torch.from_numpy(g).cuda(), sp, w, step, bucket)
        dev_msgs.append(gpu_msg(dq, pk, sc, sp, w, bucket))
        hpk, hsc = pk.cpu().pin_memory(), sc.cpu().pin_memory()
        host_msgs.append(dq.Message(hpk, hsc, sp.seed, w, sp.kind, spec_params(dq, sp, bucket)))
        keep += [pk, sc, hpk, hsc]
    whole = dq.ndqsg_decode_aggregate(dev_msgs, n, step, torch.from_numpy(side).cuda())[:n].cpu().numpy()
    out = host_output(torch, n, torch.float32)
    ws = torch.empty(dq.decode_workspace_bytes(host_msgs, n, True), dtype=torch.uint8, device="cuda")
    for _ in range(2):                                   # twice: the staging area is reused
        out.zero_()
        dq.ndqsg_decode_aggregate_host(host_msgs, n, step, torch.from_numpy(side).pin_memory(), out, ws)
        assert np.array_equal(out.numpy().view(np.uint32), whole.view(np.uint32))
    for b0 in (0, (n // bucket) // 2, n // bucket - 1):  # oracle on three bucket pairs, the ragged end included
        lo, hi = b0 * bucket, min(n, (b0 + 2) * bucket)
        om = []
        for w, sp in enumerate(specs):
            opk, osc = oracle_encode(oracle, grads[w][lo:hi], sp, w, step, bucket, i0=lo)
            om.append(oracle_msg(oracle, opk, osc, sp, w, bucket))
        ref = oracle.decode_aggregate(om, hi - lo, step, side_info=side[lo:hi], i0=lo)
        assert_fp32_close(out.numpy()[lo:hi], ref, f"buckets from {b0}")
    assert dq.device_error_flags() == 0
