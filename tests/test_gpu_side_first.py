"""GPU parity for the decoder that takes the reconstruction of message 0 as the side information of the nested
messages (Algorithm 2, server: the P1 worker is decoded first and serves the P2 workers)."""
import dataclasses

import numpy as np
import pytest

from dq_workloads.generators import DQSG, NDQSG, WorkerSpec, worker_seed

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import assert_fp32_close, gpu_msg, oracle_encode, oracle_msg  # noqa: E402
from test_gpu_parity import dq, oracle  # noqa: E402,F401


def _messages(dq, oracle, specs, grads, bucket, step):
    omsgs, gmsgs, keep = [], [], []
    for w, (sp, g) in enumerate(zip(specs, grads)):
        opk, osc = oracle_encode(oracle, g, sp, w, step, bucket)
        omsgs.append(oracle_msg(oracle, opk, osc, sp, w, bucket))
        pk = torch.from_numpy(np.concatenate([opk, np.zeros(4, np.uint32)]).view(np.int32)).cuda()
        sc = torch.from_numpy(osc.copy()).cuda()
        keep.append((pk, sc))
        gmsgs.append(gpu_msg(dq, pk, sc, sp, w, bucket))
    return omsgs, gmsgs, keep


@pytest.mark.parametrize("dither_bits", [32, 16])
@pytest.mark.parametrize("n", [1, 33, 5000, 3 * 8192 + 1000 + 7, 70 * 1024 + 5])
def test_side_first_matches_oracle_and_the_two_call_path(dq, oracle, n, dither_bits):
    rng = np.random.default_rng(7 * n + dither_bits)
    bucket = 1024 if n > 2000 else 32
    c = (0.01 * rng.standard_normal(n)).astype(np.float32)
    specs = [WorkerSpec(DQSG, 3, 5, seed=worker_seed(5, 0)),
             WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, worker_seed(5, 1)),
             WorkerSpec(NDQSG, 3, 0, 8, 8.0, 0.9, worker_seed(5, 2)),
             WorkerSpec(DQSG, 2, 3, seed=worker_seed(5, 3)),
             WorkerSpec(NDQSG, 3, 0, 5, 6.0, 1.0, worker_seed(5, 4)),
             WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, worker_seed(5, 5))]
    specs = [dataclasses.replace(s, dither_bits=dither_bits) for s in specs]
    grads = [(c + 0.003 * rng.standard_normal(n)).astype(np.float32) for _ in specs]
    omsgs, gmsgs, _keep = _messages(dq, oracle, specs, grads, bucket, step=9)
    # the oracle's definition: decode message 0 alone, give the result to the fused decode as side information
    y = oracle.decode_aggregate(omsgs[:1], n, 9, threads=4)
    ref = oracle.decode_aggregate(omsgs, n, 9, side_info=y, threads=4)
    got = dq.ndqsg_decode_aggregate_side_first(gmsgs, n, 9)
    side = dq.dqsg_decode_aggregate(gmsgs[:1], n, 9)
    two = dq.ndqsg_decode_aggregate(gmsgs, n, 9, side)
    torch.cuda.synchronize()
    got_h, two_h = got[:n].cpu().numpy(), two[:n].cpu().numpy()
    assert_fp32_close(got_h, ref, f"n={n}")
    assert np.array_equal(got_h.view(np.uint32), two_h.view(np.uint32)), "differs from the two-call path"
    assert dq.device_error_flags() == 0


def test_side_first_needs_a_dqsg_message_first(dq):
    sp = WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, worker_seed(5, 1))
    pk = torch.zeros(64, dtype=torch.int32, device="cuda")
    sc = torch.ones(4, dtype=torch.float32, device="cuda")
    with pytest.raises(dq.DqError):
        dq.ndqsg_decode_aggregate_side_first([gpu_msg(dq, pk, sc, sp, 0, 32)], 64, 0)


def test_side_first_from_host_buffers(dq, oracle):
    from dq_testlib import host_output
    n, bucket, step = 70 * 1024 + 5, 1024, 3
    rng = np.random.default_rng(99)
    c = (0.01 * rng.standard_normal(n)).astype(np.float32)
    specs = [WorkerSpec(DQSG, 3, 5, seed=worker_seed(6, 0)), WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, worker_seed(6, 1)),
             WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, worker_seed(6, 2))]
    grads = [(c + 0.003 * rng.standard_normal(n)).astype(np.float32) for _ in specs]
    omsgs, gmsgs, _keep = _messages(dq, oracle, specs, grads, bucket, step)
    host_msgs = [dq.Message(torch.from_numpy(om.packed.view(np.int32).copy()).pin_memory(),
                            torch.from_numpy(om.scale.copy()).pin_memory(), sp.seed, w, sp.kind, gm.params)
                 for w, (om, gm, sp) in enumerate(zip(omsgs, gmsgs, specs))]
    ws = torch.empty(dq.decode_workspace_bytes(host_msgs, n, False), dtype=torch.uint8, device="cuda")
    out = host_output(torch, n, torch.float32)
    dq.ndqsg_decode_aggregate_side_first_host(host_msgs, n, step, out, ws)
    dev = dq.ndqsg_decode_aggregate_side_first(gmsgs, n, step)
    torch.cuda.synchronize()
    assert np.array_equal(out.numpy().view(np.uint32), dev[:n].cpu().numpy().view(np.uint32))
