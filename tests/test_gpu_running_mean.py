"""GPU parity for Algorithm 2's server loop (side information = running mean of the messages decoded so far)."""
import dataclasses

import numpy as np
import pytest

import dq_workloads as wl
from dq_workloads.generators import DQSG, NDQSG, WorkerSpec, worker_seed

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import assert_fp32_close, gpu_msg, oracle_encode, oracle_msg  # noqa: E402
from test_gpu_parity import dq, oracle  # noqa: E402,F401


def _run(dq, oracle, specs, grads, n, bucket, step):
    omsgs, gmsgs, keep = [], [], []
    for w, (sp, g) in enumerate(zip(specs, grads)):
        opk, osc = oracle_encode(oracle, g, sp, w, step, bucket)
        omsgs.append(oracle_msg(oracle, opk, osc, sp, w, bucket))
        pk = torch.from_numpy(np.concatenate([opk, np.zeros(4, np.uint32)]).view(np.int32)).cuda()
        sc = torch.from_numpy(osc.copy()).cuda()
        keep.append((pk, sc))
        gmsgs.append(gpu_msg(dq, pk, sc, sp, w, bucket))
    ref = oracle.decode_aggregate(omsgs, n, step, running=True, threads=4)
    out = dq.ndqsg_decode_aggregate_running(gmsgs, n, step)
    torch.cuda.synchronize()
    return out[:n].cpu().numpy(), ref


@pytest.mark.parametrize("dither_bits", [32, 16])
@pytest.mark.parametrize("n", [33, 5000, 3 * 8192 + 1000 + 7])
def test_running_mean_decode_matches_oracle(dq, oracle, n, dither_bits):
    rng = np.random.default_rng(n + dither_bits)
    bucket = 1024 if n > 2000 else 32
    c = rng.standard_normal(n).astype(np.float32)
    specs = [WorkerSpec(DQSG, 3, 5, seed=worker_seed(3, 0)), WorkerSpec(DQSG, 4, 15, seed=worker_seed(3, 1)),
             WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, worker_seed(3, 2)), WorkerSpec(NDQSG, 3, 0, 8, 8.0, 0.9, worker_seed(3, 3)),
             WorkerSpec(NDQSG, 3, 0, 5, 6.0, 1.0, worker_seed(3, 4)), WorkerSpec(DQSG, 2, 3, seed=worker_seed(3, 5)),
             WorkerSpec(NDQSG, 1, 0, 2, 1.0, 1.0, worker_seed(3, 6))]
    specs = [dataclasses.replace(s, dither_bits=dither_bits) for s in specs]
    grads = [(c + 0.1 * rng.standard_normal(n)).astype(np.float32) for _ in specs]
    got, ref = _run(dq, oracle, specs, grads, n, bucket, step=4)
    assert assert_fp32_close(got, ref, f"n={n}")


def test_running_mean_full_size_resnet50_mix(dq, oracle):
    """The ResNet-50-sized workload with Algorithm 2's own side information; oracle on sampled bucket ranges."""
    cfg = wl.ndqsg_resnet50()
    n, B, step = cfg.n, cfg.bucket, cfg.step
    ranges = [(0, 4), (3000, 3004), (12476, 12480)]
    gmsgs, keep = [], []
    om = {r: [] for r in ranges}
    for w, sp in enumerate(cfg.workers):
        g = cfg.grad(w)
        p = dq.binding.make_params(B, sp.bits, sp.levels, sp.coarse_K, sp.fine_M, sp.alpha, sp.dither_bits)
        fn = dq.dqsg_encode if sp.kind == DQSG else dq.ndqsg_encode
        pk, sc = fn(torch.from_numpy(g).cuda(), sp.seed, w, step, p)
        keep.append((pk, sc))
        gmsgs.append(dq.Message(pk, sc, sp.seed, w, sp.kind, p))
        for (b0, b1) in ranges:
            lo, hi = b0 * B, min(n, b1 * B)
            opk, osc = oracle_encode(oracle, g[lo:hi], sp, w, step, B, i0=lo)
            om[(b0, b1)].append(oracle_msg(oracle, opk, osc, sp, w, B))
    out = dq.ndqsg_decode_aggregate_running(gmsgs, n, step)
    torch.cuda.synchronize()
    out_h = out[:n].cpu().numpy()
    for (b0, b1) in ranges:
        lo, hi = b0 * B, min(n, b1 * B)
        ref = oracle.decode_aggregate(om[(b0, b1)], hi - lo, step, i0=lo, running=True)
        assert assert_fp32_close(out_h[lo:hi], ref, f"buckets {b0}..{b1}")


def test_running_mean_requires_a_dqsg_message_first(dq):
    import ctypes as C
    P = dq.binding.make_params
    fake = 0x1000
    nd = dq.DqMsg(fake, fake, 1, 0, dq.DQ_KIND_NDQSG, P(512, 2, 0, 4, 4.0, 1.0))
    d = dq.DqMsg(fake, fake, 1, 0, dq.DQ_KIND_DQSG, P(512, 2))
    arr = (dq.DqMsg * 2)(nd, d)
    assert dq.lib().ndqsg_decode_aggregate_running(arr, 2, 1024, 0, fake, None, None) == 1
