"""Bandwidth sweep of the encode and fused decode-aggregate kernels: n from 2^16 to 2^28, W in {2, 8, 32}, 1-4
bits, buckets of 256 to 8192 elements.

    python -m bench_tools.sweep [--quick] [--out FILE]

Star design around (n = 2^26, W = 8, b = 2, B = 2048): one axis varies at a time; DQSG and NDQSG, both dither
streams; each kernel is timed alone with CUDA events over buffers that rotate through more than 3x the L2 size
(points whose data fits the L2 are marked).  Gradients are N(0,1) drawn on the device (timing only; parity of
sweep-shaped inputs is covered by the tests).  Prints one table row per point and, with --out, JSON lines.
"""
from __future__ import annotations

import argparse
import json

import torch

from paper_1904_01197_b200 import binding as dq

L2_BYTES = 126 * 1024 * 1024


def _time(launches, iters):
    for i in range(3):
        launches[i % len(launches)]()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        launches[i % len(launches)]()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def run_point(n, W, bits, bucket, kind, dither_bits, hbm_peak, iters=20):
    dev = torch.device("cuda")
    nested = kind == "ndqsg"
    K = 1 << bits
    p = dq.make_params(bucket, bits, 0, K if nested else 0, float(K) if nested else 0.0, 1.0 if nested else 0.0,
                       dither_bits)
    rot = max(2, min(8, -(-3 * L2_BYTES // (4 * n))))
    gen = torch.Generator(device=dev).manual_seed(n % 1000 + bits)
    grads = [torch.randn(n, device=dev, generator=gen) for _ in range(rot)]
    enc = dq.ndqsg_encode if nested else dq.dqsg_encode
    pk, sc = dq.alloc_message(n, p, dev)
    ms_enc = _time([(lambda g=g: enc(g, 1234, 0, 1, p, pk, sc)) for g in grads], iters)
    enc_bytes = 4 * n + 4 * dq.packed_words(n, bits) + 4 * dq.num_buckets(n, bucket)
    # decode: W messages (encoded from the rotating gradients), side information, output; rotate whole sets
    per_set = W * (4 * dq.packed_words(n, bits) + 4 * dq.num_buckets(n, bucket)) + 4 * n * (2 if nested else 1)
    sets = max(2, min(6, -(-3 * L2_BYTES // per_set)))
    msg_sets, sides, outs = [], [], []
    for s in range(sets):
        msgs = []
        for w in range(W):
            pkw, scw = dq.alloc_message(n, p, dev)
            enc(grads[(s + w) % rot], 1000 + w, w, 1, p, pkw, scw)
            msgs.append(dq.Message(pkw, scw, 1000 + w, w, dq.DQ_KIND_NDQSG if nested else dq.DQ_KIND_DQSG, p))
        msg_sets.append(msgs)
        sides.append(grads[s % rot] if nested else None)
        outs.append(torch.empty(n, device=dev))
    if nested:
        launches = [(lambda a=msg_sets[i], b=sides[i], c=outs[i]: dq.ndqsg_decode_aggregate(a, n, 1, b, c))
                    for i in range(sets)]
    else:
        launches = [(lambda a=msg_sets[i], c=outs[i]: dq.dqsg_decode_aggregate(a, n, 1, c)) for i in range(sets)]
    ms_dec = _time(launches, max(4, iters // 2))
    return {"n": n, "W": W, "bits": bits, "bucket": bucket, "kind": kind, "dither_bits": dither_bits,
            "l2_resident": 4 * n * rot < L2_BYTES,
            "encode_us": ms_enc * 1e3, "encode_gbs": enc_bytes / ms_enc / 1e6,
            "encode_frac_hbm": enc_bytes / ms_enc / 1e6 / hbm_peak, "encode_gelem_s": n / ms_enc / 1e6,
            "decode_us": ms_dec * 1e3, "decode_gbs": per_set / ms_dec / 1e6,
            "decode_frac_hbm": per_set / ms_dec / 1e6 / hbm_peak, "decode_gelem_worker_s": n * W / ms_dec / 1e6}


def points(quick):
    base = dict(n=1 << 26, W=8, bits=2, bucket=2048)
    pts = []
    for kind in ("dqsg", "ndqsg"):
        for d in (32, 16):
            ns = [1 << 20, 1 << 24, 1 << 26] if quick else [1 << 16, 1 << 18, 1 << 20, 1 << 22, 1 << 24, 1 << 26, 1 << 28]
            for n in ns:
                pts.append(dict(base, n=n, kind=kind, dither_bits=d, W=8 if n < (1 << 28) else 2))
            if quick:
                continue
            for W in (2, 32):
                pts.append(dict(base, W=W, kind=kind, dither_bits=d, n=1 << 24 if W == 32 else 1 << 26))
            for b in (1, 3, 4):
                pts.append(dict(base, bits=b, kind=kind, dither_bits=d))
            for B in (256, 512, 1024, 4096, 8192):
                pts.append(dict(base, bucket=B, kind=kind, dither_bits=d))
    return pts


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--out", default="")
    ap.add_argument("--hbm-peak", type=float, default=6555.0, help="GB/s used for the fractions")
    args = ap.parse_args()
    rows = []
    print(f"{'kind':6s} {'dith':>4s} {'n':>10s} {'W':>3s} {'b':>2s} {'B':>5s} | {'enc us':>8s} {'GB/s':>7s} {'%hbm':>5s} {'Gel/s':>7s} | "
          f"{'dec us':>9s} {'GB/s':>7s} {'%hbm':>5s} {'Gel*w/s':>8s}")
    for pt in points(args.quick):
        r = run_point(hbm_peak=args.hbm_peak, **pt)
        rows.append(r)
        tag = " (L2)" if r["l2_resident"] else ""
        print(f"{r['kind']:6s} {r['dither_bits']:4d} {r['n']:10d} {r['W']:3d} {r['bits']:2d} {r['bucket']:5d} | "
              f"{r['encode_us']:8.1f} {r['encode_gbs']:7.0f} {100 * r['encode_frac_hbm']:5.1f} {r['encode_gelem_s']:7.1f} | "
              f"{r['decode_us']:9.1f} {r['decode_gbs']:7.0f} {100 * r['decode_frac_hbm']:5.1f} {r['decode_gelem_worker_s']:8.1f}{tag}",
              flush=True)
        torch.cuda.empty_cache()
    if args.out:
        with open(args.out, "w") as f:
            for r in rows:
                f.write(json.dumps(r) + "\n")


if __name__ == "__main__":
    main()
