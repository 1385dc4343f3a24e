#!/usr/bin/env python
"""Benchmark of the DQSG / NDQSG hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic gradients: every worker's encode
(per-bucket scale, dither, quantize, coset, pack), the W=1 decode that produces the side information when the
workload takes it from worker 0, and the fused decode-and-average over all W messages.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is the whole-job algorithmic GB/s of a step with every input
resident in HBM; `e2e` is the same metric through the host-buffer C-ABI calls with the host<->device copies
inside the timed region; `roofline` describes the dominant kernel, `kernels` every kernel class timed alone
on rotating, larger-than-L2 buffers; `cpu_baseline` is the CPU oracle on a bounded sample of the workload.
With N > 1 every rank runs an independent replica of the workload on its own GPU (no collective on the data
path) and the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "encode / fused decode-aggregate GB/s and % of HBM peak on 1 B200; Gelem/s"
L2_BYTES = 126 * 1024 * 1024
HBM_NOMINAL_GBS = 8000.0
SM_COUNT, ISSUE_PER_SM_CLK, LANES = 148, 4, 32           # ALU-issue ceiling: SMs x schedulers x lanes x clock
# Algorithmic lane-instructions: ~22 per (element, worker) + ~10 per element for the fused decode,
# ~24 per element for the encode.
DEC_INSTR_PER_ELEM_WORKER, DEC_INSTR_PER_ELEM, ENC_INSTR_PER_ELEM = 22.0, 10.0, 24.0
# Executed lane-instructions per (element, worker) of the fused decode on the ResNet-50-sized workload, from the
# opcode counters in profiles/decode_aggregate_kernel_ndqsg_resnet50.md: (32x32->64 multiplies, fp32 adds /
# multiplies / multiply-adds, everything else).  Their scheduler cost is taken from the issue probe
# (profiles/issue_cost_probe_b200.md): 4.4 cycles per wide multiply with one other instruction hidden behind it,
# 1 cycle per fp32 instruction, 2 cycles for the rest; the classes add up.
DEC_MIX = {32: (4.34, 9.82, 12.52), 16: (2.20, 9.82, 9.88)}
ISSUE_CYCLES_WIDE, ISSUE_CYCLES_FP32, ISSUE_CYCLES_OTHER = 4.4, 1.0, 2.0
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/; keyed by (kernel class, workload, n).  None once a kernel has changed since its capture.
NCU_TRAFFIC = {
    ("encode", "ndqsg_resnet50", 25_557_032, 2): 106_543_616,    # profiles/encode_kernel_ndqsg_resnet50.md
    ("encode", "ndqsg_resnet50", 25_557_032, 3): 106_651_648,
    ("decode", "ndqsg_resnet50", 25_557_032): 223_945_472,       # profiles/decode_aggregate_kernel_ndqsg_resnet50.md
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="ndqsg_resnet50",
                    choices=["tiny", "dqsg_resnet18", "ndqsg_resnet50", "ndqsg_gpt2_small"])
    ap.add_argument("--bits", type=int, default=2, help="bits for the dqsg_resnet18 workload (1, 2 or 3)")
    ap.add_argument("--dither-bits", type=int, default=32, choices=[32, 16],
                    help="random bits per dither value: 32 (one Philox word per element) or 16 (half a word)")
    ap.add_argument("--n", type=int, default=0, help="override the gradient length (debugging / profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-kernels", action="store_true", help="skip the per-kernel isolated timings")
    ap.add_argument("--profile", action="store_true",
                    help="for runs under a profiler: only warm-up + timed steps, no sampler, no extra legs")
    ap.add_argument("--cpu-sample", type=int, default=1 << 25, help="elements per worker in the oracle sample")
    a = ap.parse_args()
    if a.profile:
        a.no_cpu_baseline = a.no_e2e = a.no_kernels = True
    return a


def make_workload(args, rank: int):
    import dq_workloads as wl
    kw = {"seed": rank}
    if args.n:
        kw["n"] = args.n
    if args.workload == "dqsg_resnet18":
        kw["bits"] = args.bits
    return wl.by_name(args.workload, dither_bits=args.dither_bits, **kw)


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            d = json.loads(p.read_text())
            return float(d["hbm_gbs"]), "measured", float(d.get("sm_max_mhz", 1965.0))
        except Exception:
            pass
    return 6650.0, "fallback", 1965.0


# ------------------------------------------------------------------------------------------ ranks
def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_value(step_bytes_per_rank: int, world: int, ms_per_step: float) -> float:
    """GB/s of the whole job: every rank processes its own replica of the workload (weak scaling)."""
    return world * step_bytes_per_rank / ms_per_step / 1e6


# ------------------------------------------------------------------------------------------ bytes
def encode_bytes(dq, n, spec, bucket):
    return 4 * n + 4 * dq.packed_words(n, spec.bits) + 4 * dq.num_buckets(n, bucket)


def decode_bytes(dq, n, specs, bucket, has_side):
    b = sum(4 * dq.packed_words(n, s.bits) + 4 * dq.num_buckets(n, bucket) for s in specs)
    return b + 4 * n + (4 * n if has_side else 0)


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        rows = [r.strip().split(", ") for r in Path(self.tmp.name).read_text().splitlines() if r.strip()]
        os.unlink(self.tmp.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for nm, v in zip(names, r[4:8]):
                if v.strip().lower().startswith("active"):
                    reasons.add(nm)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------ GPU state
class GpuState:
    """Device buffers of one replica: W gradients, W message buffers, side information, output."""

    def __init__(self, dq, torch, cfg, dev, share=None):
        """share: another GpuState of the same workload whose gradients (and side information) are reused."""
        from dq_workloads.generators import DQSG
        self.dq, self.torch, self.cfg, self.dev = dq, torch, cfg, dev
        self.DQSG = DQSG
        self.params = [dq.binding.make_params(cfg.bucket, s.bits, s.levels, s.coarse_K, s.fine_M, s.alpha,
                                              s.dither_bits)
                       for s in cfg.workers]
        if share is not None:
            self.grads_host, self.grads = share.grads_host, share.grads
        else:
            self.grads_host = [torch.from_numpy(cfg.grad(w)).pin_memory() for w in range(cfg.W)]
            self.grads = [g.to(dev, non_blocking=True) for g in self.grads_host]
        self.msg_buf = [dq.binding.alloc_message(cfg.n, p, dev) for p in self.params]
        self.msgs = [dq.Message(pk, sc, s.seed, w, s.kind, p)
                     for w, (s, p, (pk, sc)) in enumerate(zip(cfg.workers, self.params, self.msg_buf))]
        self.any_nested = any(s.kind != DQSG for s in cfg.workers)
        if cfg.side_info is not None and share is not None:
            self.side_host, self.side = share.side_host, share.side
        elif cfg.side_info is not None:
            self.side_host = torch.from_numpy(cfg.side_info()).pin_memory()
            self.side = self.side_host.to(dev)
        elif cfg.side_from_worker0:
            self.side_host = None
            self.side = torch.empty(cfg.n, dtype=torch.float32, device=dev)
        else:
            self.side_host = None
            self.side = None
        self.out = torch.empty(cfg.n, dtype=torch.float32, device=dev)
        torch.cuda.synchronize()

    def encode(self, w, grad=None, bufs=None):
        s, p = self.cfg.workers[w], self.params[w]
        pk, sc = bufs if bufs is not None else self.msg_buf[w]
        fn = self.dq.dqsg_encode if s.kind == self.DQSG else self.dq.ndqsg_encode
        fn(self.grads[w] if grad is None else grad, s.seed, w, self.cfg.step, p, pk, sc)

    def side_decode(self):
        self.dq.dqsg_decode_aggregate(self.msgs[:1], self.cfg.n, self.cfg.step, self.side)

    def decode(self, msgs=None, side=None, out=None):
        msgs = self.msgs if msgs is None else msgs
        out = self.out if out is None else out
        if self.any_nested:
            self.dq.ndqsg_decode_aggregate(msgs, self.cfg.n, self.cfg.step, self.side if side is None else side, out)
        else:
            self.dq.dqsg_decode_aggregate(msgs, self.cfg.n, self.cfg.step, out)

    def step(self, ev_mid=None):
        for w in range(self.cfg.W):
            self.encode(w)
        if ev_mid is not None:
            ev_mid.record()
        if self.cfg.side_from_worker0:
            self.side_decode()
        self.decode()

    def step_bytes(self):
        cfg, dq = self.cfg, self.dq
        enc = sum(encode_bytes(dq, cfg.n, s, cfg.bucket) for s in cfg.workers)
        dec = decode_bytes(dq, cfg.n, cfg.workers, cfg.bucket, self.any_nested)
        if cfg.side_from_worker0:
            dec += decode_bytes(dq, cfg.n, cfg.workers[:1], cfg.bucket, False)
        return enc, dec


def time_isolated(torch, launches, iters=24, warm=3):
    """Average duration (ms) of the launches in `launches` (callables on rotating buffers), CUDA events."""
    for i in range(warm):
        launches[i % len(launches)]()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        launches[i % len(launches)]()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def kernel_timings(st: GpuState, hbm_peak, sm_max_mhz):
    """Each kernel class alone, cold: rotating over buffers that together exceed the L2."""
    torch, dq, cfg = st.torch, st.dq, st.cfg
    res = {}
    n = cfg.n
    alu_peak = SM_COUNT * ISSUE_PER_SM_CLK * LANES * sm_max_mhz * 1e6      # lane-instructions / s
    # encode: one entry per distinct worker spec, rotating over the W gradients (W x 4n bytes >> L2 at full size)
    seen = {}
    for w, s in enumerate(cfg.workers):
        key = (s.kind, s.bits, s.levels, s.coarse_K)
        seen.setdefault(key, w)
    rot = max(1, min(cfg.W, -(-3 * L2_BYTES // (4 * n))))
    for key, w in seen.items():
        s = cfg.workers[w]
        launches = [(lambda gg=st.grads[(w + r) % cfg.W], ww=w: st.encode(ww, grad=gg)) for r in range(rot)]
        ms = time_isolated(torch, launches)
        by = encode_bytes(dq, n, s, cfg.bucket)
        name = f"encode_{'dqsg' if s.kind == st.DQSG else 'ndqsg'}_b{s.bits}"
        res[name] = {"ms": ms, "bytes": by, "gbs": by / ms / 1e6, "gelem_s": n / ms / 1e6,
                     "frac_hbm": by / ms / 1e6 / hbm_peak, "rotating_buffers": rot,
                     "alu_tinstr_s": ENC_INSTR_PER_ELEM * n / ms / 1e9,
                     "frac_alu": ENC_INSTR_PER_ELEM * n / ms * 1e3 / alu_peak,
                     "traffic": NCU_TRAFFIC.get(("encode", cfg.name, n, s.bits)) if s.dither_bits == 32 else None}
    # decode: rotate over message sets / side / out copies so that nothing is L2-resident
    per_set = decode_bytes(dq, n, cfg.workers, cfg.bucket, st.any_nested)
    sets = max(2, min(6, -(-3 * L2_BYTES // per_set)))
    if cfg.side_from_worker0:
        st.side_decode()
    msg_sets, sides, outs = [], [], []
    for _ in range(sets):
        ms_ = []
        for w, m in enumerate(st.msgs):
            ms_.append(dq.Message(m.packed.clone(), m.scale.clone(), m.seed, m.worker, m.kind, m.params))
        msg_sets.append(ms_)
        sides.append(st.side.clone() if st.side is not None else None)
        outs.append(torch.empty_like(st.out))
    launches = [(lambda a=msg_sets[i], b=sides[i], c=outs[i]: st.decode(a, b, c)) for i in range(sets)]
    ms = time_isolated(torch, launches, iters=12)
    if not st.any_nested:
        # the receiver without the dither (no random numbers): the memory-bound limit of the decoder
        half_l = [(lambda a=msg_sets[i], c=outs[i]: dq.dqsg_decode_aggregate_half_dithered(a, n, c)) for i in range(sets)]
        ms_h = time_isolated(torch, half_l, iters=12)
        res["decode_aggregate_half_dithered"] = {"ms": ms_h, "bytes": per_set, "gbs": per_set / ms_h / 1e6,
                                                 "gelem_s": n / ms_h / 1e6, "frac_hbm": per_set / ms_h / 1e6 / hbm_peak,
                                                 "gelem_worker_s": n * cfg.W / ms_h / 1e6}
    if st.any_nested and cfg.workers[0].kind == st.DQSG:
        # Algorithm 2's own server loop on the same messages: side information = running mean, no vector read
        run_l = [(lambda a=msg_sets[i], c=outs[i]: dq.ndqsg_decode_aggregate_running(a, n, cfg.step, c))
                 for i in range(sets)]
        ms_run = time_isolated(torch, run_l, iters=12)
        by_run = per_set - 4 * n
        res["decode_aggregate_running_mean"] = {"ms": ms_run, "bytes": by_run, "gbs": by_run / ms_run / 1e6,
                                                "gelem_s": n / ms_run / 1e6,
                                                "frac_hbm": by_run / ms_run / 1e6 / hbm_peak,
                                                "gelem_worker_s": n * cfg.W / ms_run / 1e6}
    tern = [w for w, s in enumerate(cfg.workers) if s.kind == st.DQSG and s.bits == 2 and (s.levels or 3) == 3]
    if tern:
        # three-level messages: the radix-3 container (five codes per byte) and back; only packed data is touched
        src = [m[tern[0]].packed for m in msg_sets]
        data = [dq.ternary_pack(p_, n) for p_ in src]
        by_t = 4 * dq.packed_words(n, 2) + dq.ternary_bytes(n)
        ms_p = time_isolated(torch, [(lambda a=src[i], b=data[i]: dq.ternary_pack(a, n, b)) for i in range(sets)])
        ms_u = time_isolated(torch, [(lambda a=data[i], b=src[i]: dq.ternary_unpack(a, n, b)) for i in range(sets)])
        for name, ms_t in (("ternary_pack", ms_p), ("ternary_unpack", ms_u)):
            res[name] = {"ms": ms_t, "bytes": by_t, "gbs": by_t / ms_t / 1e6, "gelem_s": n / ms_t / 1e6,
                         "frac_hbm": by_t / ms_t / 1e6 / hbm_peak,
                         "container_bits_per_element": 8 * dq.ternary_bytes(n) / n}
    elem_workers = n * cfg.W
    alg_instr = DEC_INSTR_PER_ELEM_WORKER * elem_workers + DEC_INSTR_PER_ELEM * n
    res["decode_aggregate"] = {"ms": ms, "bytes": per_set, "gbs": per_set / ms / 1e6, "gelem_s": n / ms / 1e6,
                               "frac_hbm": per_set / ms / 1e6 / hbm_peak,
                               "gelem_worker_s": elem_workers / ms / 1e6, "rotating_buffers": sets,
                               "alu_tinstr_s": alg_instr / ms / 1e9, "frac_alu": alg_instr / ms * 1e3 / alu_peak,
                               "alu_peak_tinstr_s": alu_peak / 1e12,
                               "traffic": (NCU_TRAFFIC.get(("decode", cfg.name, n))
                                           if cfg.workers[0].dither_bits == 32 else None)}
    return res


def run_e2e(st: GpuState, steps: int):
    """The same step through the host-buffer C-ABI calls: pinned host buffers in, pinned host buffers out."""
    torch, dq, cfg = st.torch, st.dq, st.cfg
    n = cfg.n
    host_msgs = []
    ws_enc = []
    for w, (s, p) in enumerate(zip(cfg.workers, st.params)):
        pk = torch.empty(max(1, dq.packed_words(n, s.bits)), dtype=torch.int32).pin_memory()
        sc = torch.empty(max(1, dq.num_buckets(n, cfg.bucket)), dtype=torch.float32).pin_memory()
        host_msgs.append(dq.Message(pk, sc, s.seed, w, s.kind, p))
        ws_enc.append(dq.encode_workspace_bytes(n, p))
    ws = torch.empty(max(max(ws_enc), dq.decode_workspace_bytes(host_msgs, n, True)), dtype=torch.uint8,
                     device=st.dev)
    side_host = st.side_host if st.side_host is not None else torch.empty(n, dtype=torch.float32).pin_memory()
    out_host = torch.empty(n, dtype=torch.float32).pin_memory()
    h2d = d2h = 0

    def one():
        nonlocal h2d, d2h
        h2d = d2h = 0
        for w, (s, p, m) in enumerate(zip(cfg.workers, st.params, host_msgs)):
            fn = dq.dqsg_encode_host if s.kind == st.DQSG else dq.ndqsg_encode_host
            fn(st.grads_host[w], s.seed, w, cfg.step, p, m.packed, m.scale, ws)
            h2d += 4 * n
            d2h += 4 * dq.packed_words(n, s.bits) + 4 * dq.num_buckets(n, cfg.bucket)
        if cfg.side_from_worker0:
            dq.ndqsg_decode_aggregate_host(host_msgs[:1], n, cfg.step, None, side_host, ws)
            h2d += 4 * dq.packed_words(n, cfg.workers[0].bits) + 4 * dq.num_buckets(n, cfg.bucket)
            d2h += 4 * n
        dq.ndqsg_decode_aggregate_host(host_msgs, n, cfg.step, side_host if st.any_nested else None, out_host, ws)
        h2d += sum(4 * dq.packed_words(n, s.bits) + 4 * dq.num_buckets(n, cfg.bucket) for s in cfg.workers)
        h2d += 4 * n if st.any_nested else 0
        d2h += 4 * n

    one()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / steps
    return dt, h2d, d2h, float(out_host[:8].sum())


# ------------------------------------------------------------------------------------------ CPU oracle
def oracle_step(cfg, sample: int, threads: int):
    """The oracle on the first `sample` elements (bucket-aligned) of every worker; returns seconds, bytes."""
    import oracle
    from dq_workloads.generators import DQSG
    ns = min(cfg.n, max(cfg.bucket, sample // cfg.bucket * cfg.bucket))
    grads = [cfg.grad(w)[:ns].copy() for w in range(cfg.W)]
    side = cfg.side_info()[:ns].copy() if cfg.side_info is not None else None
    t0 = time.perf_counter()
    msgs = []
    for w, s in enumerate(cfg.workers):
        if s.kind == DQSG:
            pk, sc = oracle.dqsg_encode(grads[w], s.seed, w, cfg.step, cfg.bucket, s.bits, s.levels, threads=threads,
                                        dither_bits=s.dither_bits)
        else:
            pk, sc = oracle.ndqsg_encode(grads[w], s.seed, w, cfg.step, cfg.bucket, s.bits, s.coarse_K, s.fine_M,
                                         s.alpha, threads=threads, dither_bits=s.dither_bits)
        msgs.append(oracle.Msg(pk, sc, s.seed, w, s.kind, cfg.bucket, s.bits, s.levels, s.coarse_K, s.fine_M,
                               s.alpha, s.dither_bits))
    if cfg.side_from_worker0:
        side = oracle.decode_aggregate(msgs[:1], ns, cfg.step, threads=threads)
    any_nd = any(s.kind != DQSG for s in cfg.workers)
    oracle.decode_aggregate(msgs, ns, cfg.step, side_info=side if any_nd else None, threads=threads)
    return time.perf_counter() - t0, ns


def algorithmic_step_bytes_host(cfg, n):
    """Same byte accounting as GpuState.step_bytes, without needing the CUDA library."""
    from dq_workloads.generators import DQSG
    words = lambda b: (n * b + 31) // 32
    nb = (n + cfg.bucket - 1) // cfg.bucket
    enc = sum(4 * n + 4 * words(s.bits) + 4 * nb for s in cfg.workers)
    any_nd = any(s.kind != DQSG for s in cfg.workers)
    dec = sum(4 * words(s.bits) + 4 * nb for s in cfg.workers) + 4 * n + (4 * n if any_nd else 0)
    if cfg.side_from_worker0:
        dec += 4 * words(cfg.workers[0].bits) + 4 * nb + 4 * n
    return enc + dec


def cpu_baseline(cfg, sample: int):
    import oracle
    oracle.build()
    threads = os.cpu_count() or 1
    secs, ns = oracle_step(cfg, sample, threads)
    by = algorithmic_step_bytes_host(cfg, ns)
    return {"value": by / secs / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": f"first {ns} elements of each of the {cfg.W} workers (whole step, {secs:.2f} s)",
            "gelem_s": ns / secs / 1e9}


def workload_config(cfg, args):
    return {"workload": cfg.name, "n": cfg.n, "W": cfg.W, "bucket": cfg.bucket, "dither_bits": args.dither_bits,
            "workers": sorted({f"{'dqsg' if s.kind == 0 else 'ndqsg'}:b{s.bits}:L{s.levels}:K{s.coarse_K}"
                               for s in cfg.workers}),
            "side_info": "decode of worker 0" if cfg.side_from_worker0 else ("given" if cfg.side_info else "none"),
            "l2_policy": "inputs larger than L2: every step streams W gradients of 4n bytes from HBM",
            "replicas": args.gpus}


# ------------------------------------------------------------------------------------------ reference arm
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = make_workload(args, 0)
    import oracle
    oracle.build()
    threads = os.cpu_count() or 1
    sample = args.cpu_sample
    for _ in range(min(args.warmup, 1)):
        oracle_step(cfg, min(sample, 1 << 20), threads)
    times, ns = [], 0
    budget_t0 = time.perf_counter()
    for _ in range(args.steps):
        secs, ns = oracle_step(cfg, sample, threads)
        times.append(secs)
        if time.perf_counter() - budget_t0 > 150:
            break
    secs = sum(times) / len(times)
    by = algorithmic_step_bytes_host(cfg, ns)
    val = by / secs / 1e9
    sample_txt = f"first {ns} elements of each of the {cfg.W} workers per step"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": len(times), "warmup": min(args.warmup, 1), "ms_per_step": secs * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(cfg, args), "gelem_s": ns / secs / 1e9,
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample_txt},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ main
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_1904_01197_b200 import build as dq_build
    if rank == 0:
        dq_build.build()
    if world > 1:
        dist.barrier()
    import paper_1904_01197_b200 as dq

    hbm_peak, peak_src, sm_max_mhz = measured_peaks()
    cfg = make_workload(args, rank)
    st = GpuState(dq, torch, cfg, dev)
    enc_bytes, dec_bytes = st.step_bytes()

    for _ in range(max(args.warmup, 3)):
        st.step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", "")
    except Exception:
        gpu_id = str(local)
    sampler = None if args.profile else ClockSampler(gpu_id)
    launches0 = dq.launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.steps + 1)]
    torch.cuda.synchronize()
    ev[0].record()
    for k in range(args.steps):
        st.step(ev_mid=ev[2 * k + 1])
        ev[2 * k + 2].record()
    torch.cuda.synchronize()
    launches = dq.launch_count() - launches0
    total_ms = ev[0].elapsed_time(ev[-1])
    enc_ms = sum(ev[2 * k].elapsed_time(ev[2 * k + 1]) for k in range(args.steps)) / args.steps
    dec_ms = sum(ev[2 * k + 1].elapsed_time(ev[2 * k + 2]) for k in range(args.steps)) / args.steps
    # keep the GPU busy a little longer if the timed region was too short for the sampler to see it
    t_end = time.perf_counter() + (0.0 if args.profile else max(0.0, 0.5 - total_ms / 1e3))
    while time.perf_counter() < t_end:
        st.step()
        torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
    assert dq.device_error_flags() == 0, "a kernel reported a copy timeout"

    total_ms, enc_ms, dec_ms = max_over_ranks([total_ms, enc_ms, dec_ms], dev)
    ms_per_step = total_ms / args.steps
    step_bytes = enc_bytes + dec_bytes
    value = whole_job_value(step_bytes, world, ms_per_step)

    kernels = {} if args.no_kernels else kernel_timings(st, hbm_peak, sm_max_mhz)
    # the same workload with the 16-bit dither stream (half the generator work), timed beside the default
    alt = None
    if not args.no_kernels and args.dither_bits == 32:
        import dq_workloads as wl
        cfg16 = wl.with_dither_bits(make_workload(args, rank), 16)
        st16 = GpuState(dq, torch, cfg16, dev, share=st)
        for _ in range(3):
            st16.step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            st16.step()
        e1.record()
        torch.cuda.synchronize()
        ms16 = max_over_ranks([e0.elapsed_time(e1) / args.steps], dev)[0]
        alt = {"ms_per_step": ms16, "value": whole_job_value(step_bytes, world, ms16), "unit": "GB/s",
               "kernels": kernel_timings(st16, hbm_peak, sm_max_mhz)}
        del st16
    e2e = None
    if not args.no_e2e:
        dt, h2d, d2h, _ = run_e2e(st, max(1, min(args.steps, 3)))
        dt = max_over_ranks([dt], dev)[0]
        e2e = {"value": world * step_bytes / dt / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": dt * 1e3}

    if rank == 0:
        n_enc = cfg.W
        enc_share = enc_ms / (enc_ms + dec_ms)
        roofline_encode = None
        if kernels:
            # the dominant kernel = the one with the largest share of the step's device time
            enc_names = [k for k in kernels if k.startswith("encode")]
            count = {k: sum(1 for s in cfg.workers if k == f"encode_{'dqsg' if s.kind == 0 else 'ndqsg'}_b{s.bits}")
                     for k in enc_names}
            dom_enc = max(enc_names, key=lambda k: count[k] * kernels[k]["ms"])
            ke, kd = kernels[dom_enc], kernels["decode_aggregate"]
            roofline_encode = {"kernel": dom_enc, "bound": "hbm", "achieved": ke["gbs"], "peak": hbm_peak,
                               "unit": "GB/s", "frac": ke["gbs"] / hbm_peak, "traffic": ke["traffic"],
                               "peak_source": f"of {peak_src}", "frac_of_nominal_8TBs": ke["gbs"] / HBM_NOMINAL_GBS,
                               "launches_per_step": count[dom_enc], "frac_alu": ke["frac_alu"]}
            roofline_decode = {"kernel": "decode_aggregate", "bound": "alu", "achieved": kd["alu_tinstr_s"],
                               "peak": kd["alu_peak_tinstr_s"], "unit": "Tlane-instr/s", "frac": kd["frac_alu"],
                               "traffic": kd["traffic"],
                               "peak_source": "148 SMs x 4 schedulers x 32 lanes x max SM clock",
                               "hbm_gbs": kd["gbs"], "frac_hbm": kd["frac_hbm"], "launches_per_step": 1}
            mix = DEC_MIX.get(cfg.workers[0].dither_bits)
            if mix and cfg.name == "ndqsg_resnet50":
                wide, fp32, other = mix
                cycles = (ISSUE_CYCLES_WIDE * wide + ISSUE_CYCLES_FP32 * fp32 +
                          ISSUE_CYCLES_OTHER * max(0.0, other - wide))
                ceiling = SM_COUNT * ISSUE_PER_SM_CLK * LANES * sm_max_mhz * 1e6 / cycles
                roofline_decode["issue_mix"] = {"wide_mul_per_unit": wide, "fp32_instr_per_unit": fp32,
                                                "other_instr_per_unit": other, "scheduler_cycles_per_unit": cycles,
                                                "ceiling_gelem_worker_s": ceiling / 1e9,
                                                "frac_of_ceiling": kd["gelem_worker_s"] * 1e9 / ceiling}
            if kd["ms"] >= count[dom_enc] * ke["ms"]:
                roofline = roofline_decode
            else:
                roofline, roofline_encode = roofline_encode, None
        else:
            avg_enc_ms = enc_ms / n_enc
            gbs = enc_bytes / n_enc / avg_enc_ms / 1e6
            roofline = {"kernel": "encode (in-step average)", "bound": "hbm", "achieved": gbs, "peak": hbm_peak,
                        "unit": "GB/s", "frac": gbs / hbm_peak, "traffic": None, "peak_source": f"of {peak_src}"}
            roofline_decode = None
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(cfg, args),
            "gelem_s": world * cfg.n / ms_per_step / 1e6,
            "pct_hbm_measured": 100.0 * value / world / hbm_peak, "pct_hbm_nominal": 100.0 * value / world / HBM_NOMINAL_GBS,
            "phases": {"encode_ms": enc_ms, "decode_ms": dec_ms, "encode_share": enc_share,
                       "encode_gbs": enc_bytes / enc_ms / 1e6, "decode_gbs": dec_bytes / dec_ms / 1e6,
                       "encode_bytes": enc_bytes, "decode_bytes": dec_bytes},
            "roofline": roofline, "kernels": kernels, "clocks": clocks, "gpu_launches": launches,
        }
        if roofline_encode is not None:
            line["roofline_encode"] = roofline_encode
        if roofline_decode is not None and roofline_decode is not roofline:
            line["roofline_decode"] = roofline_decode
        if alt is not None:
            line["dither16"] = alt
        if e2e:
            line["e2e"] = e2e
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(cfg, args.cpu_sample)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
