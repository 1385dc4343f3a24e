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
SM_COUNT, ISSUE_PER_SM_CLK, LANES = 148, 4, 32           # issue ceiling: SMs x schedulers x lanes x clock
# Algorithmic lane-instructions of the method itself: a quarter of a Philox block per dither value (4.5 wide
# multiplies + 4.75 three-input XORs), the dither conversion (2), and for the fused decode unpacking (3) plus 5
# (DQSG) to 9 (NDQSG) fp32 operations per (element, worker), about 10 per element for the mean and the stores;
# for the encode 24 per element with the scale reduction and the packing.
DEC_INSTR_PER_ELEM_WORKER, DEC_INSTR_PER_ELEM, ENC_INSTR_PER_ELEM = 22.0, 10.0, 24.0
FLAG_INPUT_READY, FLAG_OUTPUT_FREE = 1, 2


def source_hash():
    from paper_1904_01197_b200 import build as dq_build
    return dq_build.source_hash()


def committed_counters():
    """Counters taken from committed profiler summaries (profiles/counters_*.md): lines of the form
    `counter: <name> <value> csrc=<hash>`.  A counter is returned only if the library's sources still have the
    content hash it was captured at; otherwise the kernel has changed and the value is unknown (None)."""
    out, now = {}, source_hash()
    for f in sorted((ROOT / "profiles").glob("counters_*.md")):
        for line in f.read_text().splitlines():
            parts = line.strip().split()
            if len(parts) >= 4 and parts[0] == "counter:" and parts[3].startswith("csrc="):
                out[parts[1]] = float(parts[2]) if parts[3] == f"csrc={now}" else None
    return out


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
    ap.add_argument("--no-other", action="store_true", help="skip the compact record of the other workloads")
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
        mk = lambda s, flags=0: dq.binding.make_params(cfg.bucket, s.bits, s.levels, s.coarse_K, s.fine_M, s.alpha,
                                                       s.dither_bits, flags)
        self.params = [mk(s) for s in cfg.workers]
        # Inside a step the gradients are complete long before the encodes start, and the encode of worker w
        # writes buffers that the encode of worker w - 1 does not touch: every encode may read early, and all but
        # the first (whose message buffer the previous step's decode may still be reading) may also store early.
        self.step_params = [mk(s, FLAG_INPUT_READY | (FLAG_OUTPUT_FREE if w > 0 else 0))
                            for w, s in enumerate(cfg.workers)]
        self.overlap_params = [mk(s, FLAG_INPUT_READY | FLAG_OUTPUT_FREE) for s in cfg.workers]
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

    def encode(self, w, grad=None, bufs=None, params=None):
        s, p = self.cfg.workers[w], (self.params[w] if params is None else params)
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

    def decode_side_first(self, msgs=None, out=None):
        self.dq.ndqsg_decode_aggregate_side_first(self.msgs if msgs is None else msgs, self.cfg.n, self.cfg.step,
                                                  self.out if out is None else out)

    def step(self, ev_mid=None, two_call=False, plain_launches=False):
        """One pass of the whole path.  When the side information is worker 0's reconstruction it is taken
        inside the fused decode (one launch); two_call=True runs the W=1 decode and the fused decode with a side
        information vector instead.  plain_launches=True encodes without the early-read / early-store flags."""
        for w in range(self.cfg.W):
            self.encode(w, params=None if plain_launches else self.step_params[w])
        if ev_mid is not None:
            ev_mid.record()
        if self.cfg.side_from_worker0 and not two_call:
            self.decode_side_first()
        else:
            if self.cfg.side_from_worker0:
                self.side_decode()
            self.decode()

    def step_bytes(self, two_call=False):
        cfg, dq = self.cfg, self.dq
        enc = sum(encode_bytes(dq, cfg.n, s, cfg.bucket) for s in cfg.workers)
        if cfg.side_from_worker0 and not two_call:
            return enc, decode_bytes(dq, cfg.n, cfg.workers, cfg.bucket, False)
        dec = decode_bytes(dq, cfg.n, cfg.workers, cfg.bucket, self.any_nested)
        if cfg.side_from_worker0:
            dec += decode_bytes(dq, cfg.n, cfg.workers[:1], cfg.bucket, False)
        return enc, dec


def time_isolated(torch, launches, iters=24, warm=3, repeats=3):
    """Average duration (ms) of the launches in `launches` (callables on rotating buffers) between two CUDA
    events; the median of `repeats` such averages."""
    for i in range(warm):
        launches[i % len(launches)]()
    torch.cuda.synchronize()
    avgs = []
    for _ in range(repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            launches[i % len(launches)]()
        e1.record()
        torch.cuda.synchronize()
        avgs.append(e0.elapsed_time(e1) / iters)
    return statistics.median(avgs)


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
    rot = max(2, min(cfg.W, -(-3 * L2_BYTES // (4 * n))))
    counters = committed_counters()
    for key, w in seen.items():
        s = cfg.workers[w]
        by = encode_bytes(dq, n, s, cfg.bucket)
        name = f"encode_{'dqsg' if s.kind == st.DQSG else 'ndqsg'}_b{s.bits}"
        # rotating inputs AND outputs: consecutive launches share nothing, as the overlapped variant requires
        outs = [dq.binding.alloc_message(n, st.params[w], st.dev) for _ in range(rot)]
        for variant, params in (("", st.params[w]), ("_overlapped", st.overlap_params[w])):
            launches = [(lambda gg=st.grads[(w + r) % cfg.W], ww=w, oo=outs[r], pp=params:
                         st.encode(ww, grad=gg, bufs=oo, params=pp)) for r in range(rot)]
            ms = time_isolated(torch, launches)
            res[name + variant] = {
                "ms": ms, "bytes": by, "gbs": by / ms / 1e6, "gelem_s": n / ms / 1e6,
                "frac_hbm": by / ms / 1e6 / hbm_peak, "rotating_buffers": rot,
                "launch_flags": ("DQ_FLAG_INPUT_READY|DQ_FLAG_OUTPUT_FREE: back-to-back launches overlap"
                                 if variant else "none: each launch waits for the previous one"),
                "alu_tinstr_s": ENC_INSTR_PER_ELEM * n / ms / 1e9,
                "frac_alu": ENC_INSTR_PER_ELEM * n / ms * 1e3 / alu_peak,
                "traffic": counters.get(f"{cfg.name}.{name}.dram_bytes") if s.dither_bits == 32 else None}
        del outs
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

    def entry(ms_, by_, workers):
        return {"ms": ms_, "bytes": by_, "gbs": by_ / ms_ / 1e6, "gelem_s": n / ms_ / 1e6,
                "frac_hbm": by_ / ms_ / 1e6 / hbm_peak, "gelem_worker_s": n * workers / ms_ / 1e6}

    if cfg.side_from_worker0:
        # the side information taken from message 0 inside the fused pass (no vector read, no W = 1 launch)
        sf_l = [(lambda a=msg_sets[i], c=outs[i]: st.decode_side_first(a, c)) for i in range(sets)]
        res["decode_aggregate_side_first"] = entry(time_isolated(torch, sf_l, iters=12), per_set - 4 * n, cfg.W)
    # the first message alone (W = 1): the P1 decode of Algorithm 2, and the small-W end of the decoder
    by_w1 = decode_bytes(dq, n, cfg.workers[:1], cfg.bucket, cfg.workers[0].kind != st.DQSG)
    w1_sets = max(2, min(8, -(-3 * L2_BYTES // by_w1)))
    w1_outs = [torch.empty_like(st.out) for _ in range(max(0, w1_sets - sets))] + outs
    w1_l = [(lambda a=msg_sets[i % sets][:1], b=sides[i % sets], c=w1_outs[i]:
             (dq.ndqsg_decode_aggregate(a, n, cfg.step, b, c) if cfg.workers[0].kind != st.DQSG
              else dq.dqsg_decode_aggregate(a, n, cfg.step, c))) for i in range(w1_sets)]
    res["decode_aggregate_w1"] = entry(time_isolated(torch, w1_l, iters=16), by_w1, 1)
    del w1_outs
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
                               "traffic": (counters.get(f"{cfg.name}.decode_aggregate.dram_bytes")
                                           if cfg.workers[0].dither_bits == 32 else None)}
    return res


def other_workloads(torch, hbm_peak, sm_max_mhz):
    """Compact record of the other workload shapes: the ResNet-18-sized DQSG and the GPT-2-small-sized NDQSG
    configurations, three points of the bandwidth sweep (n = 2^26; W = 2, 8, 32), and the issue probe's
    Philox-only and kernel-mix ceilings.  Gradients are N(0,1) drawn on the device (timing only)."""
    from bench_tools import sweep
    keep = ("encode_us", "encode_gbs", "encode_frac_hbm", "decode_us", "decode_gbs", "decode_frac_hbm",
            "decode_gelem_worker_s")
    pts = {"dqsg_resnet18_b2": dict(n=11_689_512, W=8, bits=2, bucket=2048, kind="dqsg"),
           "ndqsg_gpt2_small": dict(n=124_439_808, W=16, bits=3, bucket=4096, kind="ndqsg"),
           "sweep_n2^26_W2": dict(n=1 << 26, W=2, bits=2, bucket=2048, kind="ndqsg"),
           "sweep_n2^26_W8": dict(n=1 << 26, W=8, bits=2, bucket=2048, kind="ndqsg"),
           "sweep_n2^26_W32": dict(n=1 << 26, W=32, bits=2, bucket=2048, kind="ndqsg")}
    out = {}
    for name, pt in pts.items():
        try:
            r = sweep.run_point(dither_bits=32, hbm_peak=hbm_peak, iters=8, **pt)
            out[name] = dict(pt, **{k: r[k] for k in keep})
        except Exception as e:                       # an out-of-memory point must not lose the line
            out[name] = dict(pt, error=str(e)[:200])
        torch.cuda.empty_cache()
    try:
        from bench_tools import issue_probe
        exe = issue_probe.build()
        probe = {}
        for key in ("wide", "round", "dec_coarse", "enc_coarse"):
            txt = subprocess.run([str(exe), key, "4"], capture_output=True, text=True, timeout=120).stdout
            probe[key + "_cycles"] = float(txt.split("instr")[1].split("cycles/group")[0])
        sched_hz = SM_COUNT * ISSUE_PER_SM_CLK * sm_max_mhz * 1e6
        out["issue_probe"] = dict(
            probe, what=("scheduler cycles per group, 4 warps per scheduler: one 32x32->64 multiply; one Philox "
                         "round; the decoder's / encoder's instruction mix for 16 elements with nothing else"),
            philox_only_gblocks_s=sched_hz * LANES / (9.0 * probe["round_cycles"]) / 1e9,
            decode_mix_ceiling_gelem_worker_s=sched_hz * LANES * 16.0 / probe["dec_coarse_cycles"] / 1e9,
            encode_mix_ceiling_gelem_s=sched_hz * LANES * 16.0 / probe["enc_coarse_cycles"] / 1e9)
    except Exception as e:
        out["issue_probe"] = {"error": str(e)[:200]}
    return out


def run_e2e(st: GpuState, steps: int):
    """The same step through the host-buffer C-ABI calls: pinned host buffers in, pinned host buffers out.
    The W encodes are issued from two host threads, each with its own stream and workspace, so that one call's
    kernel and copy-back run beside the other's copy-in; the fused decode takes its side information from
    message 0 when the workload says so (no side-information vector crosses the bus)."""
    from concurrent.futures import ThreadPoolExecutor
    torch, dq, cfg = st.torch, st.dq, st.cfg
    n = cfg.n
    host_msgs = []
    ws_enc = []
    for w, (s, p) in enumerate(zip(cfg.workers, st.params)):
        pk = torch.empty(max(1, dq.packed_words(n, s.bits)), dtype=torch.int32).pin_memory()
        sc = torch.empty(max(1, dq.num_buckets(n, cfg.bucket)), dtype=torch.float32).pin_memory()
        host_msgs.append(dq.Message(pk, sc, s.seed, w, s.kind, p))
        ws_enc.append(dq.encode_workspace_bytes(n, p))
    side_first = bool(cfg.side_from_worker0)
    has_side = st.any_nested and not side_first
    lanes = 2
    streams = [torch.cuda.Stream(device=st.dev) for _ in range(lanes)]
    ws = [torch.empty(max(max(ws_enc), dq.decode_workspace_bytes(host_msgs, n, has_side)), dtype=torch.uint8,
                      device=st.dev) for _ in range(lanes)]
    side_host = st.side_host if (has_side and st.side_host is not None) else None
    out_host = torch.empty(n, dtype=torch.float32).pin_memory()
    pool = ThreadPoolExecutor(max_workers=lanes)
    dev_index = st.dev.index

    def encode_lane(lane):
        torch.cuda.set_device(dev_index)
        for w in range(lane, cfg.W, lanes):
            s, p, m = cfg.workers[w], st.params[w], host_msgs[w]
            fn = dq.dqsg_encode_host if s.kind == st.DQSG else dq.ndqsg_encode_host
            fn(st.grads_host[w], s.seed, w, cfg.step, p, m.packed, m.scale, ws[lane], stream=streams[lane])

    def one():
        list(pool.map(encode_lane, range(lanes)))
        if side_first:
            dq.ndqsg_decode_aggregate_side_first_host(host_msgs, n, cfg.step, out_host, ws[0], stream=streams[0])
        else:
            dq.ndqsg_decode_aggregate_host(host_msgs, n, cfg.step, side_host, out_host, ws[0], stream=streams[0])

    msg_bytes = sum(4 * dq.packed_words(n, s.bits) + 4 * dq.num_buckets(n, cfg.bucket) for s in cfg.workers)
    h2d = 4 * n * cfg.W + msg_bytes + (4 * n if has_side else 0)
    d2h = msg_bytes + 4 * n
    one()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / steps
    pool.shutdown()
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

    # the step as two decode calls (W = 1 pass writes the side information, the fused pass reads it) and with
    # plain launches: the form without the fused side information and without the launch flags
    variants = None
    if not args.profile and cfg.side_from_worker0:
        for _ in range(3):
            st.step(two_call=True, plain_launches=True)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            st.step(two_call=True, plain_launches=True)
        e1.record()
        torch.cuda.synchronize()
        ms2 = max_over_ranks([e0.elapsed_time(e1) / args.steps], dev)[0]
        by2 = sum(st.step_bytes(two_call=True))
        variants = {"two_decode_calls_plain_launches": {"ms_per_step": ms2, "bytes": by2,
                                                        "value": whole_job_value(by2, world, ms2), "unit": "GB/s",
                                                        "launches_per_step": cfg.W + 2}}
    other = None
    if rank == 0 and not args.no_kernels and not args.no_other and args.workload == "ndqsg_resnet50":
        del st.msg_buf, st.msgs
        torch.cuda.empty_cache()
        other = other_workloads(torch, hbm_peak, sm_max_mhz)

    if rank == 0:
        n_enc = cfg.W
        enc_share = enc_ms / (enc_ms + dec_ms)
        roofline_encode = None
        if kernels:
            enc_names = [k for k in kernels if k.startswith("encode") and not k.endswith("_overlapped")]
            count = {k: sum(1 for s in cfg.workers if k == f"encode_{'dqsg' if s.kind == 0 else 'ndqsg'}_b{s.bits}")
                     for k in enc_names}
            dom_enc = max(enc_names, key=lambda k: count[k] * kernels[k]["ms"])
            # encode: the launch as the step issues it (inputs ready, outputs free: launches overlap)
            ke, ke_plain = kernels[dom_enc + "_overlapped"], kernels[dom_enc]
            dec_name = "decode_aggregate_side_first" if cfg.side_from_worker0 else "decode_aggregate"
            kd = kernels[dec_name]
            roofline_encode = {"kernel": dom_enc, "bound": "hbm", "achieved": ke["gbs"], "peak": hbm_peak,
                               "unit": "GB/s", "frac": ke["gbs"] / hbm_peak, "traffic": ke["traffic"],
                               "peak_source": f"of {peak_src}", "frac_of_nominal_8TBs": ke["gbs"] / HBM_NOMINAL_GBS,
                               "launches_per_step": count[dom_enc], "launch_flags": ke["launch_flags"],
                               "us_per_launch": ke["ms"] * 1e3,
                               "without_flags": {"achieved": ke_plain["gbs"], "frac": ke_plain["frac_hbm"],
                                                 "us_per_launch": ke_plain["ms"] * 1e3}}
            # decode: bound by instruction issue; algorithmic lane-instructions against the issue ceiling, and the
            # multiplier pipe beside it (a 32x32->64 multiply holds it for four cycles, 4.5 of them per dither value)
            alu_peak = SM_COUNT * ISSUE_PER_SM_CLK * LANES * sm_max_mhz * 1e6
            alg_instr = DEC_INSTR_PER_ELEM_WORKER * cfg.n * cfg.W + DEC_INSTR_PER_ELEM * cfg.n
            cyc_per_unit = SM_COUNT * ISSUE_PER_SM_CLK * LANES * sm_max_mhz * 1e6 / (kd["gelem_worker_s"] * 1e9)
            dith = cfg.workers[0].dither_bits
            wide_per_unit = 18.0 / (4 if dith == 32 else 8)
            roofline_decode = {"kernel": dec_name, "bound": "alu", "achieved": alg_instr / kd["ms"] / 1e9,
                               "peak": alu_peak / 1e12, "unit": "Tlane-instr/s",
                               "frac": alg_instr / kd["ms"] * 1e3 / alu_peak,
                               "traffic": (committed_counters().get(f"{cfg.name}.{dec_name}.dram_bytes")
                                           if dith == 32 else None),
                               "peak_source": "148 SMs x 4 schedulers x 32 lanes x max SM clock",
                               "hbm_gbs": kd["gbs"], "frac_hbm": kd["frac_hbm"], "launches_per_step": 1,
                               "gelem_worker_s": kd["gelem_worker_s"],
                               "scheduler_cycles_per_element_worker": cyc_per_unit,
                               "multiplier_pipe": {"wide_multiplies_per_element_worker": wide_per_unit,
                                                   "pipe_cycles_per_wide_multiply": 4.0,
                                                   "floor_cycles_per_element_worker": 4.0 * wide_per_unit,
                                                   "frac": 4.0 * wide_per_unit / cyc_per_unit}}
            probe = (other or {}).get("issue_probe", {})
            if dith == 32 and "decode_mix_ceiling_gelem_worker_s" in probe:
                # what the decoder's arithmetic alone (nine rounds for four blocks, then 16 NDQSG elements) reaches
                # on this GPU, measured in this run by bench_tools/issue_probe
                roofline_decode["measured_mix_ceiling"] = {
                    "gelem_worker_s": probe["decode_mix_ceiling_gelem_worker_s"],
                    "frac": kd["gelem_worker_s"] / probe["decode_mix_ceiling_gelem_worker_s"]}
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
        if variants is not None:
            line["step_variants"] = variants
        if other is not None:
            line["other_workloads"] = other
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
