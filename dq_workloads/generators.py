"""Seeded generators for the synthetic gradients the tests and the benchmark use.

Every workload stands in for gradients of a real network (the paper trains
MNIST / CIFAR-10 models; no dataset is used here).  Shapes, value
distributions and the worker-to-worker correlation follow the recipe written
next to each function.  All draws come from ``numpy.random.Generator(PCG64)``
streams derived from ``SeedSequence([seed, tag, worker])`` so any worker's
vector can be produced on its own, in any order, on any machine.

Nothing here quantizes, dithers, packs or decodes anything.
"""
from __future__ import annotations

import functools
from dataclasses import dataclass, field
from typing import Callable, List, Optional

import numpy as np

DQSG = 0
NDQSG = 1


@dataclass(frozen=True)
class WorkerSpec:
    """Quantizer settings of one worker (plain data, no arithmetic)."""

    kind: int                 # DQSG or NDQSG
    bits: int                 # b bits per element on the wire
    levels: int = 0           # DQSG level count L (0: library default for b)
    coarse_K: int = 0         # NDQSG coarse/fine ratio K
    fine_M: float = 0.0       # NDQSG 1/Delta_1 in normalised units
    alpha: float = 1.0        # NDQSG shrinkage
    seed: int = 0             # dither seed shared with the decoder
    dither_bits: int = 32     # random bits per dither value (32 or 16)


@dataclass
class Workload:
    name: str
    n: int                    # elements per gradient
    W: int                    # workers
    bucket: int               # bucket length B
    workers: List[WorkerSpec]
    grad: Callable[[int], np.ndarray]                 # worker index -> fp32[n]
    side_info: Optional[Callable[[], np.ndarray]]     # explicit side information, or None
    side_from_worker0: bool = False                   # side info = decode of worker 0's message
    step: int = 1
    notes: str = ""
    meta: dict = field(default_factory=dict)


def _rng(seed: int, tag: int, worker: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, tag, worker])))


def _normal32(rng: np.random.Generator, n: int, chunk: int = 1 << 24) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)
    for a in range(0, n, chunk):
        b = min(n, a + chunk)
        out[a:b] = rng.standard_normal(b - a, dtype=np.float32)
    return out


def default_levels(bits: int) -> int:
    return 2 if bits == 1 else (1 << bits) - 1


def worker_seed(seed: int, w: int) -> int:
    """A distinct 64-bit dither seed per worker (a fixed odd multiplier; not part of the method)."""
    return (0x9E3779B97F4A7C15 * (w + 1) + seed) & 0xFFFFFFFFFFFFFFFF


# --------------------------------------------------------------------------
# config 1: tiny
# --------------------------------------------------------------------------
def tiny(n: int = 65536, W: int = 2, bucket: int = 512, seed: int = 0, bits: int = 2,
         kind: str = "mixed") -> Workload:
    """c, n_w ~ N(0, 1e-2) iid; g_w = c + 0.3 n_w; side information y = c.

    kind: "dqsg" (all workers b-bit DQSG), "ndqsg" (all NDQSG, K = M1 = 2^b), or
    "mixed" (worker 0 DQSG, the rest NDQSG).
    """
    @functools.lru_cache(maxsize=1)
    def common():
        return (0.1 * _normal32(_rng(seed, 1), n)).astype(np.float32)

    def grad(w):
        nw = 0.1 * _normal32(_rng(seed, 2, w), n)
        return (common() + np.float32(0.3) * nw).astype(np.float32)

    K = 1 << bits
    workers = []
    for w in range(W):
        nd = (kind == "ndqsg") or (kind == "mixed" and w > 0)
        if nd:
            workers.append(WorkerSpec(NDQSG, bits, 0, K, float(K), 1.0, worker_seed(seed, w)))
        else:
            workers.append(WorkerSpec(DQSG, bits, default_levels(bits), 0, 0.0, 1.0, worker_seed(seed, w)))
    return Workload("tiny", n, W, bucket, workers, grad, common, notes="config 1")


# --------------------------------------------------------------------------
# config 2: DQSG only, ResNet-18-sized, per-layer scales
# --------------------------------------------------------------------------
def _layer_sizes(n: int, layers: int, seed: int) -> np.ndarray:
    r = _rng(seed, 3)
    raw = np.exp(r.uniform(np.log(1e2), np.log(3e6), size=layers))
    sizes = np.maximum(1, np.floor(raw / raw.sum() * n)).astype(np.int64)
    sizes[-1] += n - sizes.sum()
    assert sizes.sum() == n and (sizes > 0).all()
    return sizes


def dqsg_resnet18(n: int = 11_689_512, W: int = 8, bucket: int = 2048, seed: int = 0,
                  bits: int = 2, layers: int = 62) -> Workload:
    """62 'layers' with log-uniform sizes summing to n; sigma_l log-uniform in [1e-4, 1e-1];
    g_w ~ N(0, sigma_l^2) independently per worker."""
    layers = min(layers, max(1, n // 4))
    sizes = _layer_sizes(n, layers, seed)
    sig = np.exp(_rng(seed, 4).uniform(np.log(1e-4), np.log(1e-1), size=layers)).astype(np.float32)
    sigma_vec = np.repeat(sig, sizes)

    def grad(w):
        return (_normal32(_rng(seed, 5, w), n) * sigma_vec).astype(np.float32)

    workers = [WorkerSpec(DQSG, bits, default_levels(bits), 0, 0.0, 1.0, worker_seed(seed, w)) for w in range(W)]
    return Workload("dqsg_resnet18", n, W, bucket, workers, grad, None, notes="config 2",
                    meta={"layers": int(layers)})


# --------------------------------------------------------------------------
# config 3: NDQSG, ResNet-50-sized, correlation 0.9, side info = decode of worker 0
# --------------------------------------------------------------------------
def ndqsg_resnet50(n: int = 25_557_032, W: int = 8, bucket: int = 2048, seed: int = 0) -> Workload:
    """c ~ N(0,1e-4), n_w ~ N(0,1e-4), g_w = c + n_w/3 (pairwise correlation 0.9).
    Worker 0: DQSG with L=5 (M=2, Delta=0.5, 3 bits); workers 1..W-1: NDQSG K=4 (2 bits), M1=2, alpha=1.
    Side information for the NDQSG workers is worker 0's decoded gradient."""
    @functools.lru_cache(maxsize=1)
    def common():
        return (np.float32(1e-2) * _normal32(_rng(seed, 6), n)).astype(np.float32)

    def grad(w):
        nw = np.float32(1e-2) * _normal32(_rng(seed, 7, w), n)
        return (common() + nw / np.float32(3.0)).astype(np.float32)

    workers = [WorkerSpec(DQSG, 3, 5, 0, 0.0, 1.0, worker_seed(seed, 0))]
    workers += [WorkerSpec(NDQSG, 2, 0, 4, 2.0, 1.0, worker_seed(seed, w)) for w in range(1, W)]
    return Workload("ndqsg_resnet50", n, W, bucket, workers, grad, None, side_from_worker0=True,
                    notes="config 3")


# --------------------------------------------------------------------------
# config 4: NDQSG large, GPT-2-small-sized
# --------------------------------------------------------------------------
def ndqsg_gpt2_small(n: int = 124_439_808, W: int = 16, bucket: int = 4096, seed: int = 0) -> Workload:
    """c ~ Laplace(0,1e-3); g_w = c + N(0,(3e-4)^2); y = c + N(0,(1e-4)^2); all NDQSG K=8 (3 bits), M1=16."""
    @functools.lru_cache(maxsize=1)
    def common():
        r = _rng(seed, 8)
        out = np.empty(n, dtype=np.float32)
        chunk = 1 << 24
        for a in range(0, n, chunk):
            b = min(n, a + chunk)
            out[a:b] = r.laplace(0.0, 1e-3, size=b - a).astype(np.float32)
        return out

    def grad(w):
        return (common() + np.float32(3e-4) * _normal32(_rng(seed, 9, w), n)).astype(np.float32)

    def side():
        return (common() + np.float32(1e-4) * _normal32(_rng(seed, 10), n)).astype(np.float32)

    workers = [WorkerSpec(NDQSG, 3, 0, 8, 16.0, 1.0, worker_seed(seed, w)) for w in range(W)]
    return Workload("ndqsg_gpt2_small", n, W, bucket, workers, grad, side, notes="config 4")


# --------------------------------------------------------------------------
# config 5: one point of the bandwidth sweep
# --------------------------------------------------------------------------
def sweep_point(n: int, W: int, bits: int, bucket: int, kind: str = "dqsg", seed: int = 0) -> Workload:
    """N(0,1) gradients; NDQSG uses K = M1 = 2^b and y = g_0 + 0.05 N(0,1)."""
    def grad(w):
        return _normal32(_rng(seed, 11, w), n)

    def side():
        return (grad(0) + np.float32(0.05) * _normal32(_rng(seed, 12), n)).astype(np.float32)

    if kind == "dqsg":
        workers = [WorkerSpec(DQSG, bits, default_levels(bits), 0, 0.0, 1.0, worker_seed(seed, w)) for w in range(W)]
        return Workload("sweep_dqsg", n, W, bucket, workers, grad, None, notes="config 5")
    K = 1 << bits
    workers = [WorkerSpec(NDQSG, bits, 0, K, float(K), 1.0, worker_seed(seed, w)) for w in range(W)]
    return Workload("sweep_ndqsg", n, W, bucket, workers, grad, side, notes="config 5")


WORKLOAD_NAMES = ("tiny", "dqsg_resnet18", "ndqsg_resnet50", "ndqsg_gpt2_small")


def with_dither_bits(cfg: Workload, dither_bits: int) -> Workload:
    """The same workload with every worker switched to the given dither stream."""
    import dataclasses
    cfg.workers = [dataclasses.replace(s, dither_bits=dither_bits) for s in cfg.workers]
    cfg.meta = dict(cfg.meta, dither_bits=dither_bits)
    return cfg


def by_name(name: str, dither_bits: int = 32, **kw) -> Workload:
    cfg = {"tiny": tiny, "dqsg_resnet18": dqsg_resnet18, "ndqsg_resnet50": ndqsg_resnet50,
           "ndqsg_gpt2_small": ndqsg_gpt2_small}[name](**kw)
    return with_dither_bits(cfg, dither_bits) if dither_bits != 32 else cfg
