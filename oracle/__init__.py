"""ctypes front end of the CPU oracle (``dq_oracle.c``).

TEST INFRASTRUCTURE.  Only ``tests/``, the smoke check and the benchmark's
CPU-baseline leg import this package.  The CUDA library and its Python binding
never do, and nothing here touches the CUDA library.

``build()`` compiles the C file with gcc (``-O2 -ffp-contract=off -fopenmp``)
into ``oracle/_build/``; it is called on first use.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path
from typing import List, Optional, Sequence

import numpy as np

_HERE = Path(__file__).resolve().parent
# DQ_ORACLE_SOURCE / DQ_ORACLE_LIBRARY let the mutation test point a subprocess at a deliberately broken copy of
# the C file (to check that the pins notice); nothing else sets them.
_SRC = Path(os.environ.get("DQ_ORACLE_SOURCE", _HERE / "dq_oracle.c"))
_OUT = Path(os.environ.get("DQ_ORACLE_LIBRARY", _HERE / "_build" / "libdq_oracle.so"))

KIND_DQSG = 0
KIND_NDQSG = 1


def build(force: bool = False) -> Path:
    if force or not _OUT.exists() or _OUT.stat().st_mtime < _SRC.stat().st_mtime:
        _OUT.parent.mkdir(parents=True, exist_ok=True)
        tmp = _OUT.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC",
               "-shared", "-Wall", "-Wextra", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _OUT)
    return _OUT


class _Msg(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("bucket", C.c_uint32), ("bits", C.c_uint32),
                ("levels", C.c_uint32), ("coarse_K", C.c_uint32), ("fine_M", C.c_float),
                ("alpha", C.c_float), ("worker", C.c_uint32), ("dither_bits", C.c_uint32),
                ("reserved", C.c_uint32), ("seed", C.c_uint64),
                ("packed", C.c_void_p), ("scale", C.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(str(build()))
        u32p, f32p, i32p = C.POINTER(C.c_uint32), C.POINTER(C.c_float), C.POINTER(C.c_int32)
        L.dqo_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.dqo_philox4x32_10.restype = None
        L.dqo_dither_bits.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64]
        L.dqo_dither_bits.restype = C.c_uint32
        L.dqo_dither_from_bits.argtypes = [C.c_uint32]
        L.dqo_dither_from_bits.restype = C.c_float
        L.dqo_dither.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64]
        L.dqo_dither.restype = C.c_float
        L.dqo_dither16_half.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64]
        L.dqo_dither16_half.restype = C.c_uint32
        L.dqo_dither16_from_half.argtypes = [C.c_uint32]
        L.dqo_dither16_from_half.restype = C.c_float
        L.dqo_dither_stream.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint32]
        L.dqo_dither_stream.restype = C.c_float
        for name, nargs in (("dqo_Q", 2), ("dqo_dithered", 3), ("dqo_nested_encode_scalar", 5),
                            ("dqo_nested_decode_scalar", 5)):
            f = getattr(L, name)
            f.argtypes = [C.c_double] * nargs
            f.restype = C.c_double
        L.dqo_raw_bits.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
        L.dqo_raw_bits.restype = C.c_double
        L.dqo_packed_words.argtypes = [C.c_uint64, C.c_uint32]
        L.dqo_packed_words.restype = C.c_uint64
        L.dqo_num_buckets.argtypes = [C.c_uint64, C.c_uint32]
        L.dqo_num_buckets.restype = C.c_uint64
        L.dqo_default_levels.argtypes = [C.c_uint32]
        L.dqo_default_levels.restype = C.c_uint32
        L.dqo_pack.argtypes = [u32p, C.c_uint64, C.c_uint32, u32p]
        L.dqo_pack.restype = None
        L.dqo_unpack.argtypes = [u32p, C.c_uint64, C.c_uint32, u32p]
        L.dqo_unpack.restype = None
        L.dqo_ternary_bytes.argtypes = [C.c_uint64]
        L.dqo_ternary_bytes.restype = C.c_uint64
        L.dqo_ternary_pack.argtypes = [u32p, C.c_uint64, C.POINTER(C.c_uint8)]
        L.dqo_ternary_pack.restype = None
        L.dqo_ternary_unpack.argtypes = [C.POINTER(C.c_uint8), C.c_uint64, u32p]
        L.dqo_ternary_unpack.restype = None
        L.dqo_dqsg_encode.argtypes = [f32p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64,
                                      C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, u32p, f32p, i32p, C.c_int]
        L.dqo_dqsg_encode.restype = C.c_int
        L.dqo_ndqsg_encode.argtypes = [f32p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint64,
                                       C.c_uint32, C.c_uint32, C.c_uint32, C.c_float, C.c_float, C.c_uint32,
                                       u32p, f32p, i32p, C.c_int]
        L.dqo_ndqsg_encode.restype = C.c_int
        L.dqo_decode_aggregate.argtypes = [C.POINTER(_Msg), C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64,
                                           f32p, f32p, f32p, i32p, C.c_int]
        L.dqo_decode_aggregate.restype = C.c_int
        L.dqo_decode_aggregate_running.argtypes = [C.POINTER(_Msg), C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64,
                                                   f32p, f32p, i32p, C.c_int]
        L.dqo_decode_aggregate_running.restype = C.c_int
        L.dqo_nearest_coset_bruteforce.argtypes = [C.c_uint32, C.c_int32, C.c_double, C.c_double,
                                                   C.c_double, C.c_int32, C.POINTER(C.c_double)]
        L.dqo_nearest_coset_bruteforce.restype = C.c_int32
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray], ty):
    return None if a is None else a.ctypes.data_as(C.POINTER(ty))


# ---------------------------------------------------------------- scalars
def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> List[int]:
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().dqo_philox4x32_10(c, k, o)
    return list(o)


def dither_bits(seed: int, worker: int, step: int, i: int) -> int:
    return int(lib().dqo_dither_bits(seed, worker, step, i))


def dither_from_bits(x: int) -> float:
    return float(lib().dqo_dither_from_bits(x))


def dither(seed: int, worker: int, step: int, i: int) -> float:
    return float(lib().dqo_dither(seed, worker, step, i))


def dither_vector(seed: int, worker: int, step: int, n: int, i0: int = 0, dither_bits: int = 32) -> np.ndarray:
    L = lib()
    return np.array([L.dqo_dither_stream(seed, worker, step, i0 + i, dither_bits) for i in range(n)],
                    dtype=np.float32)


def dither16_half(seed: int, worker: int, step: int, i: int) -> int:
    return int(lib().dqo_dither16_half(seed, worker, step, i))


def dither16_from_half(h: int) -> float:
    return float(lib().dqo_dither16_from_half(h))


def Q(v: float, Delta: float) -> float:
    return float(lib().dqo_Q(v, Delta))


def dithered(x: float, u: float, Delta: float) -> float:
    return float(lib().dqo_dithered(x, u, Delta))


def nested_encode_scalar(x, u, Delta1, Delta2, alpha) -> float:
    return float(lib().dqo_nested_encode_scalar(x, u, Delta1, Delta2, alpha))


def nested_decode_scalar(s, u, y, Delta2, alpha) -> float:
    return float(lib().dqo_nested_decode_scalar(s, u, y, Delta2, alpha))


def raw_bits(n: int, levels: int, partitions: int) -> float:
    return float(lib().dqo_raw_bits(n, levels, partitions))


def packed_words(n: int, bits: int) -> int:
    return int(lib().dqo_packed_words(n, bits))


def num_buckets(n: int, bucket: int) -> int:
    return int(lib().dqo_num_buckets(n, bucket))


def default_levels(bits: int) -> int:
    return int(lib().dqo_default_levels(bits))


# ---------------------------------------------------------------- vectors
def pack(code: np.ndarray, bits: int) -> np.ndarray:
    code = np.ascontiguousarray(code, dtype=np.uint32)
    out = np.zeros(packed_words(code.size, bits), dtype=np.uint32)
    lib().dqo_pack(_p(code, C.c_uint32), code.size, bits, _p(out, C.c_uint32))
    return out


def unpack(words: np.ndarray, n: int, bits: int) -> np.ndarray:
    words = np.ascontiguousarray(words, dtype=np.uint32)
    out = np.zeros(n, dtype=np.uint32)
    lib().dqo_unpack(_p(words, C.c_uint32), n, bits, _p(out, C.c_uint32))
    return out


def ternary_bytes(n: int) -> int:
    return int(lib().dqo_ternary_bytes(n))


def ternary_pack(code: np.ndarray) -> np.ndarray:
    """Five ternary codes per byte (radix-3 container of a three-level message)."""
    code = np.ascontiguousarray(code, dtype=np.uint32)
    out = np.zeros(ternary_bytes(code.size), dtype=np.uint8)
    lib().dqo_ternary_pack(_p(code, C.c_uint32), code.size, _p(out, C.c_uint8))
    return out


def ternary_unpack(data: np.ndarray, n: int) -> np.ndarray:
    data = np.ascontiguousarray(data, dtype=np.uint8)
    assert data.size >= ternary_bytes(n)
    out = np.zeros(n, dtype=np.uint32)
    lib().dqo_ternary_unpack(_p(data, C.c_uint8), n, _p(out, C.c_uint32))
    return out


def ternary_pack_stream(words: np.ndarray, n: int) -> np.ndarray:
    """The radix-3 container of a 2-bit packed three-level message."""
    return ternary_pack(unpack(words, n, 2))


def ternary_unpack_stream(data: np.ndarray, n: int) -> np.ndarray:
    """Back to the 2-bit packed stream."""
    return pack(ternary_unpack(data, n), 2)


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what}: bad argument (rc={rc})")


def dqsg_encode(g: np.ndarray, seed: int, worker: int, step: int, bucket: int, bits: int,
                levels: int = 0, i0: int = 0, want_codes: bool = False, threads: int = 1, dither_bits: int = 32):
    """Returns (packed uint32[NW], scale fp32[NB][, code int32[n]])."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    n = g.size
    packed = np.zeros(max(1, packed_words(n, bits)), dtype=np.uint32)
    scale = np.zeros(max(1, num_buckets(n, bucket)), dtype=np.float32)
    codes = np.zeros(max(1, n), dtype=np.int32) if want_codes else None
    _check(lib().dqo_dqsg_encode(_p(g, C.c_float), n, i0, seed, worker, step, bucket, bits, levels, dither_bits,
                                 _p(packed, C.c_uint32), _p(scale, C.c_float), _p(codes, C.c_int32),
                                 threads), "dqsg_encode")
    packed, scale = packed[:packed_words(n, bits)], scale[:num_buckets(n, bucket)]
    return (packed, scale, codes[:n]) if want_codes else (packed, scale)


def ndqsg_encode(g: np.ndarray, seed: int, worker: int, step: int, bucket: int, bits: int,
                 coarse_K: int, fine_M: float, alpha: float = 1.0, i0: int = 0,
                 want_q1: bool = False, threads: int = 1, dither_bits: int = 32):
    """Returns (packed uint32[NW], scale fp32[NB][, q1 int32[n]])."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    n = g.size
    packed = np.zeros(max(1, packed_words(n, bits)), dtype=np.uint32)
    scale = np.zeros(max(1, num_buckets(n, bucket)), dtype=np.float32)
    q1 = np.zeros(max(1, n), dtype=np.int32) if want_q1 else None
    _check(lib().dqo_ndqsg_encode(_p(g, C.c_float), n, i0, seed, worker, step, bucket, bits, coarse_K,
                                  fine_M, alpha, dither_bits, _p(packed, C.c_uint32), _p(scale, C.c_float),
                                  _p(q1, C.c_int32), threads), "ndqsg_encode")
    packed, scale = packed[:packed_words(n, bits)], scale[:num_buckets(n, bucket)]
    return (packed, scale, q1[:n]) if want_q1 else (packed, scale)


class Msg:
    """One worker's message plus the quantizer settings the decoder needs."""

    def __init__(self, packed: np.ndarray, scale: np.ndarray, seed: int, worker: int, kind: int,
                 bucket: int, bits: int, levels: int = 0, coarse_K: int = 0, fine_M: float = 0.0,
                 alpha: float = 1.0, dither_bits: int = 32):
        self.packed = np.ascontiguousarray(packed, dtype=np.uint32)
        self.scale = np.ascontiguousarray(scale, dtype=np.float32)
        self.seed, self.worker, self.kind = seed, worker, kind
        self.bucket, self.bits, self.levels = bucket, bits, levels
        self.coarse_K, self.fine_M, self.alpha = coarse_K, fine_M, alpha
        self.dither_bits = dither_bits


def decode_aggregate(msgs: Sequence[Msg], n: int, step: int, side_info: Optional[np.ndarray] = None,
                     i0: int = 0, want_recon: bool = False, want_qhat: bool = False, threads: int = 1,
                     running: bool = False):
    """Returns out_avg fp32[n] (plus recon fp32[W][n] and/or qhat int32[W][n] when asked).
    running=True: Algorithm 2's server loop, side information = mean of everything decoded before."""
    W = len(msgs)
    arr = (_Msg * max(1, W))()
    for w, m in enumerate(msgs):
        arr[w] = _Msg(m.kind, m.bucket, m.bits, m.levels, m.coarse_K, m.fine_M, m.alpha, m.worker,
                      m.dither_bits, 0, m.seed, m.packed.ctypes.data, m.scale.ctypes.data)
    if side_info is not None:
        side_info = np.ascontiguousarray(side_info, dtype=np.float32)
        assert side_info.size >= n
    out = np.zeros(max(1, n), dtype=np.float32)
    recon = np.zeros((max(1, W), max(1, n)), dtype=np.float32) if want_recon else None
    qhat = np.zeros((max(1, W), max(1, n)), dtype=np.int32) if want_qhat else None
    if running:
        _check(lib().dqo_decode_aggregate_running(arr, W, n, i0, step, _p(out, C.c_float),
                                                  _p(recon, C.c_float), _p(qhat, C.c_int32), threads),
               "decode_aggregate_running")
    else:
        _check(lib().dqo_decode_aggregate(arr, W, n, i0, step, _p(side_info, C.c_float), _p(out, C.c_float),
                                          _p(recon, C.c_float), _p(qhat, C.c_int32), threads),
               "decode_aggregate")
    res = [out[:n]]
    if want_recon:
        res.append(recon[:, :n])
    if want_qhat:
        res.append(qhat[:, :n])
    return res[0] if len(res) == 1 else tuple(res)


def nearest_coset_bruteforce(m: int, K: int, a: float, delta: float, y: float, T: int = 64):
    margin = C.c_double()
    q = lib().dqo_nearest_coset_bruteforce(m, K, a, delta, y, T, C.byref(margin))
    return int(q), float(margin.value)
