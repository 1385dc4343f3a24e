"""ctypes binding of ``libdq_b200.so``.  Argument marshalling only.

Tensors are ``torch`` CUDA tensors (device entry points) or CPU tensors / numpy arrays (``*_host`` entry
points); the binding passes their addresses and the current CUDA stream to the C ABI and raises
``DqError`` on a non-zero status.  There is no fallback: if the shared library is missing the import of
``lib()`` fails.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path
from typing import Optional, Sequence

import torch

DQ_KIND_DQSG = 0
DQ_KIND_NDQSG = 1
DQ_WARN_NONFINITE_SCALE = 0x1
DQ_ERR_COPY_TIMEOUT = 0x2
DQ_WARN_CODE_RANGE = 0x4
DQ_FLAG_INPUT_READY = 0x1
DQ_FLAG_OUTPUT_FREE = 0x2
DQ_FLAG_TEST_DROP_COPY = 0x80000000

_LIB_PATH = Path(__file__).resolve().parent / "lib" / "libdq_b200.so"


class DqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status})")


class DqParams(C.Structure):
    _fields_ = [("bucket", C.c_uint32), ("bits", C.c_uint32), ("levels", C.c_uint32),
                ("coarse_K", C.c_uint32), ("fine_M", C.c_float), ("alpha", C.c_float),
                ("dither_bits", C.c_uint32), ("flags", C.c_uint32)]


class DqMsg(C.Structure):
    _fields_ = [("packed", C.c_void_p), ("scale", C.c_void_p), ("seed", C.c_uint64),
                ("worker", C.c_uint32), ("kind", C.c_int), ("p", DqParams)]


_lib = None


def lib() -> C.CDLL:
    """Loads the CUDA library (built by ``paper_1904_01197_b200.build``).  Fails loudly if absent."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_1904_01197_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(str(_LIB_PATH))
        vp, u64, u32 = C.c_void_p, C.c_uint64, C.c_uint32
        pp = C.POINTER(DqParams)
        pm = C.POINTER(DqMsg)
        L.dq_packed_words.argtypes = [u64, u32]; L.dq_packed_words.restype = u64
        L.dq_num_buckets.argtypes = [u64, u32]; L.dq_num_buckets.restype = u64
        L.dq_default_levels.argtypes = [u32]; L.dq_default_levels.restype = u32
        L.dq_status_string.argtypes = [C.c_int]; L.dq_status_string.restype = C.c_char_p
        for f in (L.dqsg_encode, L.ndqsg_encode):
            f.argtypes = [vp, u64, u64, u32, u64, pp, vp, vp, vp]; f.restype = C.c_int
        L.dqsg_decode_aggregate.argtypes = [pm, u32, u64, u64, vp, vp]
        L.dqsg_decode_aggregate.restype = C.c_int
        L.ndqsg_decode_aggregate.argtypes = [pm, u32, u64, u64, vp, vp, vp, vp]
        L.ndqsg_decode_aggregate.restype = C.c_int
        L.dqsg_decode_aggregate_half_dithered.argtypes = [pm, u32, u64, vp, vp]
        L.dqsg_decode_aggregate_half_dithered.restype = C.c_int
        L.ndqsg_decode_aggregate_running.argtypes = [pm, u32, u64, u64, vp, vp, vp]
        L.ndqsg_decode_aggregate_running.restype = C.c_int
        L.ndqsg_decode_aggregate_side_first.argtypes = [pm, u32, u64, u64, vp, vp, vp]
        L.ndqsg_decode_aggregate_side_first.restype = C.c_int
        L.dq_code_histogram.argtypes = [vp, u64, u32, vp, vp]
        L.dq_code_histogram.restype = C.c_int
        L.dq_code_entropy.argtypes = [C.POINTER(C.c_uint64), u32, C.POINTER(C.c_double)]
        L.dq_code_entropy.restype = C.c_int
        for f in (L.dqsg_encode_range, L.ndqsg_encode_range):
            f.argtypes = [vp, u64, u64, u64, u32, u64, pp, vp, vp, vp]; f.restype = C.c_int
        L.ndqsg_decode_aggregate_range.argtypes = [pm, u32, u64, u64, u64, vp, vp, vp, vp]
        L.ndqsg_decode_aggregate_range.restype = C.c_int
        L.dq_ternary_bytes.argtypes = [u64]; L.dq_ternary_bytes.restype = u64
        L.dq_ternary_pack.argtypes = [vp, u64, vp, vp, vp]; L.dq_ternary_pack.restype = C.c_int
        L.dq_ternary_unpack.argtypes = [vp, u64, vp, vp]; L.dq_ternary_unpack.restype = C.c_int
        L.dq_encode_workspace_bytes.argtypes = [u64, pp]; L.dq_encode_workspace_bytes.restype = u64
        L.dq_decode_workspace_bytes.argtypes = [pm, u32, u64, C.c_int]; L.dq_decode_workspace_bytes.restype = u64
        for f in (L.dqsg_encode_host, L.ndqsg_encode_host):
            f.argtypes = [vp, u64, u64, u32, u64, pp, vp, vp, vp, u64, vp]; f.restype = C.c_int
        L.dqsg_encode_host_static.argtypes = [vp, u64, u64, u32, u64, pp, vp, vp, vp]
        L.dqsg_encode_host_static.restype = C.c_int
        L.ndqsg_decode_aggregate_host.argtypes = [pm, u32, u64, u64, vp, vp, vp, u64, vp]
        L.ndqsg_decode_aggregate_host.restype = C.c_int
        L.ndqsg_decode_aggregate_side_first_host.argtypes = [pm, u32, u64, u64, vp, vp, u64, vp]
        L.ndqsg_decode_aggregate_side_first_host.restype = C.c_int
        L.dq_device_error_flags.argtypes = [C.POINTER(u32)]; L.dq_device_error_flags.restype = C.c_int
        L.dq_launch_count.argtypes = []; L.dq_launch_count.restype = u64
        _lib = L
    return _lib


def packed_words(n: int, bits: int) -> int:
    return int(lib().dq_packed_words(n, bits))


def num_buckets(n: int, bucket: int) -> int:
    return int(lib().dq_num_buckets(n, bucket))


def default_levels(bits: int) -> int:
    return int(lib().dq_default_levels(bits))


def status_string(status: int) -> str:
    return lib().dq_status_string(status).decode()


def _check(status: int, what: str):
    if status != 0:
        raise DqError(status, what)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev_ptr(t: Optional[torch.Tensor], dtype, what: str) -> Optional[int]:
    if t is None:
        return None
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{what}: expected a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _host_ptr(t, dtype, what: str) -> Optional[int]:
    if t is None:
        return None
    if not isinstance(t, torch.Tensor):
        t = torch.from_numpy(t)
    if t.is_cuda or not t.is_contiguous() or t.dtype != dtype:
        raise TypeError(f"{what}: expected a contiguous CPU tensor of {dtype}")
    return t.data_ptr()


def make_params(bucket: int, bits: int, levels: int = 0, coarse_K: int = 0, fine_M: float = 0.0,
                alpha: float = 0.0, dither_bits: int = 0, flags: int = 0) -> DqParams:
    return DqParams(bucket, bits, levels, coarse_K, fine_M, alpha, dither_bits, flags)


class Message:
    """A worker's message on the device plus what the decoder must know about it."""

    def __init__(self, packed: torch.Tensor, scale: torch.Tensor, seed: int, worker: int, kind: int,
                 params: DqParams):
        self.packed, self.scale = packed, scale
        self.seed, self.worker, self.kind, self.params = seed, worker, kind, params

    def as_struct(self, host: bool = False) -> DqMsg:
        if host:
            pk = _host_ptr(self.packed, torch.int32, "packed")
            sc = _host_ptr(self.scale, torch.float32, "scale")
        else:
            pk = _dev_ptr(self.packed, torch.int32, "packed")
            sc = _dev_ptr(self.scale, torch.float32, "scale")
        return DqMsg(pk, sc, self.seed, self.worker, self.kind, self.params)


def new_output(numel: int, dtype, device) -> torch.Tensor:
    """Every output tensor that this binding allocates on behalf of the caller comes from here (one place to
    hook, e.g. for tests that surround outputs with guard words)."""
    return torch.empty(numel, dtype=dtype, device=device)


def alloc_message(n: int, params: DqParams, device="cuda"):
    """Uninitialised output buffers for one encode call (packed words as int32, scales as fp32)."""
    packed = new_output(max(1, packed_words(n, params.bits)), torch.int32, device)
    scale = new_output(max(1, num_buckets(n, params.bucket)), torch.float32, device)
    return packed, scale


def _encode(fn, what, grad, seed, worker, step, params, out_packed, out_scale, stream):
    n = grad.numel()
    if out_packed is None or out_scale is None:
        out_packed, out_scale = alloc_message(n, params, grad.device)
    if out_packed.numel() < packed_words(n, params.bits) or out_scale.numel() < num_buckets(n, params.bucket):
        raise ValueError(f"{what}: output buffers too small")
    _check(fn(_dev_ptr(grad, torch.float32, "grad"), n, seed, worker, step, C.byref(params),
              _dev_ptr(out_packed, torch.int32, "out_packed"), _dev_ptr(out_scale, torch.float32, "out_scale"),
              _stream_ptr(stream)), what)
    return out_packed, out_scale


def dqsg_encode(grad: torch.Tensor, seed: int, worker: int, step: int, params: DqParams,
                out_packed: Optional[torch.Tensor] = None, out_scale: Optional[torch.Tensor] = None,
                stream=None):
    return _encode(lib().dqsg_encode, "dqsg_encode", grad, seed, worker, step, params, out_packed, out_scale, stream)


def ndqsg_encode(grad: torch.Tensor, seed: int, worker: int, step: int, params: DqParams,
                 out_packed: Optional[torch.Tensor] = None, out_scale: Optional[torch.Tensor] = None,
                 stream=None):
    return _encode(lib().ndqsg_encode, "ndqsg_encode", grad, seed, worker, step, params, out_packed, out_scale, stream)


def bucket_ranges(n: int, bucket: int, parts: int):
    """Cuts [0, n) into `parts` consecutive bucket-aligned ranges of nearly equal bucket counts (host arithmetic).

    Returns [(first_element, count), ...]; ranges at the end may be empty when there are fewer buckets than parts.
    Feed them to the *_range calls: one range per GPU, per transfer chunk or per layer group.
    """
    if n < 0 or bucket <= 0 or parts <= 0:
        raise ValueError("bucket_ranges: n >= 0, bucket > 0 and parts > 0 are required")
    nb = -(-n // bucket)
    out = []
    for r in range(parts):
        b0 = nb * r // parts
        b1 = nb * (r + 1) // parts
        lo, hi = min(n, b0 * bucket), min(n, b1 * bucket)
        out.append((lo, hi - lo))
    return out


def _encode_range(fn, what, grad, first_element, seed, worker, step, params, out_packed, out_scale, stream):
    n = grad.numel()
    if out_packed is None or out_scale is None:
        out_packed, out_scale = alloc_message(n, params, grad.device)
    if out_packed.numel() < packed_words(n, params.bits) or out_scale.numel() < num_buckets(n, params.bucket):
        raise ValueError(f"{what}: output buffers too small")
    _check(fn(_dev_ptr(grad, torch.float32, "grad"), n, first_element, seed, worker, step, C.byref(params),
              _dev_ptr(out_packed, torch.int32, "out_packed"), _dev_ptr(out_scale, torch.float32, "out_scale"),
              _stream_ptr(stream)), what)
    return out_packed, out_scale


def dqsg_encode_range(grad: torch.Tensor, first_element: int, seed: int, worker: int, step: int, params: DqParams,
                      out_packed: Optional[torch.Tensor] = None, out_scale: Optional[torch.Tensor] = None,
                      stream=None):
    """DQSG encode of the elements [first_element, first_element + grad.numel()) of a longer gradient."""
    return _encode_range(lib().dqsg_encode_range, "dqsg_encode_range", grad, first_element, seed, worker, step,
                         params, out_packed, out_scale, stream)


def ndqsg_encode_range(grad: torch.Tensor, first_element: int, seed: int, worker: int, step: int, params: DqParams,
                       out_packed: Optional[torch.Tensor] = None, out_scale: Optional[torch.Tensor] = None,
                       stream=None):
    return _encode_range(lib().ndqsg_encode_range, "ndqsg_encode_range", grad, first_element, seed, worker, step,
                         params, out_packed, out_scale, stream)


def _msg_array(msgs: Sequence[Message], host: bool = False):
    arr = (DqMsg * max(1, len(msgs)))()
    for i, m in enumerate(msgs):
        arr[i] = m.as_struct(host)
    return arr


def dqsg_decode_aggregate(msgs: Sequence[Message], n: int, step: int, out_avg: Optional[torch.Tensor] = None,
                          stream=None) -> torch.Tensor:
    if out_avg is None:
        out_avg = new_output(max(1, n), torch.float32, msgs[0].packed.device)
    _check(lib().dqsg_decode_aggregate(_msg_array(msgs), len(msgs), n, step,
                                       _dev_ptr(out_avg, torch.float32, "out_avg"), _stream_ptr(stream)),
           "dqsg_decode_aggregate")
    return out_avg


def ndqsg_decode_aggregate(msgs: Sequence[Message], n: int, step: int, side_info: Optional[torch.Tensor],
                           out_avg: Optional[torch.Tensor] = None, status_word: Optional[torch.Tensor] = None,
                           stream=None) -> torch.Tensor:
    if out_avg is None:
        out_avg = new_output(max(1, n), torch.float32, msgs[0].packed.device)
    _check(lib().ndqsg_decode_aggregate(_msg_array(msgs), len(msgs), n, step,
                                        _dev_ptr(side_info, torch.float32, "side_info"),
                                        _dev_ptr(out_avg, torch.float32, "out_avg"),
                                        _dev_ptr(status_word, torch.int32, "status_word"), _stream_ptr(stream)),
           "ndqsg_decode_aggregate")
    return out_avg


def ndqsg_decode_aggregate_range(msgs: Sequence[Message], n: int, first_element: int, step: int,
                                 side_info: Optional[torch.Tensor], out_avg: Optional[torch.Tensor] = None,
                                 status_word: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Fused decode-and-average of a bucket range: every buffer holds the range's data only."""
    if out_avg is None:
        out_avg = new_output(max(1, n), torch.float32, msgs[0].packed.device)
    _check(lib().ndqsg_decode_aggregate_range(_msg_array(msgs), len(msgs), n, first_element, step,
                                              _dev_ptr(side_info, torch.float32, "side_info"),
                                              _dev_ptr(out_avg, torch.float32, "out_avg"),
                                              _dev_ptr(status_word, torch.int32, "status_word"),
                                              _stream_ptr(stream)), "ndqsg_decode_aggregate_range")
    return out_avg


def dqsg_decode_aggregate_half_dithered(msgs: Sequence[Message], n: int, out_avg: Optional[torch.Tensor] = None,
                                        stream=None) -> torch.Tensor:
    """Mean of the DQSG messages reconstructed without subtracting the dither (Section 2.1, Lemma 1)."""
    if out_avg is None:
        out_avg = new_output(max(1, n), torch.float32, msgs[0].packed.device)
    _check(lib().dqsg_decode_aggregate_half_dithered(_msg_array(msgs), len(msgs), n,
                                                     _dev_ptr(out_avg, torch.float32, "out_avg"),
                                                     _stream_ptr(stream)), "dqsg_decode_aggregate_half_dithered")
    return out_avg


def ndqsg_decode_aggregate_running(msgs: Sequence[Message], n: int, step: int,
                                   out_avg: Optional[torch.Tensor] = None,
                                   status_word: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Algorithm 2's server loop: NDQSG messages are decoded against the mean of the messages before them."""
    if out_avg is None:
        out_avg = new_output(max(1, n), torch.float32, msgs[0].packed.device)
    _check(lib().ndqsg_decode_aggregate_running(_msg_array(msgs), len(msgs), n, step,
                                                _dev_ptr(out_avg, torch.float32, "out_avg"),
                                                _dev_ptr(status_word, torch.int32, "status_word"),
                                                _stream_ptr(stream)), "ndqsg_decode_aggregate_running")
    return out_avg


def ndqsg_decode_aggregate_side_first(msgs: Sequence[Message], n: int, step: int,
                                      out_avg: Optional[torch.Tensor] = None,
                                      status_word: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Algorithm 2 with one P1 worker: the reconstruction of message 0 is the side information of the rest."""
    if out_avg is None:
        out_avg = new_output(max(1, n), torch.float32, msgs[0].packed.device)
    _check(lib().ndqsg_decode_aggregate_side_first(_msg_array(msgs), len(msgs), n, step,
                                                   _dev_ptr(out_avg, torch.float32, "out_avg"),
                                                   _dev_ptr(status_word, torch.int32, "status_word"),
                                                   _stream_ptr(stream)), "ndqsg_decode_aggregate_side_first")
    return out_avg


def code_histogram(packed: torch.Tensor, n: int, bits: int, hist: Optional[torch.Tensor] = None,
                   stream=None) -> torch.Tensor:
    """hist[c] = number of elements of the packed message whose code is c (int64[2^bits] on the device)."""
    if hist is None:
        hist = new_output(1 << bits, torch.int64, packed.device)
    _check(lib().dq_code_histogram(_dev_ptr(packed, torch.int32, "packed"), n, bits,
                                   _dev_ptr(hist, torch.int64, "hist"), _stream_ptr(stream)), "dq_code_histogram")
    return hist


def entropy_bits_per_element(hist) -> float:
    """Empirical entropy of a code histogram in bits per element (dq_code_entropy on a host copy of it)."""
    counts = [int(c) for c in hist.tolist()]
    bits = max(1, (len(counts) - 1).bit_length())
    arr = (C.c_uint64 * (1 << bits))(*counts)
    out = C.c_double(0.0)
    _check(lib().dq_code_entropy(arr, bits, C.byref(out)), "dq_code_entropy")
    return float(out.value)


# ------------------------------------------------------------------------------------------ radix-3 container
def ternary_bytes(n: int) -> int:
    return int(lib().dq_ternary_bytes(n))


def ternary_pack(packed: torch.Tensor, n: int, out: Optional[torch.Tensor] = None,
                 status_word: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """2-bit stream of a three-level message -> five codes per byte (uint8[ternary_bytes(n)] on the device)."""
    if out is None:
        out = new_output(max(1, ternary_bytes(n)), torch.uint8, packed.device)
    _check(lib().dq_ternary_pack(_dev_ptr(packed, torch.int32, "packed"), n, _dev_ptr(out, torch.uint8, "out"),
                                 _dev_ptr(status_word, torch.int32, "status_word"), _stream_ptr(stream)),
           "dq_ternary_pack")
    return out


def ternary_unpack(data: torch.Tensor, n: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Five codes per byte -> the 2-bit stream (int32[packed_words(n, 2)] on the device)."""
    if out is None:
        out = new_output(max(1, packed_words(n, 2)), torch.int32, data.device)
    _check(lib().dq_ternary_unpack(_dev_ptr(data, torch.uint8, "data"), n, _dev_ptr(out, torch.int32, "out"),
                                   _stream_ptr(stream)), "dq_ternary_unpack")
    return out


# ------------------------------------------------------------------------------------------ host buffers
def encode_workspace_bytes(n: int, params: DqParams) -> int:
    return int(lib().dq_encode_workspace_bytes(n, C.byref(params)))


def decode_workspace_bytes(msgs: Sequence[Message], n: int, has_side_info: bool) -> int:
    return int(lib().dq_decode_workspace_bytes(_msg_array(msgs, host=True), len(msgs), n, int(has_side_info)))


def _encode_host(fn, what, grad, seed, worker, step, params, out_packed, out_scale, workspace, stream):
    n = grad.numel()
    _check(fn(_host_ptr(grad, torch.float32, "grad"), n, seed, worker, step, C.byref(params),
              _host_ptr(out_packed, torch.int32, "out_packed"), _host_ptr(out_scale, torch.float32, "out_scale"),
              workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(stream)), what)
    return out_packed, out_scale


def dqsg_encode_host(grad, seed, worker, step, params, out_packed, out_scale, workspace, stream=None):
    return _encode_host(lib().dqsg_encode_host, "dqsg_encode_host", grad, seed, worker, step, params,
                        out_packed, out_scale, workspace, stream)


def ndqsg_encode_host(grad, seed, worker, step, params, out_packed, out_scale, workspace, stream=None):
    return _encode_host(lib().ndqsg_encode_host, "ndqsg_encode_host", grad, seed, worker, step, params,
                        out_packed, out_scale, workspace, stream)


STATIC_SCRATCH_BYTES = 32 * 1024 * 1024


def dqsg_encode_host_static(grad, seed, worker, step, params, out_packed, out_scale, stream=None):
    """DQSG encode from host buffers to host buffers without any device allocation by the caller: the
    staging area is the library's built-in array (at most STATIC_SCRATCH_BYTES for input plus outputs).
    For callers that cannot allocate GPU memory themselves; calls on one device must not overlap."""
    n = grad.numel() if isinstance(grad, torch.Tensor) else grad.size
    _check(lib().dqsg_encode_host_static(_host_ptr(grad, torch.float32, "grad"), n, seed, worker, step,
                                         C.byref(params), _host_ptr(out_packed, torch.int32, "out_packed"),
                                         _host_ptr(out_scale, torch.float32, "out_scale"),
                                         None if stream is None else _stream_ptr(stream)),
           "dqsg_encode_host_static")
    return out_packed, out_scale


def ndqsg_decode_aggregate_host(msgs: Sequence[Message], n: int, step: int, side_info, out_avg, workspace,
                                stream=None):
    _check(lib().ndqsg_decode_aggregate_host(_msg_array(msgs, host=True), len(msgs), n, step,
                                             _host_ptr(side_info, torch.float32, "side_info"),
                                             _host_ptr(out_avg, torch.float32, "out_avg"),
                                             workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                             _stream_ptr(stream)), "ndqsg_decode_aggregate_host")
    return out_avg


def ndqsg_decode_aggregate_side_first_host(msgs: Sequence[Message], n: int, step: int, out_avg, workspace,
                                           stream=None):
    _check(lib().ndqsg_decode_aggregate_side_first_host(_msg_array(msgs, host=True), len(msgs), n, step,
                                                        _host_ptr(out_avg, torch.float32, "out_avg"),
                                                        workspace.data_ptr(),
                                                        workspace.numel() * workspace.element_size(),
                                                        _stream_ptr(stream)), "ndqsg_decode_aggregate_side_first_host")
    return out_avg


def device_error_flags() -> int:
    v = C.c_uint32(0)
    _check(lib().dq_device_error_flags(C.byref(v)), "dq_device_error_flags")
    return int(v.value)


def launch_count() -> int:
    return int(lib().dq_launch_count())
