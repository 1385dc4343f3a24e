"""Host-side checks that need no GPU: the C-ABI library builds, loads, exports every symbol the header
declares, and rejects invalid arguments before touching the device."""
import ctypes as C
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def dq():
    from paper_1904_01197_b200 import build
    build.build()
    import paper_1904_01197_b200 as dq
    return dq


def _declared_functions():
    text = (ROOT / "include" / "dq.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(?:dq_status|uint64_t|uint32_t|const char\*)\s+(\w+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(dq):
    names = _declared_functions()
    assert {"dqsg_encode", "ndqsg_encode", "dqsg_decode_aggregate", "ndqsg_decode_aggregate",
            "dq_packed_words", "dq_num_buckets", "dq_status_string"} <= set(names)
    L = dq.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in include/dq.h but not exported"


def test_struct_layout_matches_header(dq):
    assert C.sizeof(dq.DqParams) == 32
    assert C.sizeof(dq.DqMsg) == 64
    assert dq.DqMsg.p.offset == 32 and dq.DqMsg.seed.offset == 16


def test_size_helpers(dq):
    assert dq.packed_words(65536, 2) == 4096
    assert dq.packed_words(33, 3) == 4
    assert dq.packed_words(0, 3) == 0
    assert dq.num_buckets(25_557_032, 2048) == 12480
    assert dq.num_buckets(124_439_808, 4096) == 30381
    assert [dq.default_levels(b) for b in range(1, 9)] == [2, 3, 7, 15, 31, 63, 127, 255]
    assert dq.status_string(0) == "ok"


def test_invalid_arguments_are_rejected_before_any_launch(dq):
    L = dq.lib()
    launches_before = L.dq_launch_count()
    P = dq.binding.make_params
    fake = 0x1000                                      # never dereferenced: checks come first
    bad = [
        (P(48, 2), 1),                                 # bucket not a multiple of 32
        (P(16, 2), 1),                                 # bucket too small
        (P(131072, 2), 1),                             # bucket too large
        (P(512, 0), 1),                                # bits
        (P(512, 9), 1),
        (P(512, 2, 5), 1),                             # 5 levels do not fit 2 bits
        (P(512, 2, 1), 1),                             # one level
        (P(512, 2, 3, dither_bits=8), 1),              # unknown dither stream
    ]
    for p, want in bad:
        assert L.dqsg_encode(fake, 1024, 1, 0, 0, C.byref(p), fake, fake, None) == want
    nbad = [
        (P(512, 2, 0, 5, 4.0, 1.0), 1),                # K > 2^bits
        (P(512, 2, 0, 1, 4.0, 1.0), 1),                # K < 2
        (P(512, 2, 0, 4, 0.0, 1.0), 1),                # M1 = 0
        (P(512, 2, 0, 4, 4.0, 1.5), 1),                # alpha > 1
        (P(512, 2, 0, 4, 4.0, -0.5), 1),
        (P(512, 2, 0, 4, 4194304.0, 1.0), 2),          # alpha*M1 above the supported range
    ]
    for p, want in nbad:
        assert L.ndqsg_encode(fake, 1024, 1, 0, 0, C.byref(p), fake, fake, None) == want
    ok = P(512, 2)
    assert L.dqsg_encode(None, 1024, 1, 0, 0, C.byref(ok), fake, fake, None) == 1         # NULL grad
    assert L.dqsg_encode(fake + 4, 1024, 1, 0, 0, C.byref(ok), fake, fake, None) == 3     # misaligned
    assert L.dqsg_encode(fake, 1 << 34, 1, 0, 0, C.byref(ok), fake, fake, None) == 2      # n too large
    assert L.dqsg_encode(fake, 0, 1, 0, 0, C.byref(ok), fake, fake, None) == 0            # n = 0: no-op
    assert L.dqsg_encode(fake, 1024, 1, 0, 0, None, fake, fake, None) == 1                # NULL params

    m = dq.DqMsg(fake, fake, 1, 0, dq.DQ_KIND_DQSG, ok)
    arr = (dq.DqMsg * 2)(m, m)
    assert L.dqsg_decode_aggregate(arr, 0, 1024, 0, fake, None) == 1                      # W = 0
    assert L.dqsg_decode_aggregate(arr, 65, 1024, 0, fake, None) == 1                     # W too large
    assert L.dqsg_decode_aggregate(None, 1, 1024, 0, fake, None) == 1
    nd = dq.DqMsg(fake, fake, 1, 0, dq.DQ_KIND_NDQSG, P(512, 2, 0, 4, 4.0, 1.0))
    arr2 = (dq.DqMsg * 2)(m, nd)
    assert L.dqsg_decode_aggregate(arr2, 2, 1024, 0, fake, None) == 1                     # NDQSG in a DQSG-only call
    assert L.ndqsg_decode_aggregate(arr2, 2, 1024, 0, None, fake, None, None) == 1        # side info missing
    other = dq.DqMsg(fake, fake, 1, 0, dq.DQ_KIND_DQSG, P(1024, 2))
    arr3 = (dq.DqMsg * 2)(m, other)
    assert L.dqsg_decode_aggregate(arr3, 2, 1024, 0, fake, None) == 2                     # mixed bucket sizes
    d16 = dq.DqMsg(fake, fake, 1, 0, dq.DQ_KIND_DQSG, P(512, 2, dither_bits=16))
    arr4 = (dq.DqMsg * 2)(m, d16)
    assert L.dqsg_decode_aggregate(arr4, 2, 1024, 0, fake, None) == 2                     # mixed dither streams
    assert L.dqsg_decode_aggregate(arr, 2, 0, 0, fake, None) == 0                         # n = 0
    assert L.dq_launch_count() == launches_before


def test_workspace_sizes(dq):
    p = dq.binding.make_params(2048, 2)
    n = 10_000
    need = dq.encode_workspace_bytes(n, p)
    assert need >= n * 4 + dq.packed_words(n, 2) * 4 + dq.num_buckets(n, 2048) * 4
    assert need % 256 == 0


def test_host_decode_rejects_bad_message_sets_before_any_copy(dq):
    """Mixed bucket sizes, mixed dither widths and a nested message without side information are refused by the
    host-buffer decode before a single byte is copied: every pointer here is a fake that must not be touched."""
    L = dq.lib()
    P = dq.binding.make_params
    fake = 0x1000

    def msg(kind, p):
        return dq.DqMsg(fake, fake, 1, 0, kind, p)

    def call(msgs, side):
        arr = (dq.DqMsg * len(msgs))(*msgs)
        return L.ndqsg_decode_aggregate_host(arr, len(msgs), 4096, 0, side, fake, fake, 1 << 30, None)

    dqsg, nd = dq.DQ_KIND_DQSG, dq.DQ_KIND_NDQSG
    assert call([msg(dqsg, P(512, 2)), msg(dqsg, P(1024, 2))], None) == 2            # mixed buckets
    assert call([msg(dqsg, P(512, 2, dither_bits=32)), msg(dqsg, P(512, 2, dither_bits=16))], None) == 2
    assert call([msg(dqsg, P(512, 2)), msg(nd, P(512, 2, 0, 4, 2.0, 1.0))], None) == 1   # nested, no side info
    p = P(512, 2)
    assert L.dqsg_encode_host(fake, 1 << 34, 1, 0, 0, C.byref(p), fake, fake, fake, 1 << 40, None) == 2
