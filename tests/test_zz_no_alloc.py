"""`dqsg_encode_host_static`: the DQSG encoder for callers that cannot allocate GPU memory.

A process whose framework already owns the device's memory, a plug-in that only receives host buffers, or a
latency-critical loop that must not call cudaMalloc can still encode: the staging area lives inside the library
as a fixed device array.  This test drives the entry point through the C ABI with plain numpy buffers (no device
tensor is created for it), twice in a row with different inputs, because the array is shared between calls and
keeps the previous call's bytes: the second result must not depend on the first.  The results are compared,
bit for bit, with `dqsg_encode_host`, which gets its workspace from the caller, and with the CPU oracle's
encoder, so that the comparison does not rest on the CUDA path alone.

The file is named so that pytest collects it last.
"""
import ctypes as C

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def dq():
    from paper_1904_01197_b200 import build
    build.build()
    import paper_1904_01197_b200 as dq
    assert torch.cuda.is_available()
    return dq


def _reference(dq, g, seed, worker, step, params):
    """The existing host-buffer entry point, with a caller-provided workspace."""
    n = g.size
    ws = torch.empty(dq.encode_workspace_bytes(n, params), dtype=torch.uint8, device="cuda")
    pk = torch.empty(dq.packed_words(n, params.bits), dtype=torch.int32)
    sc = torch.empty(dq.num_buckets(n, params.bucket), dtype=torch.float32)
    dq.dqsg_encode_host(torch.from_numpy(g), seed, worker, step, params, pk, sc, ws)
    return pk.numpy().copy(), sc.numpy().copy()


def _oracle(g, seed, worker, step, params):
    """The CPU oracle's DQSG encoder on the same input."""
    import oracle
    oracle.build()
    return oracle.dqsg_encode(g, seed, worker, step, params.bucket, params.bits, params.levels)


def _static(dq, g, seed, worker, step, params):
    """The entry point under test, called straight through ctypes with numpy buffers."""
    n = g.size
    pk = np.full(dq.packed_words(n, params.bits), -1, dtype=np.int32)
    sc = np.full(dq.num_buckets(n, params.bucket), np.nan, dtype=np.float32)
    rc = dq.lib().dqsg_encode_host_static(g.ctypes.data, n, seed, worker, step, C.byref(params),
                                          pk.ctypes.data, sc.ctypes.data, None)
    assert rc == 0, dq.status_string(rc)
    return pk, sc


def test_static_scratch_encode_matches_workspace_encode_twice_in_a_row(dq):
    rng = np.random.default_rng(2024)
    # first call: a long vector (tiles + ragged end), 3 bits; second call: shorter, other bucket size and width,
    # so stale bytes of the first call lie behind and inside the regions the second call uses
    cases = [
        (rng.standard_normal(1_500_000 + 77).astype(np.float32) * 0.01, dq.binding.make_params(2048, 3, 5), 11, 3, 7),
        (rng.standard_normal(300_000 + 5).astype(np.float32) * 3.0, dq.binding.make_params(512, 2, 3), 12, 1, 8),
    ]
    for g, params, seed, worker, step in cases:
        got_pk, got_sc = _static(dq, g, seed, worker, step, params)
        ref_pk, ref_sc = _reference(dq, g, seed, worker, step, params)
        assert np.array_equal(got_sc.view(np.uint32), ref_sc.view(np.uint32))      # scales: bit-exact
        assert np.array_equal(got_pk, ref_pk)                                      # packed words: bit-exact
        ora_pk, ora_sc = _oracle(g, seed, worker, step, params)
        assert np.array_equal(got_pk.view(np.uint32), ora_pk), "packed words differ from the oracle's"
        assert np.array_equal(got_sc.view(np.uint32), ora_sc.view(np.uint32)), "scales differ from the oracle's"
    # and once more with the first input: same answer as before, whatever the array held in between
    g, params, seed, worker, step = cases[0]
    again_pk, again_sc = _static(dq, g, seed, worker, step, params)
    ref_pk, ref_sc = _reference(dq, g, seed, worker, step, params)
    assert np.array_equal(again_pk, ref_pk) and np.array_equal(again_sc, ref_sc)
    assert dq.device_error_flags() == 0


def test_static_scratch_rejects_inputs_beyond_its_size(dq):
    params = dq.binding.make_params(2048, 2, 3)
    n = 9_000_000                                            # 36 MB of gradient alone: over the 32 MiB array
    assert dq.encode_workspace_bytes(n, params) > dq.STATIC_SCRATCH_BYTES
    fake = 0x1000                                            # never dereferenced: the size check comes first
    rc = dq.lib().dqsg_encode_host_static(fake, n, 1, 0, 0, C.byref(params), fake, fake, None)
    assert rc == 5 and "scratch" in dq.status_string(rc)
    # the largest vector that fits is accepted by the size check (n = 0 needs no buffers at all)
    assert dq.lib().dqsg_encode_host_static(fake, 0, 1, 0, 0, C.byref(params), fake, fake, None) == 0
