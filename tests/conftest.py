import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

GOLDEN = Path(__file__).resolve().parent / "golden"


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def _have_gpu():
    try:
        import torch
        return torch.cuda.is_available()
    except Exception:
        return False


def pytest_collection_modifyitems(config, items):
    if _have_gpu():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(scope="session")
def golden_dir():
    return GOLDEN


GUARD_BYTES = 256
CURRENT_GUARD = None        # the GuardedOutputs of the GPU test that is running
GUARD_PATTERN = 0xA5


class GuardedOutputs:
    """Stands in for the out-of-bounds checker of a sanitizer: every output buffer that the binding allocates is
    carved out of a larger one with GUARD_BYTES of a known pattern before and after it, and the pattern is checked
    when the test ends.  A kernel that writes one byte past (or before) an output fails the test that ran it."""

    def __init__(self, torch):
        self.torch = torch
        self.buffers = []

    def new_output(self, numel, dtype, device):
        torch = self.torch
        nbytes = numel * torch.empty((), dtype=dtype).element_size()
        padded = (nbytes + 15) // 16 * 16                     # the view must keep 16-byte alignment on both sides
        buf = torch.full((GUARD_BYTES + padded + GUARD_BYTES,), GUARD_PATTERN, dtype=torch.uint8, device=device)
        self.buffers.append((buf, nbytes))
        return buf[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype)

    def host_output(self, numel, dtype):
        """The same for a pinned host buffer that a *_host entry point fills."""
        torch = self.torch
        nbytes = numel * torch.empty((), dtype=dtype).element_size()
        padded = (nbytes + 15) // 16 * 16
        buf = torch.full((GUARD_BYTES + padded + GUARD_BYTES,), GUARD_PATTERN, dtype=torch.uint8).pin_memory()
        self.buffers.append((buf, nbytes))
        return buf[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype)

    def check(self):
        torch = self.torch
        if self.buffers and torch.cuda.is_available():
            torch.cuda.synchronize()
        for k, (buf, nbytes) in enumerate(self.buffers):
            front = buf[:GUARD_BYTES]
            back = buf[GUARD_BYTES + nbytes:]
            assert bool((front == GUARD_PATTERN).all()), f"output {k} ({nbytes} bytes): bytes before it were overwritten"
            assert bool((back == GUARD_PATTERN).all()), f"output {k} ({nbytes} bytes): bytes after it were overwritten"
        self.buffers.clear()


@pytest.fixture(autouse=True)
def guarded_outputs(request, monkeypatch):
    """GPU tests run with guard words around every output the binding allocates (see GuardedOutputs)."""
    if "gpu" not in request.keywords or not _have_gpu():
        yield None
        return
    import torch
    from paper_1904_01197_b200 import binding
    global CURRENT_GUARD
    g = GuardedOutputs(torch)
    monkeypatch.setattr(binding, "new_output", g.new_output)
    CURRENT_GUARD = g
    yield g
    CURRENT_GUARD = None
    g.check()
