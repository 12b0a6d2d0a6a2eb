import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")
    config.addinivalue_line("markers", "guard_each_call: check the guard zones after every library call, not only "
                                       "at the end of the test (synchronises the device each time)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session", autouse=True)
def _library_is_built():
    """A fresh checkout has no built library (it is kept out of the history): build it once, with nvcc."""
    from paper_2609_07008_b200 import build
    build.ensure_built()


# ---- guard zones around every buffer the binding allocates (a stand-in for a memory checker) ---------------
GUARD_BYTES = 4096
GUARD_BYTE = 0xA5


class GuardedAllocator:
    """Hands out buffers with 4 KB of sentinel bytes on either side and checks the sentinels after every
    library call of the test (the device is synchronised first: test mode only)."""

    def __init__(self):
        self.live = []          # (name, whole uint8 buffer, payload bytes)

    def __call__(self, shape, dtype, device):
        import math
        import torch
        shape = (shape,) if isinstance(shape, int) else tuple(shape)
        n = math.prod(shape) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % 256                                  # keep the trailing guard 256-byte aligned too
        raw = torch.full((GUARD_BYTES + n + pad + GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device=device)
        self.live.append((f"{dtype} {shape}", raw, n))
        return raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)

    def verify(self):
        import torch
        if not self.live:
            return
        torch.cuda.synchronize()
        for name, raw, n in self.live:
            head, tail = raw[:GUARD_BYTES], raw[GUARD_BYTES + n:]
            assert bool((head == GUARD_BYTE).all()), f"bytes written in front of output buffer {name}"
            assert bool((tail == GUARD_BYTE).all()), f"bytes written behind output buffer {name}"


@pytest.fixture(autouse=True)
def _guard_zones(request, monkeypatch):
    """Every GPU test runs with guard zones around the binding's output and scratch buffers; buffers above
    512 MB (the full-size cases' big outputs) are guarded too, the cost is 8 KB each."""
    if "gpu" not in request.keywords:
        yield
        return
    from paper_2609_07008_b200 import binding
    alloc = GuardedAllocator()
    monkeypatch.setattr(binding, "_empty", alloc)
    plain_check = binding.Context.check

    def check_then_verify(self, status):
        plain_check(self, status)
        if request.node.get_closest_marker("guard_each_call") is not None:
            alloc.verify()

    monkeypatch.setattr(binding.Context, "check", check_then_verify)
    yield
    alloc.verify()
    alloc.live.clear()
