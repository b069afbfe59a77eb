import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


class _GuardedAllocator:
    """Stands in for torch.empty inside the binding during GPU tests: every output and workspace sits between two
    256-byte margins filled with a fixed byte, and the margins are checked after the test.  (No memory checker
    runs on this code, so writes past the end of a buffer are looked for this way, next to the comparison with
    the oracle.)"""
    MARGIN, BYTE = 256, 0xA5

    def __init__(self):
        self.live = []

    def __call__(self, *size, dtype=None, device=None, **kw):
        import torch
        if kw or device is None or torch.device(device).type != "cuda":
            return torch.empty(*size, dtype=dtype, device=device, **kw)
        shape = tuple(size[0]) if len(size) == 1 and isinstance(size[0], (tuple, list, torch.Size)) else tuple(size)
        dtype = dtype or torch.float32
        n = 1
        for s in shape:
            n *= int(s)
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        body = (nbytes + 255) // 256 * 256
        buf = torch.empty(self.MARGIN + body + self.MARGIN, dtype=torch.uint8, device=device)
        buf[: self.MARGIN] = self.BYTE
        buf[self.MARGIN + nbytes:] = self.BYTE
        self.live.append((buf, nbytes))
        return buf[self.MARGIN: self.MARGIN + nbytes].view(dtype).view(shape)

    def check(self):
        import torch
        torch.cuda.synchronize()
        for buf, nbytes in self.live:
            head = buf[: self.MARGIN]
            tail = buf[self.MARGIN + nbytes:]
            assert bool((head == self.BYTE).all()), "write before the start of a buffer"
            assert bool((tail == self.BYTE).all()), "write past the end of a buffer"
        self.live.clear()


@pytest.fixture(autouse=True)
def _guard_bytes_around_every_device_buffer(request):
    if "gpu" not in request.keywords:
        yield
        return
    from paper_2608_04962_b200 import binding
    g = _GuardedAllocator()
    binding.set_allocator(g)
    try:
        yield
        g.check()
    finally:
        binding.set_allocator(None)
