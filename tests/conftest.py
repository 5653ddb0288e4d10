import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (run with -m gpu)")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped, not failed, where no device is present."""
    try:
        import torch
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


# --------------------------------------------------------------------------- guard bands
#
# Every buffer the binding allocates for a GPU test (outputs and workspaces) sits between two
# bands of a known byte pattern; after the test (and, for large buffers, as soon as enough of
# them have piled up) the bands are read back.  A kernel that writes one element before or
# past a buffer fails the test that ran it.

BAND = 4096                 # bytes on each side; keeps the interior 32-byte aligned
PATTERN = 0xA5
KEEP_BYTES = 1 << 30        # guarded buffers kept alive for the end-of-test check


class GuardedAllocator:
    def __init__(self):
        self.live = []       # (base uint8 tensor, nbytes)
        self.bytes = 0
        self.checked = 0

    def __call__(self, numel, dtype, device, zero):
        import torch
        esize = torch.empty(0, dtype=dtype).element_size()
        nbytes = numel * esize
        pad = -nbytes % 32                      # the right band starts on a 32-byte boundary
        base = torch.empty(BAND + nbytes + pad + BAND, dtype=torch.uint8, device=device)
        base[:BAND] = PATTERN
        base[BAND + nbytes:] = PATTERN
        inner = base[BAND:BAND + nbytes]
        if zero:
            inner.zero_()
        self.live.append((base, nbytes))
        self.bytes += base.numel()
        while self.bytes > KEEP_BYTES and len(self.live) > 1:
            self._check(*self.live.pop(0))      # stream-ordered: after the calls enqueued so far
        return inner.view(dtype)

    def _check(self, base, nbytes):
        left, right = base[:BAND], base[BAND + nbytes:]
        ok = bool((left == PATTERN).all().item()) and bool((right == PATTERN).all().item())
        self.bytes -= base.numel()
        self.checked += 1
        assert ok, "a kernel wrote outside a %d-byte buffer (guard band damaged)" % nbytes

    def finish(self):
        while self.live:
            self._check(*self.live.pop(0))


@pytest.fixture(autouse=True)
def guard_bands(request):
    if "gpu" not in request.keywords:
        yield None
        return
    import torch
    if not torch.cuda.is_available():
        yield None
        return
    from paper_2505_06653_b200 import binding
    alloc = GuardedAllocator()
    binding.set_output_allocator(alloc)
    try:
        yield alloc
        torch.cuda.synchronize()
        alloc.finish()
    finally:
        binding.set_output_allocator(None)
