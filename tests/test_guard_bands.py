"""The guard-band harness itself (tests/conftest.py), on the CPU: a write past either end of a
guarded buffer is reported, a clean buffer is not."""
import pytest
import torch

from conftest import BAND, GuardedAllocator


def test_guarded_allocator_reports_writes_outside_the_buffer():
    g = GuardedAllocator()
    t = g(100, torch.float32, torch.device("cpu"), True)
    assert t.numel() == 100 and t.dtype == torch.float32 and not t.any() and t.data_ptr() % 32 == 0
    t.fill_(1.0)
    g.finish()                                           # clean
    for where in (-1, 400, 400 + 11, -BAND):
        g = GuardedAllocator()
        t = g(100, torch.float32, torch.device("cpu"), False)
        base, nbytes = g.live[0]
        assert nbytes == 400
        base[BAND + where] = 0                           # one byte before / past the interior
        with pytest.raises(AssertionError):
            g.finish()
    g = GuardedAllocator()
    e = g(0, torch.uint8, torch.device("cpu"), False)     # empty buffers are fine
    assert e.numel() == 0
    g.finish()
