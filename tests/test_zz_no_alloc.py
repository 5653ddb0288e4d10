"""opq_split_static: the outlier split for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits (another component owns the
memory pool, the host framework forbids device-synchronising calls, or no allocator exists
yet).  For them the library carries its own 4 MiB of scratch.  This file checks, through the
C ABI, that the allocation-free entry point returns exactly what opq_split returns with a
caller-provided workspace, on two calls in a row that share the built-in scratch, and that it
refuses tensors beyond its limit.  It is collected last on purpose."""
import ctypes

import numpy as np
import pytest
import torch

import workloads

pytestmark = pytest.mark.gpu

I = 64
MAX_N = 1 << 24


@pytest.fixture(scope="module")
def L():
    import __graft_entry__ as entry
    entry.build()
    from paper_2505_06653_b200 import binding
    assert torch.cuda.is_available()
    return binding.lib()


def _split(L, static, w, tau, cap, ws):
    """One call through the C ABI; every buffer is allocated here, before the call."""
    from paper_2505_06653_b200 import binding as b
    n = w.numel()
    clean = torch.empty_like(w)
    idx = torch.full((cap,), -1, dtype=torch.int32, device="cuda")
    val = torch.zeros(cap, dtype=torch.bfloat16, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if static:
        rc = L.opq_split_static(w.data_ptr(), b.BF16, n, I, tau, clean.data_ptr(), idx.data_ptr(),
                                val.data_ptr(), cap, cnt.data_ptr(), stream)
    else:
        rc = L.opq_split(w.data_ptr(), b.BF16, n, I, tau, clean.data_ptr(), idx.data_ptr(),
                         val.data_ptr(), cap, cnt.data_ptr(), ws.data_ptr(), ws.numel(), stream)
    assert rc == 0, L.bof4_last_error()
    torch.cuda.synchronize()
    return clean, idx, val, int(cnt.item())


def test_static_scratch_matches_workspace_version_twice_in_a_row(L):
    from paper_2505_06653_b200 import binding as b
    tau = float(np.float32(b.bof4_opq_threshold(0.95, I)))
    # second tensor is smaller and denser in outliers: stale scratch of call 1 must not leak
    cases = [(512 * 300 + 5 * I, 11, 2e-3), (512 * 41 + I, 12, 2e-2)]
    for n, seed, rate in cases:
        w = workloads.inject_outliers(workloads.gaussian(n, 0.02, seed, torch.bfloat16), 0.02, rate,
                                      10.0, 40.0, seed + 1)
        w[512 * 7: 512 * 7 + 30] = 5.0          # more outliers in one tile than a staging slot holds
        wd = w.cuda()
        ws = torch.empty(b.bof4_workspace_bytes(b.OP_OPQ, n, I), dtype=torch.uint8, device="cuda")
        ref = _split(L, False, wd, tau, n, ws)
        got = _split(L, True, wd, tau, n, None)
        assert got[3] == ref[3] and got[3] > 30
        k = ref[3]
        assert torch.equal(got[0], ref[0])                      # cleaned weights, bit for bit
        assert torch.equal(got[1][:k], ref[1][:k])              # outlier indices
        assert torch.equal(got[2][:k].view(torch.int16), ref[2][:k].view(torch.int16))
        assert bool((got[1][k:] == -1).all())                   # nothing written past the count
        # the point of the entry point: with its outputs in place, a call takes no device memory,
        # neither through torch's allocator nor behind its back
        clean = torch.empty_like(wd)
        idx = torch.empty(n, dtype=torch.int32, device="cuda")
        val = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
        stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        free0, used0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        rc = L.opq_split_static(wd.data_ptr(), b.BF16, n, I, tau, clean.data_ptr(), idx.data_ptr(),
                                val.data_ptr(), n, cnt.data_ptr(), stream)
        torch.cuda.synchronize()
        assert rc == 0
        assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == used0
        assert int(cnt.item()) == k


def test_static_entry_point_rejects_oversized_input(L):
    from paper_2505_06653_b200 import binding as b
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: the size check comes first
    rc = L.opq_split_static(fake, b.BF16, MAX_N + I, I, 3.0, None, fake, fake, 8, fake, None)
    assert rc == -2
    assert b"at most" in L.bof4_last_error()
    # whole blocks only: the ragged last block of opq_split is not offered here
    rc = L.opq_split_static(fake, b.BF16, 4 * I + 3, I, 3.0, None, fake, fake, 8, fake, None)
    assert rc == -2
    assert b"multiple" in L.bof4_last_error()
