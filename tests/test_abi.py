"""CPU-only checks of the C ABI: the library loads, exports every declared symbol, and the
host-side logic (argument validation, workspace sizes, host helpers) behaves as documented.
No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

import __graft_entry__ as entry
import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    entry.build()
    from paper_2505_06653_b200 import binding
    return binding.lib()


def _declared():
    src = open(os.path.join(ROOT, "include", "bof4.h")).read()
    return sorted(set(re.findall(r"^BOF4_API\s+[\w\s\*]+?\b(\w+)\s*\(", src, flags=re.M)))


def test_every_declared_symbol_is_exported(L):
    from paper_2505_06653_b200 import binding
    names = _declared()
    assert len(names) >= 10
    for name in names:
        assert hasattr(L, name), name
    assert sorted(binding.EXPORTS) == names


def test_stats_struct_size_matches_header(L):
    from paper_2505_06653_b200 import binding
    assert ctypes.sizeof(binding.EmStats) == 16 * 8 * 3 + 8 + 8 + 16 * 4


def test_opq_threshold_matches_quantile_definition(L):
    # F_M(tau) = (2 G(tau) - 1)^I = q  (App. B.1), checked through the forward formula
    from scipy.special import ndtr
    for I in (32, 64, 128, 256):
        for q in (0.9, 0.95, 0.97, 0.99):
            tau = L.bof4_opq_threshold(q, I)
            assert abs((2 * ndtr(tau) - 1) ** I - q) < 1e-12
            assert abs(tau - oracle.opq_threshold(q, I)) < 1e-10
    assert np.isnan(L.bof4_opq_threshold(1.5, 64))
    assert np.isnan(L.bof4_opq_threshold(0.5, 0))


def test_default_init(L):
    from paper_2505_06653_b200 import binding
    lv, mask = binding.bof4_default_init(binding.NORM_ABS)
    assert mask == (1 | 1 << 7 | 1 << 15)
    assert lv[0] == -1 and lv[7] == 0 and lv[15] == 1 and np.all(np.diff(lv) > 0)
    lv, mask = binding.bof4_default_init(binding.NORM_SIGNED)
    assert mask == (1 << 7 | 1 << 15)
    with pytest.raises(binding.Bof4Error):
        binding.bof4_default_init(7)


def test_workspace_sizes(L):
    from paper_2505_06653_b200 import binding as b
    assert b.bof4_workspace_bytes(b.OP_EM, 1 << 20, 64, b.METRIC_MSE) > 0
    assert b.bof4_workspace_bytes(b.OP_EM, 1 << 20, 64, 5) == 0
    assert b.bof4_workspace_bytes(b.OP_OPQ, 1 << 20, 48, 0) == 0
    assert b.bof4_workspace_bytes(b.OP_OPQ, 1 << 20, 8192, 0) == 0
    assert b.bof4_workspace_bytes(b.OP_OPQ, 1 << 20, 4096, 0) > 0
    assert b.bof4_workspace_bytes(9, 1 << 20, 64, 0) == 0
    small = b.bof4_workspace_bytes(b.OP_OPQ, 1 << 20, 64, 0)
    big = b.bof4_workspace_bytes(b.OP_OPQ, 1 << 24, 64, 0)
    assert 0 < small < big
    assert b.bof4_workspace_bytes(b.OP_OPQ, 0, 64, 0) >= 256


def test_argument_validation_happens_before_any_cuda_call(L):
    """Bad shapes / dtypes / pointers are rejected on the host with the documented codes."""
    from paper_2505_06653_b200 import binding as b
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: validation fails first
    # block size and divisibility
    assert L.bof4_quantize(fake, b.BF16, 128, 48, 0, fake, fake, fake, b.BF16, None) == -2
    assert L.bof4_quantize(fake, b.BF16, 128, 8192, 0, fake, fake, fake, b.BF16, None) == -2
    assert L.bof4_quantize(fake, b.BF16, -64, 64, 0, fake, fake, fake, b.BF16, None) == -1
    # dtypes: unknown, and fp32 weights with bf16 scales
    assert L.bof4_quantize(fake, 3, 128, 64, 0, fake, fake, fake, b.BF16, None) == -3
    assert L.bof4_quantize(fake, b.F32, 128, 64, 0, fake, fake, fake, b.BF16, None) == -3
    assert L.bof4_quantize(fake, b.BF16, 128, 64, 2, fake, fake, fake, b.BF16, None) == -1
    assert L.bof4_quantize(None, b.BF16, 128, 64, 0, fake, fake, fake, b.BF16, None) == -1
    # dequantise
    assert L.bof4_dequantize(fake, fake, b.BF16, 96, 24, fake, None, None, None, 0, fake, b.BF16, None) == -2
    assert L.bof4_dequantize(fake, fake, 9, 128, 64, fake, None, None, None, 0, fake, b.BF16, None) == -3
    assert L.bof4_dequantize(fake, fake, b.BF16, 128, 64, fake, fake, None, None, 4, fake, b.BF16, None) == -1
    assert L.bof4_dequantize(fake, fake, b.BF16, 128, 64, fake, fake, fake, fake, -1, fake, b.BF16, None) == -5
    # OPQ: size limit, capacity, workspace
    ws = ctypes.c_void_p(0x10000)
    assert L.opq_split(fake, b.BF16, 1 << 31, 64, 3.0, None, fake, fake, 8, fake, ws, 1 << 40, None) == -2
    assert L.opq_split(fake, b.BF16, 128, 64, 3.0, None, fake, fake, -1, fake, ws, 1 << 40, None) == -5
    assert L.opq_split(fake, b.BF16, 128, 64, 3.0, None, fake, fake, 8, fake, None, 1 << 40, None) == -4
    assert L.opq_split(fake, b.BF16, 128, 64, 3.0, None, fake, fake, 8, fake, ws, 16, None) == -4
    assert L.opq_split(fake, b.BF16, 128, 64, 3.0, None, fake, fake, 8, fake, ctypes.c_void_p(0x10010), 1 << 40, None) == -4
    assert L.opq_split(fake, b.BF16, 128, 64, -1.0, None, fake, fake, 8, fake, ws, 1 << 40, None) == -1
    # the synchronising count check rejects bad arguments before touching the device
    assert L.bof4_outlier_count(None, 8, None, None) == -1
    assert L.bof4_outlier_count(fake, -1, None, None) == -1
    # EM
    ptrs = (ctypes.c_void_p * 1)(0x1000)
    ns = (ctypes.c_int64 * 1)(100)
    assert L.bof4_em_step(ptrs, ns, 1, b.BF16, 48, 0, 0, fake, fake, ws, 1 << 40, None) == -2   # block size
    ns[0] = -1
    assert L.bof4_em_step(ptrs, ns, 1, b.BF16, 64, 0, 0, fake, fake, ws, 1 << 40, None) == -1
    ns[0] = 100                      # a ragged length is accepted; the small workspace is refused next
    assert L.bof4_em_step(ptrs, ns, 1, b.BF16, 64, 0, 0, fake, fake, ws, 8, None) == -4
    assert L.bof4_em_step(ptrs, ns, 1, b.BF16, 64, 0, 4, fake, fake, ws, 1 << 40, None) == -1
    assert L.bof4_em_step(ptrs, ns, 1, 7, 64, 0, 0, fake, fake, ws, 1 << 40, None) == -3
    assert L.bof4_fit_codebook(ptrs, ns, 1, b.BF16, 64, 0, 0, fake, 0, -1, None, ws, 1 << 40, None) == -1
    assert L.bof4_fit_codebook(ptrs, ns, 1, b.BF16, 64, 0, 0, None, 0, 1, None, ws, 1 << 40, None) == -1
    # fused matrix-vector product: shape, dtype, outlier-list and alignment rules
    gv = lambda *a: L.bof4_gemv(*a)
    assert gv(fake, fake, b.BF16, 4, 96, 64, fake, fake, b.BF16, None, None, None, 0, fake, None) == -2
    assert gv(fake, fake, b.BF16, 4, 65536, 64, fake, fake, b.BF16, None, None, None, 0, fake, None) == -2
    assert gv(fake, fake, b.BF16, -1, 64, 64, fake, fake, b.BF16, None, None, None, 0, fake, None) == -1
    assert gv(fake, fake, 5, 4, 64, 64, fake, fake, b.BF16, None, None, None, 0, fake, None) == -3
    assert gv(fake, fake, b.BF16, 4, 64, 64, fake, fake, b.BF16, fake, None, None, 4, fake, None) == -1
    assert gv(fake, fake, b.BF16, 4, 64, 64, fake, fake, b.BF16, fake, fake, fake, -1, fake, None) == -5
    assert gv(fake, fake, b.BF16, 1 << 20, 4096, 64, fake, fake, b.BF16, fake, fake, fake, 4, fake, None) == -2
    assert gv(fake, fake, b.BF16, 4, 64, 64, fake, ctypes.c_void_p(0x1008), b.BF16, None, None, None, 0, fake, None) == -1
    assert b"aligned" in L.bof4_last_error()
    assert gv(ctypes.c_void_p(0x1010), fake, b.BF16, 4, 64, 64, fake, fake, b.BF16, None, None, None, 0, fake, None) == -1
    assert gv(fake, fake, b.BF16, 4, 64, 64, fake, fake, b.BF16, None, None, None, 0, None, None) == -1
    assert gv(None, None, b.BF16, 0, 64, 64, None, None, b.BF16, None, None, None, 0, None, None) == 0
    # theoretical codebook: the outermost levels must be fixed, metric MSE / MAE only
    full = (1 << 0) | (1 << 7) | (1 << 15)
    assert L.bof4_theoretical_codebook(64, 0, 0, fake, 1 << 15, 1, ws, 256, None) == -1   # -1 not fixed (abs)
    assert L.bof4_theoretical_codebook(64, 1, 0, fake, 1 << 7, 1, ws, 256, None) == -1    # +1 not fixed
    assert L.bof4_theoretical_codebook(64, 0, 2, fake, full, 1, ws, 256, None) == -1
    assert L.bof4_theoretical_codebook(1, 0, 0, fake, full, 1, ws, 256, None) == -2
    assert L.bof4_theoretical_codebook(64, 0, 0, fake, full, 1, ws, 8, None) == -4
    one = lambda v, t=ctypes.c_int: (t * 1)(v)
    batch = L.bof4_theoretical_codebook_batch
    assert batch(129, one(64), one(0), one(0), one(full, ctypes.c_uint32), fake, 1, ws, 1 << 20, None) == -2
    assert batch(1, one(64), one(0), one(0), one(1 << 15, ctypes.c_uint32), fake, 1, ws, 256, None) == -1
    assert batch(1, one(64), one(0), one(0), one(full, ctypes.c_uint32), fake, 1, ws, 128, None) == -4
    assert batch(1, None, one(0), one(0), one(full, ctypes.c_uint32), fake, 1, ws, 256, None) == -1
    assert batch(0, None, None, None, None, None, 1, None, 0, None) == 0


def test_binding_refuses_cpu_tensors(L):
    import torch
    from paper_2505_06653_b200 import binding as b
    with pytest.raises(ValueError, match="no CPU path"):
        b.bof4_quantize(torch.zeros(64), 64, 0, np.linspace(-1, 1, 16))


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2505_06653_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in txt, os.path.join(dirpath, f)
