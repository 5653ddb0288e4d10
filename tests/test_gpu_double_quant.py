"""Double quantisation of the block constants (Limitations; App. F) against its definition in
oracle/double_quant.py: codes, group constants, sign bits and reconstructed constants bit for
bit, and the decoders (dequantise, matrix-vector product) fed with the reconstructed constants."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from oracle import double_quant as dq

pytestmark = pytest.mark.gpu

LV = np.array(workloads.BOF4S_MSE_I64, np.float32)


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def _constants(B, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    m = (torch.randn(B, generator=g).abs() * 0.05 + 0.003) * (torch.randint(0, 2, (B,), generator=g) * 2 - 1)
    if B > 600:
        m[256:512] *= 300.0            # a group on another scale
        m[520:530] = 0.0
    if B > 4:
        m[3] = -m[3].abs()
    return m.to(dtype).contiguous()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("norm", [0, 1])
def test_compress_expand_match_the_definition(bof4, dtype, norm):
    for B in (1, 7, 8, 9, 255, 256, 257, 1000, 256 * 1500 + 77):
        m = _constants(B, dtype, 60 + B % 97)
        if norm == 0:
            m = m.abs()
        q, g, sign = bof4.bof4_scales_compress(m.cuda(), norm)
        rq, rg, rs = dq.compress(m.float().numpy(), norm == 1)
        assert np.array_equal(q.cpu().numpy(), rq), B
        assert np.array_equal(g.cpu().numpy(), rg), B
        if norm == 1:
            assert np.array_equal(sign.cpu().numpy(), rs), B
        else:
            assert sign is None
        mh = bof4.bof4_scales_expand(q, g, sign)
        assert np.array_equal(mh.cpu().numpy(), dq.expand(rq, rg, rs, B)), B


def test_zero_group_and_empty_input(bof4):
    z = torch.zeros(300, dtype=torch.float32, device="cuda")
    q, g, sign = bof4.bof4_scales_compress(z, 1)
    assert not q.any() and not g.any() and not sign.any()
    assert not bof4.bof4_scales_expand(q, g, sign).any()
    e = torch.zeros(0, dtype=torch.float32, device="cuda")
    q, g, sign = bof4.bof4_scales_compress(e, 0)
    assert q.numel() == 0 and g.numel() == 0


@pytest.mark.parametrize("norm", [0, 1])
def test_decoders_read_the_reconstructed_constants(bof4, norm):
    """Quantise with exact constants, double-quantise them, decode with m^: the dequantised
    tensor and the fused matrix-vector product must be the oracle's with the oracle's m^."""
    I, rows, cols = 64, 96, 4096
    w = workloads.gaussian_student_mixture(rows * cols, 0.02, 0.02, 3, 71, torch.bfloat16)
    codes, scales = bof4.bof4_quantize(w.cuda(), I, norm, LV)
    q, g, sign = bof4.bof4_scales_compress(scales, norm)
    mh = bof4.bof4_scales_expand(q, g, sign)
    rc, rm = oracle.quantize(w, I, norm, LV)
    rmh = dq.expand(*dq.compress(rm, norm == 1), rm.size)
    assert np.array_equal(mh.cpu().numpy(), rmh)
    out = bof4.bof4_dequantize(codes, mh, I, LV, bof4.BF16)
    ref = oracle.dequantize(rc, rmh, I, LV)
    assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), oracle.f32_to_bf16_bits(ref))
    x = workloads.gaussian(cols, 1.0, 72, torch.float32)
    y = bof4.bof4_gemv(codes, mh, rows, cols, I, LV, x.cuda())
    yr, mag = oracle.gemv(rc, rmh, rows, cols, I, LV, x.numpy())
    assert np.all(np.abs(y.cpu().numpy() - yr) <= 1e-5 * mag + 1e-30)
