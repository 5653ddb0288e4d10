"""Tensors that do not end on a block boundary: bof4_quantize, bof4_dequantize, opq_split and
bof4_quantize_opq treat the last, shorter block as a block of its own (the paper only uses whole
blocks; the reading is stated in the header and pinned in the oracle).  Bit-exact as everywhere."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

LV = np.array(workloads.init_levels_7_0_8(), np.float32)


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _weights(n, dtype, seed, tail_start):
    w = workloads.gaussian_student_mixture(n, 0.02, 0.02, 3, seed, dtype)
    if n - tail_start >= 3:
        w[tail_start + 1] = 0.9          # an outlier inside the short block
    if tail_start >= 8:
        w[3] = -0.7                      # and one in the whole blocks
    return w


CASES = [(I, whole, tail) for I in (32, 64, 256, 1024, 4096) for whole in (0, 1, 5)
         for tail in (1, 2, 15, 16, 17, 31, I // 2 + 3, I - 1)]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("norm", [0, 1])
def test_ragged_quantize_dequantize(bof4, dtype, norm):
    for I, whole, tail in CASES:
        n = whole * I + tail
        w = _weights(n, dtype, 500 + I + tail, whole * I)
        codes, scales = bof4.bof4_quantize(w.cuda(), I, norm, LV)
        rc, rs = oracle.quantize(w, I, norm, LV)
        tag = "I=%d whole=%d tail=%d" % (I, whole, tail)
        assert codes.numel() == (n + 1) // 2 and scales.numel() == whole + 1, tag
        assert np.array_equal(codes.cpu().numpy(), rc), tag
        assert np.array_equal(scales.float().cpu().numpy(), rs), tag
        for out_dtype in (bof4.BF16, bof4.F32):
            out = bof4.bof4_dequantize(codes, scales, I, LV, out_dtype, n=n)
            ref = oracle.dequantize(rc, rs, I, LV, n=n)
            if out_dtype == bof4.BF16:
                assert np.array_equal(_bits(out), oracle.f32_to_bf16_bits(ref)), tag
            else:
                assert np.array_equal(out.cpu().numpy(), ref), tag


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_ragged_opq(bof4, dtype):
    for I, whole, tail in CASES:
        n = whole * I + tail
        w = _weights(n, dtype, 900 + I + tail, whole * I)
        tau = float(np.float32(bof4.bof4_opq_threshold(0.9, I)))
        tag = "I=%d whole=%d tail=%d" % (I, whole, tail)
        rclean, ridx, rval, rk = oracle.opq_split(w, I, tau)
        clean, idx, val, cnt = bof4.opq_split(w.cuda(), I, tau, n)
        k = int(cnt.item())
        assert k == rk, tag
        assert np.array_equal(idx[:k].cpu().numpy().astype(np.int64), ridx), tag
        assert np.array_equal(_bits(val[:k]), rval), tag
        assert np.array_equal(clean.float().cpu().numpy(), rclean), tag
        for norm in (0, 1):
            codes, scales, idx2, val2, cnt2 = bof4.bof4_quantize_opq(w.cuda(), I, norm, LV, tau, n)
            rc, rs = oracle.quantize(rclean, I, norm, LV)
            assert int(cnt2.item()) == rk, tag
            assert np.array_equal(idx2[:rk].cpu().numpy().astype(np.int64), ridx), tag
            assert np.array_equal(codes.cpu().numpy(), rc), tag
            assert np.array_equal(scales.float().cpu().numpy(), rs), tag
            out = bof4.bof4_dequantize(codes, scales, I, LV, bof4.BF16, (idx2, val2, cnt2), n=n)
            ref = oracle.opq_restore(oracle.dequantize(rc, rs, I, LV, n=n), ridx, rval)
            assert np.array_equal(_bits(out), oracle.f32_to_bf16_bits(ref)), tag


def test_ragged_outlier_list_capacity(bof4):
    """The short block's outliers come after those of the whole blocks; the count stays exact
    when the list is too small for them."""
    I, whole, tail = 64, 4, 40
    n = whole * I + tail
    w = workloads.gaussian(n, 0.02, 7, torch.float32)
    w[[5, 70, 200]] = 1.0
    w[[whole * I + 2, whole * I + 30]] = -1.0
    tau = 3.0
    _, ridx, rval, rk = oracle.opq_split(w, I, tau)
    assert rk >= 5 and (ridx >= whole * I).sum() >= 2
    cap = int((ridx < whole * I).sum()) + 1          # room for one of the short block's outliers only
    _, idx, val, cnt = bof4.opq_split(w.cuda(), I, tau, cap)
    assert int(cnt.item()) == rk
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), ridx[:cap])
    assert np.array_equal(_bits(val), rval[:cap])


def test_fit_still_needs_whole_blocks(bof4):
    w = torch.zeros(100, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bof4.Bof4Error) as e:
        bof4.bof4_em_step([w], 64, 0, bof4.METRIC_MSE, LV)
    assert e.value.code == -2
