"""Tensors that do not end on a block boundary: bof4_quantize, bof4_dequantize, opq_split,
bof4_quantize_opq and the codebook fit treat the last, shorter block as a block of its own (the paper only uses whole
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


# --------------------------------------------------------------------------- ragged tensors in the fit

RTOL = 1e-5


def _ragged_list(I, dtype, seed, lens):
    out = []
    for k, n in enumerate(lens):
        w = workloads.gaussian_student_mixture(max(n, 1), 0.02 * (1 + k % 3), 0.02, 3, seed + k, dtype)[:n].clone()
        if n % I >= 2:
            w[n - 1] = -0.5 if k % 2 else 0.5            # the short block's maximum is its own
        out.append(w.contiguous())
    return out


def _check_stats(got, ref_mse, ref_mae, metric, lv):
    if metric in (0, 2):
        assert np.array_equal(got["count"], ref_mse["count"])
        np.testing.assert_allclose(got["s1"], ref_mse["s1"], rtol=RTOL, atol=1e-6 * np.abs(ref_mse["s1"]).max())
        np.testing.assert_allclose(got["s0"], ref_mse["s0"], rtol=RTOL)
        np.testing.assert_allclose(got["err_sum"], ref_mse["err_sum"], rtol=RTOL)
        assert got["n"] == ref_mse["n"]
    else:
        assert np.array_equal(got["count"], ref_mae["count"])
        assert np.array_equal(got["median"], ref_mae["median"])
        np.testing.assert_allclose(got["s0"], ref_mae["wsum"], rtol=RTOL)
        np.testing.assert_allclose(got["err_sum"], ref_mae["err_sum"], rtol=RTOL)


EM_LENS = [
    lambda I: [5 * I + 7],
    lambda I: [I - 1],
    lambda I: [1, 2],                                   # no whole block anywhere
    lambda I: [3 * I, 2 * I + 1, 0, I // 2, 4 * I + I - 1, 1],
    lambda I: [40 * I + 3 + k for k in range(70)],      # more short blocks than one launch's table holds
]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("norm", [0, 1])
@pytest.mark.parametrize("metric", [0, 1, 2, 3])
def test_em_step_on_ragged_tensor_lists(bof4, dtype, norm, metric):
    """bof4_em_step over tensors whose lengths are not multiples of the block size: the short last
    block of every tensor is a block of its own, in the sums (MSE) as in the weighted medians
    (MAE), for both weight-domain and normalised-domain variants."""
    for I in (32, 64, 1024, 4096):
        for make in EM_LENS:
            ws = _ragged_list(I, dtype, 40 + I, make(I))
            got = bof4.bof4_em_step([w.cuda() for w in ws], I, norm, metric, LV)
            ref_mse = oracle.em_accumulate_mse(ws, I, norm, LV, normdom=metric == 2) if metric in (0, 2) else None
            ref_mae = oracle.em_accumulate_mae(ws, I, norm, LV, normdom=metric == 3) if metric in (1, 3) else None
            _check_stats(got, ref_mse, ref_mae, metric, LV)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("metric", [0, 1])
def test_em_step_ragged_over_many_rows(bof4, dtype, metric):
    """Several rows per CTA of whole blocks plus short blocks: both kernels' contributions land
    in the same statistics."""
    I = 64
    ws = _ragged_list(I, dtype, 77, [148 * 32768 * 2 + 64 * 11 + 37, (1 << 20) + 5, 63])
    got = bof4.bof4_em_step([w.cuda() for w in ws], I, 1, metric, LV)
    ref_mse = oracle.em_accumulate_mse(ws, I, 1, LV) if metric == 0 else None
    ref_mae = oracle.em_accumulate_mae(ws, I, 1, LV) if metric == 1 else None
    _check_stats(got, ref_mse, ref_mae, metric, LV)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("norm,mask", [(0, workloads.FIXED_BOF4), (1, workloads.FIXED_BOF4S)])
@pytest.mark.parametrize("metric", [0, 1])
def test_fit_on_ragged_tensor_lists(bof4, dtype, norm, mask, metric):
    I = 64
    ws = _ragged_list(I, dtype, 91, [3000 * I + 17, 41, 2000 * I, 555 * I + 63])
    cb, log = bof4.bof4_fit_codebook([w.cuda() for w in ws], I, norm, metric, LV, mask, 8)
    rcb, rlog = oracle.fit(ws, I, norm, metric, LV, mask, 8)
    np.testing.assert_allclose(cb.cpu().numpy(), rcb, rtol=RTOL, atol=1e-7)
    np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=RTOL)


def test_mae_ragged_with_late_candidate_collection(bof4):
    """The smallest workspace moves the candidate collection of a 2^26-weight fit one pass back;
    the short blocks' samples must reach the lists in that pass too."""
    from paper_2505_06653_b200 import binding as b
    I = 64
    ws = _ragged_list(I, torch.bfloat16, 303, [(1 << 26) + (1 << 16) + 33, 31])
    ref = oracle.em_accumulate_mae(ws, I, 1, LV)
    small = torch.empty(b.bof4_workspace_bytes(b.OP_EM, 0, I, b.METRIC_MAE), dtype=torch.uint8, device="cuda")
    got = bof4.bof4_em_step([w.cuda() for w in ws], I, 1, bof4.METRIC_MAE, LV, workspace=small)
    _check_stats(got, None, ref, 1, LV)
