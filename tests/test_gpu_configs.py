"""GPU parity on the five workload configurations, at the sizes and in the launch configuration
the benchmark times (config 2 at its full 2^26 weights), element by element against the oracle
wherever the oracle finishes in seconds, and on reduced row counts of the same matrices where
it would not (configs 3 and 5)."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

RTOL = 1e-5
LV0 = np.array(workloads.init_levels_7_0_8(), np.float32)


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def bits16(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def test_config1_fit_50_iterations_then_quantize_dequantize_fp32(bof4):
    w = workloads.config1()
    wd = w.cuda()
    cb, log = bof4.bof4_fit_codebook([wd], 64, bof4.NORM_ABS, bof4.METRIC_MSE, LV0, workloads.FIXED_BOF4, 50)
    rcb, rlog = oracle.fit(w, 64, oracle.NORM_ABS, oracle.METRIC_MSE, LV0, workloads.FIXED_BOF4, 50)
    np.testing.assert_allclose(cb.cpu().numpy(), rcb, rtol=RTOL, atol=1e-7)
    np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=RTOL)
    codes, scales = bof4.bof4_quantize(wd, 64, bof4.NORM_ABS, rcb)
    out = bof4.bof4_dequantize(codes, scales, 64, rcb, bof4.F32)
    rc, rs = oracle.quantize(w, 64, oracle.NORM_ABS, rcb)
    assert scales.dtype == torch.float32
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), rs.view(np.uint32))
    assert np.array_equal(out.cpu().numpy().view(np.uint32), oracle.dequantize(rc, rs, 64, rcb).view(np.uint32))


@pytest.fixture(scope="module")
def c2():
    w = workloads.config2()
    return w, w.cuda()


def test_config2_full_size_fit_with_error_log(bof4, c2):
    w, wd = c2
    iters = 4
    cb, log = bof4.bof4_fit_codebook([wd], 64, bof4.NORM_SIGNED, bof4.METRIC_MSE, LV0, workloads.FIXED_BOF4S, iters)
    rcb, rlog = oracle.fit(w, 64, oracle.NORM_SIGNED, oracle.METRIC_MSE, LV0, workloads.FIXED_BOF4S, iters)
    np.testing.assert_allclose(cb.cpu().numpy(), rcb, rtol=RTOL, atol=1e-7)
    np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=RTOL)
    assert np.all(np.diff(log.cpu().numpy()) < 0)


def test_config2_full_size_mae_step(bof4, c2):
    w, wd = c2
    got = bof4.bof4_em_step([wd], 64, bof4.NORM_SIGNED, bof4.METRIC_MAE, LV0)
    ref = oracle.em_accumulate_mae(w, 64, oracle.NORM_SIGNED, LV0)
    assert np.array_equal(got["count"], ref["count"])
    assert np.array_equal(got["median"], ref["median"])
    np.testing.assert_allclose(got["s0"], ref["wsum"], rtol=RTOL)
    np.testing.assert_allclose(got["err_sum"], ref["err_sum"], rtol=RTOL)


def test_config2_full_size_opq_quantize_dequantize(bof4, c2):
    """The benchmark's quantise / dequantise legs, same sizes and buffers."""
    w, wd = c2
    n = w.numel()
    lv = LV0
    tau = float(np.float32(bof4.bof4_opq_threshold(0.95, 64)))
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(wd, 64, bof4.NORM_SIGNED, lv, tau, n // 64)
    out = bof4.bof4_dequantize(codes, scales, 64, lv, bof4.BF16, (idx, val, cnt))
    clean, ridx, rval, rk = oracle.opq_split(w, 64, tau)
    k = int(cnt.item())
    assert k == rk and k <= n // 64
    assert np.array_equal(idx[:k].cpu().numpy().astype(np.int64), ridx)
    assert np.array_equal(bits16(val[:k]), rval)
    rc, rs = oracle.quantize(clean, 64, oracle.NORM_SIGNED, lv)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(scales.float().cpu().numpy(), rs)
    rout = oracle.opq_restore(oracle.dequantize(rc, rs, 64, lv), ridx, rval)
    assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(rout))


@pytest.mark.parametrize("I", [32, 64, 128, 256])
@pytest.mark.parametrize("norm,mask", [(0, workloads.FIXED_BOF4), (1, workloads.FIXED_BOF4S)])
@pytest.mark.parametrize("metric", [0, 1])
def test_config3_sweep_on_reduced_rows(bof4, I, norm, mask, metric):
    """One layer (7 matrices, per-matrix sigma) with 1/16 of the rows; one codebook over the union."""
    mats = [m for _, m in workloads.config3_matrices(row_divisor=16, layers=1)]
    iters = 3
    cb, log = bof4.bof4_fit_codebook([m.cuda() for m in mats], I, norm, metric, LV0, mask, iters)
    rcb, rlog = oracle.fit(torch.cat(mats), I, norm, metric, LV0, mask, iters)
    np.testing.assert_allclose(cb.cpu().numpy(), rcb, rtol=RTOL, atol=1e-7)
    np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=RTOL)


def test_config4_one_layer_full_size(bof4):
    """Every distinct matrix shape of a layer, full size, BOF4-S codebook of Tab. 6."""
    lv = np.array([-0.8568463921546936, -0.6692874431610107, -0.5235266089439392, -0.4004882574081421,
                   -0.2910638153553009, -0.1900092959403992, -0.0938529595732689, 0.0,
                   0.0887671709060669, 0.1794802695512772, 0.2743096053600311, 0.3760197460651398,
                   0.4886530041694641, 0.6188603639602661, 0.7791395783424377, 1.0], np.float32)
    seen = set()
    for i, m in workloads.config4_matrices(layers=1):
        if m.numel() in seen:
            continue
        seen.add(m.numel())
        codes, scales = bof4.bof4_quantize(m.cuda(), 64, bof4.NORM_SIGNED, lv)
        out = bof4.bof4_dequantize(codes, scales, 64, lv, bof4.BF16)
        rc, rs = oracle.quantize(m, 64, oracle.NORM_SIGNED, lv)
        assert np.array_equal(codes.cpu().numpy(), rc)
        assert np.array_equal(scales.float().cpu().numpy(), rs)
        assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(oracle.dequantize(rc, rs, 64, lv)))


def test_config5_layer_on_reduced_rows(bof4):
    """The seven matrices of a 70B-shaped layer with 1/8 of the rows: fused OPQ quantise and
    dequantise with outlier write-back."""
    tau = float(np.float32(bof4.bof4_opq_threshold(0.95, 64)))
    lv = LV0
    for m in workloads.config5_layer(0, row_divisor=8):
        n = m.numel()
        codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(m.cuda(), 64, bof4.NORM_SIGNED, lv, tau, n // 32)
        out = bof4.bof4_dequantize(codes, scales, 64, lv, bof4.BF16, (idx, val, cnt))
        clean, ridx, rval, rk = oracle.opq_split(m, 64, tau)
        k = int(cnt.item())
        assert k == rk
        assert np.array_equal(idx[:k].cpu().numpy().astype(np.int64), ridx)
        assert np.array_equal(bits16(val[:k]), rval)
        rc, rs = oracle.quantize(clean, 64, oracle.NORM_SIGNED, lv)
        assert np.array_equal(codes.cpu().numpy(), rc)
        rout = oracle.opq_restore(oracle.dequantize(rc, rs, 64, lv), ridx, rval)
        assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(rout))
        frac = k / n
        assert 2e-4 < frac < 3e-3   # Gaussian tail beyond tau plus the injected 1e-4


def test_config5_largest_matrix_full_size(bof4):
    """The 28672 x 8192 matrix of a 70B-shaped layer at full size (2.3e8 weights, 459 chunks of
    the ordered compaction): fused OPQ quantise and dequantise against the oracle."""
    r, c = workloads.llama70b_layer_shapes()[4]
    s = 4_000_000 + 4
    w = workloads.gaussian(r * c, 0.015, s, torch.bfloat16)
    w = workloads.inject_outliers(w, 0.015, 1e-4, 10.0, 40.0, s + 8)
    n = w.numel()
    tau = float(np.float32(bof4.bof4_opq_threshold(0.95, 64)))
    cap = n // 256
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(w.cuda(), 64, bof4.NORM_SIGNED, LV0, tau, cap)
    out = bof4.bof4_dequantize(codes, scales, 64, LV0, bof4.BF16, (idx, val, cnt))
    clean, ridx, rval, rk = oracle.opq_split(w, 64, tau)
    k = int(cnt.item())
    assert k == rk and k <= cap
    assert np.array_equal(idx[:k].cpu().numpy().astype(np.int64), ridx)
    assert np.array_equal(bits16(val[:k]), rval)
    rc, rs = oracle.quantize(clean, 64, oracle.NORM_SIGNED, LV0)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(scales.float().cpu().numpy(), rs)
    rout = oracle.opq_restore(oracle.dequantize(rc, rs, 64, LV0), ridx, rval)
    assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(rout))
