"""Tensors beyond 2^32 elements: every index on the path is 64-bit.  One 2^32 + 192-element bf16
tensor (64 copies of a 2^26-element chunk and a short tail) is quantised, dequantised and passed
through both fit passes; codes and constants are compared with the oracle on slices around the
2^31 and 2^32 element marks and at both ends, the fit statistics with 64 times the oracle's
statistics of the chunk (blocks do not span chunk boundaries, so the sums are exact multiples)."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

LV = np.array(workloads.BOF4S_MSE_I64, np.float32)
I = 64


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def test_quantise_dequantise_and_fit_beyond_four_giga_elements(bof4):
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GB of free device memory")
    chunk = workloads.gaussian_student_mixture(1 << 26, 0.02, 0.01, 4, 91, torch.bfloat16)
    tail = workloads.gaussian(192, 0.05, 92, torch.bfloat16)
    n = 64 * chunk.numel() + tail.numel()
    w = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    cd = chunk.cuda()
    for k in range(64):
        w[k * chunk.numel():(k + 1) * chunk.numel()] = cd
    w[64 * chunk.numel():] = tail.cuda()
    codes, scales = bof4.bof4_quantize(w, I, 1, LV)
    out = bof4.bof4_dequantize(codes, scales, I, LV, bof4.BF16)
    assert codes.numel() == n // 2 and scales.numel() == n // I and out.numel() == n
    rc, rs = oracle.quantize(chunk, I, 1, LV)
    rd = oracle.f32_to_bf16_bits(oracle.dequantize(rc, rs, I, LV))
    span = 1 << 16                                           # elements checked at each position
    for start in (0, (1 << 31) - span, 1 << 31, (1 << 32) - span):
        off = start % chunk.numel()
        assert np.array_equal(codes[start // 2:(start + span) // 2].cpu().numpy(), rc[off // 2:(off + span) // 2]), start
        assert np.array_equal(scales[start // I:(start + span) // I].float().cpu().numpy(), rs[off // I:(off + span) // I]), start
        got = out[start:start + span].view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got, rd[off:off + span]), start
    tc, ts = oracle.quantize(tail, I, 1, LV)                 # the last three blocks, past 2^32
    assert np.array_equal(codes[(1 << 32) // 2:].cpu().numpy(), tc)
    assert np.array_equal(scales[(1 << 32) // I:].float().cpu().numpy(), ts)
    del codes, scales, out
    # fit passes: 64 x the chunk's statistics + the tail's
    st_c = oracle.em_accumulate_mse(chunk, I, 1, LV)
    st_t = oracle.em_accumulate_mse(tail, I, 1, LV)
    got = bof4.bof4_em_step([w], I, 1, bof4.METRIC_MSE, LV)
    assert got["n"] == n
    assert np.array_equal(got["count"], 64 * st_c["count"] + st_t["count"])
    np.testing.assert_allclose(got["s0"], 64 * st_c["s0"] + st_t["s0"], rtol=1e-5)
    np.testing.assert_allclose(got["s1"], 64 * st_c["s1"] + st_t["s1"], rtol=1e-5,
                               atol=1e-6 * np.abs(64 * st_c["s1"]).max())
    np.testing.assert_allclose(got["err_sum"], 64 * st_c["err_sum"] + st_t["err_sum"], rtol=1e-5)
    # The weighted median of 64 copies of a multiset is that of one copy; the 192 extra samples can
    # move a crossing by a few samples at most.  Counts and weights exactly, medians against the
    # chunk's with that allowance.
    ma = oracle.em_accumulate_mae(chunk, I, 1, LV)
    mt = oracle.em_accumulate_mae(tail, I, 1, LV)
    gm = bof4.bof4_em_step([w], I, 1, bof4.METRIC_MAE, LV)
    assert np.array_equal(gm["count"], 64 * ma["count"] + mt["count"])
    np.testing.assert_allclose(gm["s0"], 64 * ma["wsum"] + mt["wsum"], rtol=1e-5)
    np.testing.assert_allclose(gm["err_sum"], 64 * ma["err_sum"] + mt["err_sum"], rtol=1e-5)
    same = gm["median"] == ma["median"]
    assert same.sum() >= 14, (gm["median"], ma["median"])     # at most the tail's few samples can shift a crossing
    assert np.all(np.abs(gm["median"] - ma["median"]) < 1e-4)
