"""Fits at the iteration counts the workload configurations specify, and inputs aimed at the
places where the kernels' arithmetic differs most from the oracle's: many fused M steps in a
row, block constants spread over many binades (fixed-point weights of the median selection),
and a huge block at the start of an fp32 accumulation window."""
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


def _check_fit(bof4, mats, I, norm, metric, mask, iters):
    cb, log = bof4.bof4_fit_codebook([m.cuda() for m in mats], I, norm, metric, LV0, mask, iters)
    rcb, rlog = oracle.fit(torch.cat(mats), I, norm, metric, LV0, mask, iters)
    cb, log = cb.cpu().numpy(), log.cpu().numpy()
    np.testing.assert_allclose(cb, rcb, rtol=RTOL, atol=1e-7)
    np.testing.assert_allclose(log, rlog, rtol=RTOL)        # every entry of the error log
    assert np.all(np.diff(log) <= 1e-12 * log[0])            # Lloyd never increases the error
    for l in range(16):
        if (mask >> l) & 1:
            assert cb[l] == LV0[l]
    return cb, log


def test_config2_full_size_100_iterations(bof4):
    """BOF4-S, 2^26 bf16 weights, MSE, 100 iterations with the error log: the whole run of the
    second workload configuration, every level and every log entry within 1e-5."""
    w = workloads.config2()
    _check_fit(bof4, [w], 64, 1, 0, workloads.FIXED_BOF4S, 100)


@pytest.mark.parametrize("metric", [0, 1])
@pytest.mark.parametrize("norm,mask", [(0, workloads.FIXED_BOF4), (1, workloads.FIXED_BOF4S)])
def test_config3_recipe_30_iterations_on_reduced_rows(bof4, norm, mask, metric):
    """The fitting sweep's 30 iterations (MSE and MAE) over the union of one layer's seven
    matrices with 1/8 of the rows (2.7e7 weights), through the multi-tensor call."""
    mats = [m for _, m in workloads.config3_matrices(row_divisor=8, layers=1)]
    _check_fit(bof4, mats, 64, norm, metric, mask, 30)


# --------------------------------------------------------------------------- wide dynamic range


def _spread_blocks(n_blocks, I, dtype, seed, octaves):
    """Gaussian blocks whose scale falls by powers of two from 1 down to 2^-octaves (cyclically),
    so that block constants lie up to `octaves` binades below the largest magnitude of the data."""
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(n_blocks, I, generator=g, dtype=torch.float32)
    e = -(torch.arange(n_blocks) % (octaves + 1)).float()
    return (x * torch.exp2(e)[:, None]).to(dtype).reshape(-1).contiguous()


@pytest.mark.parametrize("dtype,octaves", [(torch.float32, 10), (torch.float32, 35), (torch.bfloat16, 25),
                                           (torch.bfloat16, 40)])
@pytest.mark.parametrize("norm", [0, 1])
def test_mae_medians_with_block_constants_far_below_the_largest_weight(bof4, dtype, octaves, norm):
    """The median selection weighs a sample by |m| held as a 31-bit fixed-point number below
    the largest |w| of the data: exact down to 2^-7 (fp32 input) / 2^-23 (bf16 input) of it,
    truncated below, zero beyond 2^-31.  The oracle sums the same weights in fp64.  On data whose
    block constants reach 2^-10 ... 2^-40 of the largest magnitude the selected samples must
    still be the oracle's: the truncated part of the weights is far smaller than the gap between
    the cumulative weight and half of the total at the crossing."""
    I = 64
    w = _spread_blocks(8192, I, dtype, 900 + octaves, octaves)
    got = bof4.bof4_em_step([w.cuda()], I, norm, bof4.METRIC_MAE, LV0)
    ref = oracle.em_accumulate_mae(w, I, norm, LV0)
    assert np.array_equal(got["count"], ref["count"])
    assert np.array_equal(got["median"], ref["median"])
    np.testing.assert_allclose(got["s0"], ref["wsum"], rtol=RTOL)
    np.testing.assert_allclose(got["err_sum"], ref["err_sum"], rtol=RTOL)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_mse_sums_with_a_huge_block_at_the_start_of_an_accumulation_window(bof4, dtype):
    """The MSE pass keeps m^2 x and m^2 in fp32 per thread between its folds into fp64.  A block
    1000 times larger than its neighbours in the first row a CTA sees swamps the small terms
    that follow it in those fp32 cells; the totals must still agree with the oracle's fp64 sums
    to 1e-5 (what is lost is small against the large block's own contribution)."""
    I = 64
    n = 16384 * 148 * 3                       # three rows per CTA
    w = workloads.gaussian(n, 0.02, 77, torch.float32)
    w[:16384] *= 1000.0                       # CTA 0, first row: every thread's first 16 weights
    w[16384 * 5 + 64 * 3: 16384 * 5 + 64 * 4] *= 1000.0   # and one block of another CTA
    w = w.to(dtype)
    got = bof4.bof4_em_step([w.cuda()], I, 1, bof4.METRIC_MSE, LV0)
    ref = oracle.em_accumulate_mse(w, I, 1, LV0)
    assert np.array_equal(got["count"], ref["count"])
    np.testing.assert_allclose(got["s1"], ref["s1"], rtol=RTOL, atol=1e-7 * np.abs(ref["s1"]).max())
    np.testing.assert_allclose(got["s0"], ref["s0"], rtol=RTOL)
    np.testing.assert_allclose(got["err_sum"], ref["err_sum"], rtol=RTOL)
