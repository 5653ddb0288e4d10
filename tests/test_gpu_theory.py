"""The data-free (theoretical) codebook solver against the paper's printed codebooks and the
oracle's independent quadrature."""
import os

import numpy as np
import pytest
import torch

import workloads
from oracle import theory

pytestmark = pytest.mark.gpu

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
TAB8 = np.loadtxt(os.path.join(GOLD, "tab8_bof4_mse_emp_theo.txt"))
TAB6 = np.loadtxt(os.path.join(GOLD, "tab6_levels_I64.txt"))
FIX4, FIX4S = workloads.FIXED_BOF4, workloads.FIXED_BOF4S


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def test_printed_theoretical_column_is_a_fixed_point(bof4):
    """Tab. 8, theoretical column (BOF4, MSE, I = 64): one iteration must leave it in place."""
    theo = TAB8[:, 2].astype(np.float32)
    one = bof4.bof4_theoretical_codebook(64, bof4.NORM_ABS, bof4.METRIC_MSE, theo, FIX4, 1).cpu().numpy()
    assert np.abs(one - theo).max() < 3e-7


def test_converges_to_the_printed_theoretical_column(bof4):
    lv = bof4.bof4_theoretical_codebook(64, bof4.NORM_ABS, bof4.METRIC_MSE,
                                        workloads.init_levels_7_0_8(), FIX4, 1500).cpu().numpy()
    assert np.abs(lv - TAB8[:, 2]).max() < 5e-6
    assert lv[0] == -1 and lv[7] == 0 and lv[15] == 1


def test_printed_mae_codebooks_are_fixed_points(bof4):
    """Tab. 6, MAE columns (Monte-Carlo results): residual of one theoretical step within their noise."""
    for norm, col, mask in ((bof4.NORM_ABS, 1, FIX4), (bof4.NORM_SIGNED, 3, FIX4S)):
        start = TAB6[:, col].astype(np.float32)
        one = bof4.bof4_theoretical_codebook(64, norm, bof4.METRIC_MAE, start, mask, 1).cpu().numpy()
        assert np.abs(one - start).max() < 1.5e-4


@pytest.mark.parametrize("I", [32, 100, 256, 2048])
@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("metric", ["mse", "mae"])
def test_agrees_with_the_oracles_quadrature(bof4, I, signed, metric):
    mask = FIX4S if signed else FIX4
    start = workloads.init_levels_7_0_8()
    ref = theory.lloyd(I, signed, metric, start, mask, 3, theory.GaussianBlockModel(I, m_max=12.0, points=24001))
    got = bof4.bof4_theoretical_codebook(I, bof4.NORM_SIGNED if signed else bof4.NORM_ABS,
                                         bof4.METRIC_MSE if metric == "mse" else bof4.METRIC_MAE,
                                         start, mask, 3).cpu().numpy()
    assert np.abs(got - ref).max() < 2e-6
    assert np.all(np.diff(got) > 0)


def test_batched_solver_equals_single_calls(bof4):
    """Every block size of a sweep under both normalisations and metrics in one call: bit for bit
    the results of the single calls."""
    probs = [(I, norm, metric) for I in (32, 64, 100, 1024) for norm in (bof4.NORM_ABS, bof4.NORM_SIGNED)
             for metric in (bof4.METRIC_MSE, bof4.METRIC_MAE)]
    masks = [FIX4 if norm == bof4.NORM_ABS else FIX4S for _, norm, _ in probs]
    start = workloads.init_levels_7_0_8()
    got = bof4.bof4_theoretical_codebook_batch([p[0] for p in probs], [p[1] for p in probs], [p[2] for p in probs],
                                               start, masks, 25).cpu().numpy()
    assert got.shape == (len(probs), 16)
    for row, (I, norm, metric), mask in zip(got, probs, masks):
        one = bof4.bof4_theoretical_codebook(I, norm, metric, start, mask, 25).cpu().numpy()
        assert np.array_equal(row, one), (I, norm, metric)
    assert bof4.bof4_theoretical_codebook_batch([], [], [], start, [], 3).shape == (0, 16)
    with pytest.raises(bof4.Bof4Error):
        bof4.bof4_theoretical_codebook_batch([64] * 129, [0] * 129, [0] * 129, start, [FIX4] * 129, 1)


# --------------------------------------------------------------------------- tabulated densities


def _density(name, n=20001):
    if name == "gauss":
        w = np.linspace(0.0, 12.0, n)
        return 12.0, np.exp(-0.5 * w * w)
    if name == "laplace":
        w = np.linspace(0.0, 40.0, n)
        return 40.0, 0.5 * np.exp(-w)
    w = np.linspace(0.0, 400.0, n)                     # Student-t, 5 degrees of freedom (unnormalised)
    return 400.0, (1.0 + w * w / 5.0) ** -3.0


@pytest.mark.parametrize("name", ["gauss", "laplace", "student5"])
@pytest.mark.parametrize("I", [32, 64, 500])
@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("metric", ["mse", "mae"])
def test_general_density_solver_agrees_with_the_oracle(bof4, name, I, signed, metric):
    """Eq. 5 / Eq. 7 for a tabulated p_W: the device solver against the oracle's tabulated model
    on the same samples (both read the same table; levels within 1e-5 after three iterations)."""
    w_max, pdf = _density(name, 20001 if name != "student5" else 80001)
    mask = FIX4S if signed else FIX4
    start = workloads.init_levels_7_0_8()
    ref = theory.lloyd(I, signed, metric, start, mask, 3, theory.TabulatedBlockModel(I, w_max, pdf))
    got = bof4.bof4_theoretical_codebook_general(I, bof4.NORM_SIGNED if signed else bof4.NORM_ABS,
                                                 bof4.METRIC_MSE if metric == "mse" else bof4.METRIC_MAE,
                                                 pdf, w_max, start, mask, 3).cpu().numpy()
    assert np.abs(got - ref).max() < 1e-5
    assert np.all(np.diff(got) > 0)


def test_general_solver_with_a_gaussian_table_matches_the_gaussian_solver(bof4):
    w_max, pdf = _density("gauss", 40001)
    for norm, mask in ((bof4.NORM_ABS, FIX4), (bof4.NORM_SIGNED, FIX4S)):
        for metric in (bof4.METRIC_MSE, bof4.METRIC_MAE):
            a = bof4.bof4_theoretical_codebook_general(64, norm, metric, pdf, w_max, workloads.init_levels_7_0_8(),
                                                       mask, 20).cpu().numpy()
            b = bof4.bof4_theoretical_codebook(64, norm, metric, workloads.init_levels_7_0_8(), mask, 20).cpu().numpy()
            assert np.abs(a - b).max() < 2e-6


def test_general_solver_rejects_bad_arguments(bof4):
    w_max, pdf = _density("gauss", 101)
    with pytest.raises(bof4.Bof4Error):
        bof4.bof4_theoretical_codebook_general(64, bof4.NORM_ABS, bof4.METRIC_MSE, pdf, -1.0, workloads.init_levels_7_0_8(),
                                               FIX4, 1)
    with pytest.raises(bof4.Bof4Error):          # the outermost levels must be fixed
        bof4.bof4_theoretical_codebook_general(64, bof4.NORM_ABS, bof4.METRIC_MSE, pdf, w_max,
                                               workloads.init_levels_7_0_8(), 0, 1)
