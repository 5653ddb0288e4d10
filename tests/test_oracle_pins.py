"""Pins of the CPU oracle: what the paper prints and what the mathematics fixes.

None of these tests touches the CUDA library.  Each one is chosen so that a plausible mistake
in the oracle (wrong sign, dropped weight, off-by-one in the median, transposed nibble, abs
instead of signed maximum, ...) fails it.
"""
import os

import numpy as np
import pytest
import torch

import oracle
import workloads
from oracle import theory

GOLD = os.path.join(os.path.dirname(__file__), "golden")
TAB6 = np.loadtxt(os.path.join(GOLD, "tab6_levels_I64.txt"))
TAB7 = np.loadtxt(os.path.join(GOLD, "tab7_bof4s_mse_levels.txt"))
TAB8 = np.loadtxt(os.path.join(GOLD, "tab8_bof4_mse_emp_theo.txt"))

ABS, SGN = oracle.NORM_ABS, oracle.NORM_SIGNED
MSE, MAE = oracle.METRIC_MSE, oracle.METRIC_MAE
FIX4, FIX4S = workloads.FIXED_BOF4, workloads.FIXED_BOF4S


@pytest.fixture(scope="module")
def gauss24():
    """2^24 N(0,1) samples (the paper fits its codebooks on Gaussian samples, Sec. 4)."""
    return oracle.as_f32(workloads.gaussian(1 << 24, 1.0, 123))


@pytest.fixture(scope="module")
def model64():
    return theory.GaussianBlockModel(64)


# ------------------------------------------------------------------ theoretical solution


def test_theory_fixed_point_of_printed_theoretical_column(model64):
    """Tab. 8, theoretical column: one Lloyd step with the Gaussian MSE centroid (boxed
    equation of App. B.2 with its minus sign restored, midpoint thresholds) leaves it fixed."""
    theo = TAB8[:, 2]
    one = theory.lloyd(64, False, "mse", theo, FIX4, 1, model64)
    assert np.abs(one - theo).max() < 3e-7


def test_theory_wrong_sign_is_caught(model64):
    """Without the restored minus sign the centroid lands on the other side of zero."""
    c = model64.mse_centroid(0.05, 0.13)
    assert 0.05 < c < 0.13
    assert not (0.05 < -c < 0.13)


def test_theory_converges_to_printed_theoretical_column():
    mdl = theory.GaussianBlockModel(64, points=6001)
    lv = theory.lloyd(64, False, "mse", workloads.init_levels_7_0_8(), FIX4, 1500, mdl)
    assert np.abs(lv - TAB8[:, 2]).max() < 5e-6


def test_tab8_deviation_column_is_consistent():
    """Tab. 8: the printed third column is the absolute difference of the first two (a check of
    the golden file, and the 1.3e-4 bound the Monte-Carlo pins below rely on)."""
    theo, emp = TAB8[:, 2], TAB8[:, 1]
    assert np.abs(theo - emp).max() <= 1.3e-4
    assert np.allclose(np.abs(theo - emp), TAB8[:, 3], atol=1e-12)


@pytest.mark.parametrize("signed,norm", [(False, ABS), (True, SGN)])
def test_region_probabilities_match_member_counts(gauss24, model64, signed, norm):
    """P[X in R_l] from the cdf of the normalised weights (App. B.1: a continuous part of mass
    (I-1)/I and the point mass 1/I of the block maximum) against the member counts the
    data-driven oracle finds on 2^24 Gaussian samples: binomial noise only.  A missing point
    mass, a wrong (I-1)/I factor or a one-sided split under absolute normalisation fails it."""
    lv = TAB6[:, 4 if signed else 2].astype(np.float32)
    p = theory.region_probabilities(lv.astype(np.float64), 64, signed, model64)
    assert abs(p.sum() - 1.0) < 1e-9
    st = oracle.em_accumulate_mse(gauss24, 64, norm, lv)
    freq = st["count"] / float(gauss24.size)
    sd = np.sqrt(p * (1.0 - p) / gauss24.size)
    assert np.all(np.abs(freq - p) < 6.0 * sd + 2e-6)   # 2e-6: fp32 thresholds vs fp64 midpoints
    # the planted mistake: all of the block maximum's mass at +1 under absolute normalisation
    # (or split under signed normalisation) is far outside the noise
    wrong = theory.region_probabilities(lv.astype(np.float64), 64, not signed, model64)
    assert np.abs(freq - wrong).max() > 100.0 * sd.max()


def test_data_driven_centroid_agrees_with_theory(gauss24, model64):
    """Eq. 6 (Monte-Carlo) against Eq. 5 (integration): started at the theoretical solution,
    the data-driven EM stays within Monte-Carlo noise (the paper reports <= 1.3e-4, Tab. 8)."""
    theo = TAB8[:, 2]
    lv, _ = oracle.fit(gauss24, 64, ABS, MSE, theo, FIX4, 3)
    assert np.abs(lv - theo).max() < 3e-4
    # signed normalisation: leftmost level is free and owns [-1, xi_0)
    theo_s = theory.lloyd(64, True, "mse", TAB6[:, 4], FIX4S, 200, model64)
    lv, _ = oracle.fit(gauss24, 64, SGN, MSE, theo_s, FIX4S, 3)
    assert np.abs(lv - theo_s).max() < 3e-4


@pytest.mark.parametrize("signed,norm,mask", [(False, ABS, FIX4), (True, SGN, FIX4S)])
@pytest.mark.parametrize("metric", ["mse", "mae"])
def test_one_em_step_agrees_with_theory_from_any_start(gauss24, signed, norm, mask, metric):
    """The Monte-Carlo centroids (Eq. 6: weights m^2; Eq. 8: weighted median, weights |m|) and
    the analytical ones (Eq. 5; root of Eq. 7) of the SAME regions agree within Monte-Carlo
    noise, here for the regions of an evenly spaced start far from the optimum."""
    mdl = theory.GaussianBlockModel(64, points=4001)
    start = workloads.init_levels_7_0_8()
    theo = theory.lloyd(64, signed, metric, start, mask, 1, mdl)
    lv, _ = oracle.fit(gauss24, 64, norm, MSE if metric == "mse" else MAE, start, mask, 1)
    assert np.abs(lv - theo).max() < 2.5e-4
    assert np.abs(lv - np.array(start)).max() > 5e-3  # the step is not a no-op


def test_printed_mae_codebooks_are_theoretical_fixed_points():
    """Tab. 6, MAE columns, against the root of Eq. 7 (read with the conditional cdf of its
    derivation): residual of one theoretical step within the tables' Monte-Carlo noise."""
    mdl = theory.GaussianBlockModel(64, points=4001)
    for signed, col, mask in ((False, 1, FIX4), (True, 3, FIX4S)):
        one = theory.lloyd(64, signed, "mae", TAB6[:, col], mask, 1, mdl)
        assert np.abs(one - TAB6[:, col]).max() < 1.5e-4


# ------------------------------------------------------------------ printed codebooks


@pytest.mark.parametrize("col,norm,metric,mask,tol", [
    (1, ABS, MAE, FIX4, 4e-4), (2, ABS, MSE, FIX4, 3e-4),
    (3, SGN, MAE, FIX4S, 4e-4), (4, SGN, MSE, FIX4S, 3e-4)])
def test_tab6_codebooks_are_fixed_points(gauss24, col, norm, metric, mask, tol):
    """Tab. 6 (I = 64): one EM step on Gaussian samples moves no printed level by more than
    Monte-Carlo noise."""
    lv0 = TAB6[:, col].astype(np.float32)
    lv, _ = oracle.fit(gauss24, 64, norm, metric, lv0, mask, 1)
    assert np.abs(lv - lv0).max() < tol
    for l in range(16):
        if (mask >> l) & 1:
            assert lv[l] == lv0[l]


@pytest.mark.parametrize("col,I", [(1, 32), (2, 64), (3, 128), (4, 256)])
def test_tab7_codebooks_are_fixed_points(gauss24, col, I):
    lv0 = TAB7[:, col].astype(np.float32)
    lv, _ = oracle.fit(gauss24, I, SGN, MSE, lv0, FIX4S, 1)
    assert np.abs(lv - lv0).max() < 3e-4


def test_wrong_normalisation_or_block_size_is_caught(gauss24):
    """The fixed-point pins discriminate: the BOF4-S codebook is not a fixed point under
    absolute normalisation, nor is the I = 64 codebook one at I = 256."""
    lv0 = TAB6[:, 4].astype(np.float32)
    sub = gauss24[: 1 << 22]
    lv, _ = oracle.fit(sub, 64, ABS, MSE, lv0, FIX4S, 1)
    assert np.abs(lv - lv0).max() > 5e-3
    lv, _ = oracle.fit(sub, 256, SGN, MSE, lv0, FIX4S, 1)
    assert np.abs(lv - lv0).max() > 5e-3


def test_error_ordering_on_gaussian_samples(gauss24):
    """Sec. 5, "Quantization Error": error grows with the block size; BOF4-S is below BOF4;
    each codebook wins on the metric it was optimised for."""
    sub = gauss24[: 1 << 22]
    mse = [oracle.quant_error(sub, I, SGN, TAB7[:, c])[0] for c, I in
           ((1, 32), (2, 64), (3, 128), (4, 256))]
    assert mse[0] < mse[1] < mse[2] < mse[3]
    e = {}
    for name, col, norm in (("b_mae", 1, ABS), ("b_mse", 2, ABS), ("s_mae", 3, SGN),
                            ("s_mse", 4, SGN)):
        e[name] = oracle.quant_error(sub, 64, norm, TAB6[:, col])
    assert e["s_mse"][0] < e["b_mse"][0] and e["s_mae"][1] < e["b_mae"][1]
    assert e["b_mse"][0] < e["b_mae"][0] and e["b_mae"][1] < e["b_mse"][1]
    assert e["s_mse"][0] < e["s_mae"][0] and e["s_mae"][1] < e["s_mse"][1]
    # Tab. 1 soft pin: MSE ratio BOF4 / BOF4-S of the Llama-3.1 8B row is 1.566 / 1.441
    assert abs(e["b_mse"][0] / e["s_mse"][0] - 1.566 / 1.441) < 0.02


# ------------------------------------------------------------------ encoding (Eq. 1-4)


def test_block_constant_abs_and_signed():
    w = np.array([0.5, -2.0, 2.0, 1.0, -0.25, 0.25, 0.0, 0.125], np.float32)
    assert oracle.block_constants(w, 4, ABS).tolist() == [2.0, 0.25]
    # signed: first element of maximal magnitude wins, with its sign
    assert oracle.block_constants(w, 4, SGN).tolist() == [-2.0, -0.25]
    assert oracle.block_constants(np.zeros(4, np.float32), 4, SGN).tolist() == [0.0]


def test_codes_nibbles_and_thresholds_by_hand():
    lv = np.array(workloads.init_levels_7_0_8(), np.float32)
    xi = oracle.thresholds(lv)
    assert xi[7] == np.float32(0.0625) and xi[6] == (lv[6] + lv[7]) * np.float32(0.5)
    # block of 4 with m = 1: x = w
    w = np.array([1.0, -1.0, 0.0625, 0.06], np.float32)
    codes, scales = oracle.quantize(w, 4, ABS, lv)
    assert scales.tolist() == [1.0]
    # 1.0 -> level 15, -1.0 -> level 0, tie at xi_7 goes up (level 8), 0.06 -> level 7
    assert codes.tolist() == [(15 << 4) | 0, (8 << 4) | 7]
    out = oracle.dequantize(codes, scales, 4, lv)
    assert out.tolist() == [1.0, -1.0, 0.125, 0.0]


@pytest.mark.parametrize("norm,mask", [(ABS, FIX4), (SGN, FIX4S)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_block_maximum_is_reconstructed_exactly(norm, mask, dtype):
    """Sec. 2.2 / 3.1: with -1 and 1 (or only 1, signed) among the levels, the weight of
    largest magnitude in every block is reproduced bit for bit."""
    w = workloads.gaussian(64 * 500, 0.02, 7, dtype)
    a = oracle.as_f32(w)
    lv = TAB6[:, 2 if norm == ABS else 4]
    codes, scales = oracle.quantize(a, 64, norm, lv)
    out = oracle.dequantize(codes, scales, 64, lv).reshape(-1, 64)
    blk = a.reshape(-1, 64)
    j = np.abs(blk).argmax(1)
    r = np.arange(blk.shape[0])
    assert np.array_equal(out[r, j].view(np.uint32), blk[r, j].view(np.uint32))
    if norm == SGN:
        assert np.array_equal(scales, blk[r, j])
    else:
        assert np.array_equal(scales, np.abs(blk[r, j]))


def test_bf16_rounding_matches_torch():
    x = torch.randn(100000, generator=torch.Generator().manual_seed(3)) * 3
    x[:4] = torch.tensor([1.00390625, 1.01171875, -1.00390625, 0.0])  # exact ties
    ref = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.f32_to_bf16_bits(x.numpy()), ref)
    assert np.array_equal(oracle.bf16_bits_to_f32(ref), x.to(torch.bfloat16).float().numpy())


# ------------------------------------------------------------------ EM: exact optimum


def _dp_optimum(x, a, fixed, power):
    """Exact optimum of sum a |x - level(x)|^power over ordered contiguous partitions of the
    sorted points into 16 cells; cell l uses the prescribed value if l is fixed, else its best
    constant.  Returns (cost, levels, cell boundaries)."""
    order = np.argsort(x, kind="stable")
    x, a = x[order].astype(np.float64), a[order].astype(np.float64)
    P = len(x)

    def cell(i, j, l):
        if i == j:
            return 0.0, fixed.get(l, None)
        xs, ws = x[i:j], a[i:j]
        if l in fixed:
            v = fixed[l]
            return float(np.sum(ws * np.abs(xs - v) ** power)), v
        if power == 2:
            v = float(np.sum(ws * xs) / np.sum(ws))
            return float(np.sum(ws * (xs - v) ** 2)), v
        costs = [float(np.sum(ws * np.abs(xs - c))) for c in xs]  # minimiser is a sample
        k = int(np.argmin(costs))
        return costs[k], float(xs[k])

    INF = float("inf")
    dp = np.full((17, P + 1), INF)
    arg = np.zeros((17, P + 1), dtype=int)
    dp[0, 0] = 0.0
    for l in range(16):
        for j in range(P + 1):
            for i in range(j + 1):
                if dp[l, i] == INF:
                    continue
                c, _ = cell(i, j, l)
                if dp[l, i] + c < dp[l + 1, j]:
                    dp[l + 1, j] = dp[l, i] + c
                    arg[l + 1, j] = i
    bounds = [P]
    for l in range(16, 0, -1):
        bounds.append(arg[l, bounds[-1]])
    bounds = bounds[::-1]
    levels = [cell(bounds[l], bounds[l + 1], l)[1] for l in range(16)]
    return dp[16, P], levels, bounds


def _tiny_blocks(seed, nblocks, I):
    g = np.random.default_rng(seed)
    w = g.normal(0, 1, (nblocks, I)).astype(np.float32)
    scale = g.uniform(0.5, 2.0, (nblocks, 1)).astype(np.float32)
    w = w / np.abs(w).max(1, keepdims=True) * scale  # varied block constants
    w[0, 1] = 0.0
    return w.reshape(-1)


@pytest.mark.parametrize("metric,nblocks", [(MSE, 20), (MAE, 12)])
def test_em_against_exact_optimum_on_tiny_input(metric, nblocks):
    """Brute force: EM can never beat the exact optimum, and it does not move away from it."""
    I = 4
    w = _tiny_blocks(11, nblocks, I)
    m = oracle.block_constants(w, I, ABS)
    x = (w.reshape(-1, I) / m[:, None]).reshape(-1)
    a = np.repeat(m.astype(np.float64) ** (2 if metric == MSE else 1), I)
    fixed = {0: -1.0, 7: 0.0, 15: 1.0}
    best, levels, bounds = _dp_optimum(x, a, fixed, 2 if metric == MSE else 1)
    n = w.size
    # from the default start, any number of iterations stays above the optimum
    lv, log = oracle.fit(w, I, ABS, metric, workloads.init_levels_7_0_8(), FIX4, 40)
    assert log[-1] * n >= best * (1 - 1e-9)
    assert best > 0
    # Started at the optimum (when its levels are ascending, which the EM's index order needs)
    # the error equals the optimum and stays there.  Cells the optimum leaves empty get
    # interpolated levels: whatever they capture, the nearest-neighbour error can neither
    # rise above the optimum nor fall below it.
    lv0 = np.array([np.nan if v is None else v for v in levels], np.float64)
    known = np.flatnonzero(~np.isnan(lv0))
    lv0 = np.interp(np.arange(16), known, lv0[known])
    ascending = bool(np.all(np.diff(lv0) > 0))
    full = all(bounds[l + 1] > bounds[l] for l in range(16))
    if metric == MSE:
        assert ascending and full, "pick a seed whose optimum is ascending and uses every level"
    if ascending:
        lv0 = lv0.astype(np.float32)
        lv, log = oracle.fit(w, I, ABS, metric, lv0, FIX4, 3)
        assert np.all(np.abs(log * n - best) <= 1e-5 * best)
        if full and metric == MSE:
            assert np.allclose(lv, lv0, rtol=2e-6, atol=1e-7)


def test_em_error_is_monotone():
    """App. B.2: nearest-neighbour assignment and the modified centroid are both necessary
    conditions, so the error of successive codebooks never increases."""
    w = workloads.config2(1 << 18)
    for norm, metric, mask in ((ABS, MSE, FIX4), (SGN, MSE, FIX4S), (SGN, MAE, FIX4S),
                               (ABS, MAE, 0)):
        _, log = oracle.fit(w, 64, norm, metric, workloads.init_levels_7_0_8(), mask, 25)
        assert np.all(np.diff(log) <= 1e-12 * log[0]), (norm, metric)
        assert log[-1] < 0.9 * log[0]


# ------------------------------------------------------------------ EM: library special cases


def _unit_constant_blocks(seed, nblocks, I):
    """Blocks whose absolute maximum is exactly 1, so every weight m^2 (or |m|) equals 1 and
    the modified centroid reduces to the textbook one (App. D)."""
    g = np.random.default_rng(seed)
    w = g.uniform(-0.999, 0.999, (nblocks, I)).astype(np.float32)
    w[np.arange(nblocks), g.integers(0, I, nblocks)] = g.choice([-1.0, 1.0], nblocks)
    return w.reshape(-1)


def test_equal_constants_reduce_to_library_kmeans():
    from sklearn.cluster import KMeans
    w = _unit_constant_blocks(5, 512, 64)
    init = np.array(workloads.init_levels_linspace(), np.float32)
    T = 4
    lv, _ = oracle.fit(w, 64, ABS, MSE, init, 0, T)
    km = KMeans(n_clusters=16, init=init.astype(np.float64).reshape(-1, 1), n_init=1,
                max_iter=T, tol=0.0, algorithm="lloyd").fit(w.astype(np.float64).reshape(-1, 1))
    assert np.allclose(lv, km.cluster_centers_.reshape(-1), rtol=0, atol=2e-6)


def test_equal_constants_reduce_to_plain_median():
    w = _unit_constant_blocks(6, 300, 32)
    init = np.array(workloads.init_levels_linspace(), np.float32)
    st = oracle.em_accumulate_mae(w, 32, ABS, init)
    xi = oracle.thresholds(init)
    code = (xi[None, :] <= w[:, None]).sum(1)
    for l in range(16):
        mem = w[code == l]
        assert st["count"][l] == mem.size and mem.size > 0
        assert st["median"][l] == np.quantile(mem, 0.5, method="inverted_cdf")
        assert st["wsum"][l] == mem.size


def test_weighted_median_minimises_the_stated_objective():
    """Reading of Eq. 8: the returned sample minimises f(xh) = sum a_k |x_k - xh|, also where
    the printed max-formula would be empty (single member) or off by one."""
    g = np.random.default_rng(9)
    for trial in range(20):
        nb = int(g.integers(1, 30))
        w = (g.normal(0, 1, (nb, 4)) * g.uniform(0.1, 3, (nb, 1))).astype(np.float32).reshape(-1)
        lv = np.array(workloads.init_levels_7_0_8(), np.float32)
        st = oracle.em_accumulate_mae(w, 4, SGN, lv)
        m = oracle.block_constants(w, 4, SGN)
        x = (w.reshape(-1, 4) / m[:, None]).reshape(-1).astype(np.float32)
        a = np.repeat(np.abs(m).astype(np.float64), 4)
        code = (oracle.thresholds(lv)[None, :] <= x[:, None]).sum(1)
        for l in range(16):
            xs, ws = x[code == l].astype(np.float64), a[code == l]
            if xs.size == 0:
                assert st["median"][l] == lv[l]
                continue
            f = lambda c: np.sum(ws * np.abs(xs - c))
            fmin = min(f(c) for c in xs)
            assert f(float(st["median"][l])) <= fmin * (1 + 1e-12)
            assert st["median"][l] in x[code == l]


# ------------------------------------------------------------------ invariants


def test_scaling_by_power_of_two():
    w = oracle.as_f32(workloads.config2(1 << 16))
    lv = TAB6[:, 4]
    c1, s1 = oracle.quantize(w, 64, SGN, lv)
    c2, s2 = oracle.quantize(w * np.float32(8.0), 64, SGN, lv)
    assert np.array_equal(c1, c2) and np.array_equal(s1 * np.float32(8.0), s2)
    f1, _ = oracle.fit(w, 64, SGN, MSE, workloads.init_levels_7_0_8(), FIX4S, 5)
    f2, _ = oracle.fit(w * np.float32(8.0), 64, SGN, MSE, workloads.init_levels_7_0_8(), FIX4S, 5)
    assert np.allclose(f1, f2, rtol=1e-6)


def test_signed_normalisation_is_invariant_to_global_negation():
    w = oracle.as_f32(workloads.config2(1 << 16))
    lv = TAB6[:, 4]
    c1, s1 = oracle.quantize(w, 64, SGN, lv)
    c2, s2 = oracle.quantize(-w, 64, SGN, lv)
    assert np.array_equal(c1, c2) and np.array_equal(s1, -s2)


def test_block_permutation_and_sorted_codebook():
    w = oracle.as_f32(workloads.config2(1 << 16))
    perm = np.random.default_rng(1).permutation(w.size // 64)
    wp = w.reshape(-1, 64)[perm].reshape(-1)
    lv = workloads.init_levels_7_0_8()
    a = oracle.em_accumulate_mse(w, 64, ABS, lv)
    b = oracle.em_accumulate_mse(wp, 64, ABS, lv)
    assert np.array_equal(a["count"], b["count"])
    assert np.allclose(a["s1"], b["s1"], rtol=1e-11) and np.allclose(a["s0"], b["s0"], rtol=1e-11)
    assert int(a["count"].sum()) == w.size
    f, _ = oracle.fit(w, 64, ABS, MSE, lv, FIX4, 10)
    assert np.all(np.diff(f) > 0)


def test_all_zero_block_and_empty_region():
    w = np.zeros(128, np.float32)
    w[64:] = np.linspace(-1, 1, 64, dtype=np.float32)
    lv = np.array(workloads.init_levels_7_0_8(), np.float32)
    codes, scales = oracle.quantize(w, 64, ABS, lv)
    assert scales[0] == 0.0 and np.all(codes[:32] == ((7 << 4) | 7))
    assert np.all(oracle.dequantize(codes, scales, 64, lv)[:64] == 0.0)
    # a region nobody falls into keeps its level; the zero block adds no weight anywhere
    lv2 = lv.copy()
    lv2[1] = -0.9999
    out, _ = oracle.fit(np.zeros(64, np.float32), 64, ABS, MSE, lv2, 0, 1)
    assert np.array_equal(out, lv2)
    out, _ = oracle.fit(np.zeros(64, np.float32), 64, ABS, MAE, lv2, 0, 1)
    assert np.array_equal(out, lv2)


# ------------------------------------------------------------------ OPQ (Sec. 3.3, App. E)


def test_sigma_by_hand_and_against_numpy():
    # tree order: (a+b)+(c+d); values chosen so that the order matters in fp32
    w = np.array([1e8, 1.0, -1e8, 1.0], np.float32)
    s_tree = np.float32(np.float32(1e8 + 1.0) + np.float32(-1e8 + 1.0))  # = 0 in fp32
    mean = s_tree / np.float32(4)
    d = (w - mean).astype(np.float32)
    sq = (d * d).astype(np.float32)
    ss = np.float32(np.float32(sq[0] + sq[1]) + np.float32(sq[2] + sq[3]))
    expect = np.sqrt(np.float32(ss / np.float32(3)))
    assert oracle.block_sigmas(w, 4)[0] == expect
    x = oracle.as_f32(workloads.gaussian(64 * 200, 0.02, 21))
    ref = x.reshape(-1, 64).astype(np.float64).std(axis=1, ddof=1)
    assert np.allclose(oracle.block_sigmas(x, 64), ref, rtol=2e-6)


def test_opq_threshold_values():
    """tau = F_M^{-1}(q), F_M = F_|W|^I (App. B.1); checked through the defining identity."""
    from scipy.special import ndtr
    for I in (32, 64, 128, 256):
        for q in (0.9, 0.95, 0.97, 0.99):
            tau = oracle.opq_threshold(q, I)
            assert abs((2 * ndtr(tau) - 1) ** I - q) < 1e-12
    assert abs(oracle.opq_threshold(0.95, 64) - 3.352402) < 1e-6


def test_opq_split_semantics_and_rates():
    I, q = 64, 0.95
    tau = oracle.opq_threshold(q, I)
    w = oracle.as_f32(workloads.gaussian(I * 20000, 0.015, 31, torch.bfloat16))
    clean, idx, val, k = oracle.opq_split(w, I, tau)
    assert k == idx.size and np.all(np.diff(idx) > 0)
    thr = np.repeat(oracle.block_sigmas(w, I) * np.float32(tau), I)
    flag = np.abs(w) > thr
    assert np.array_equal(np.nonzero(flag)[0], idx)
    assert np.array_equal(oracle.bf16_bits_to_f32(val), w[idx])  # bf16 input: exact
    assert np.all(clean[idx] == 0) and np.array_equal(clean[~flag], w[~flag])
    # By construction of tau a fraction 1-q of Gaussian blocks would hold an outlier if sigma_b
    # were the true sigma; the block's own maximum inflates the estimate, so it is a bit less.
    frac_blocks = flag.reshape(-1, I).any(1).mean()
    assert 0.02 < frac_blocks < 0.05
    # App. E.2: extra memory (16-bit value + 64-bit index per outlier) relative to the 4-bit
    # codes plus 16-bit constants is 0.96 % at I = 64, q = 0.95 on Llama-3.1 8B; Gaussian
    # data gives the same figure within sampling noise.
    overhead = 80.0 * (k / w.size) / (4 + 16 / I)
    assert abs(overhead - 0.0096) < 0.0012
    # capacity: count is exact, nothing written beyond it
    _, idx2, _, k2 = oracle.opq_split(w, I, tau, capacity=5)
    assert k2 == k and np.array_equal(idx2, idx[:5])
    # decoding side: outliers are restored exactly
    lv = TAB6[:, 4]
    codes, scales = oracle.quantize(clean, I, SGN, lv)
    out = oracle.opq_restore(oracle.dequantize(codes, scales, I, lv), idx, val)
    assert np.array_equal(out[idx], w[idx])


def test_opq_zero_variance_block_literal_rule():
    w = np.full(64, 0.5, np.float32)
    _, idx, _, k = oracle.opq_split(w, 64, 3.0)
    assert k == 64  # sigma_b = 0: every non-zero element exceeds the threshold
    _, idx, _, k = oracle.opq_split(np.zeros(64, np.float32), 64, 3.0)
    assert k == 0


# --------------------------------------------------------------------------- App. D variants


def _normalised(w, I, signed):
    """x = w / m by its definition, in numpy (independent of the oracle's code)."""
    wb = w.reshape(-1, I)
    j = np.abs(wb).argmax(1)
    m = wb[np.arange(wb.shape[0]), j] if signed else np.abs(wb).max(1)
    return (wb / m[:, None]).astype(np.float32).reshape(-1)


@pytest.mark.parametrize("norm,signed", [(ABS, False), (SGN, True)])
def test_normalised_domain_mse_is_library_kmeans_on_x(norm, signed):
    """Minimising the error of the normalised weights is textbook Lloyd on x (App. D, the
    plain-mean centroid): a library k-means on x = w / m must give the same levels, also for
    blocks of very different scale (where the BOF4 centroid differs)."""
    from sklearn.cluster import KMeans
    g = np.random.default_rng(9)
    w = (g.standard_normal((400, 64)) * g.uniform(0.01, 3.0, (400, 1))).astype(np.float32).reshape(-1)
    init = np.array(workloads.init_levels_linspace(), np.float32)
    T = 3
    lv, log = oracle.fit(w, 64, norm, oracle.METRIC_MSE_NORMDOM, init, 0, T)
    x = _normalised(w, 64, signed).astype(np.float64)
    km = KMeans(n_clusters=16, init=init.astype(np.float64).reshape(-1, 1), n_init=1, max_iter=T,
                tol=0.0, algorithm="lloyd").fit(x.reshape(-1, 1))
    assert np.allclose(lv, km.cluster_centers_.reshape(-1), rtol=0, atol=2e-6)
    # the logged error is the mean squared error of x under the entering levels
    xi = oracle.thresholds(init)
    code = (xi[None, :] <= x[:, None].astype(np.float32)).sum(1)
    assert np.isclose(log[0], np.mean((x - init[code]) ** 2), rtol=1e-9)
    # and it differs from the BOF4 centroid on such data
    lv_bof, _ = oracle.fit(w, 64, norm, MSE, init, 0, T)
    assert np.abs(lv_bof - lv).max() > 1e-3


def test_normalised_domain_mae_is_the_plain_median_of_x():
    g = np.random.default_rng(10)
    w = (g.standard_normal((300, 32)) * g.uniform(0.01, 3.0, (300, 1))).astype(np.float32).reshape(-1)
    init = np.array(workloads.init_levels_linspace(), np.float32)
    st = oracle.em_accumulate_mae(w, 32, SGN, init, normdom=True)
    x = _normalised(w, 32, True)
    xi = oracle.thresholds(init)
    code = (xi[None, :] <= x[:, None]).sum(1)
    err = 0.0
    for l in range(16):
        mem = x[code == l]
        assert st["count"][l] == mem.size and st["wsum"][l] == mem.size
        if mem.size:
            assert st["median"][l] == np.quantile(mem, 0.5, method="inverted_cdf")
            err += np.abs(mem.astype(np.float64) - float(init[l])).sum()
    assert np.isclose(st["err_sum"], err, rtol=1e-9)


# --------------------------------------------------------------------------- decode fused into y = W x


def test_gemv_closed_forms_by_hand():
    """Eq. 3 inside a matrix-vector product, on a 2 x 64 matrix whose result is known in closed
    form: a row of codes 15 (level 1) gives scale * sum(x); nibble order (even column = high
    nibble) and the row / block bookkeeping are fixed by one odd entry per row."""
    lv = np.linspace(-1, 1, 16).astype(np.float32)
    lv[7] = 0.0
    rows, cols, I = 2, 64, 32
    codes = np.full(rows * cols // 2, 0xFF, np.uint8)
    scales = np.array([2.0, 3.0, 0.5, 0.25], np.float32)  # blocks (r0,b0) (r0,b1) (r1,b0) (r1,b1)
    x = np.arange(1, cols + 1, dtype=np.float32)
    y, mag = oracle.gemv(codes, scales, rows, cols, I, lv, x)
    assert y[0] == 2.0 * x[:32].sum() + 3.0 * x[32:].sum()
    assert y[1] == 0.5 * x[:32].sum() + 0.25 * x[32:].sum()
    assert np.array_equal(y, mag)
    # column 5 of row 0 -> code 0 (level -1): byte 2 holds columns 4 (high) and 5 (low)
    codes2 = codes.copy()
    codes2[2] = 0xF0
    y2, _ = oracle.gemv(codes2, scales, rows, cols, I, lv, x)
    assert y2[0] == y[0] - 2 * 2.0 * x[5] and y2[1] == y[1]
    # column 40 of row 1 -> code 7 (level 0): byte (64 + 40) / 2 = 52, high nibble
    codes3 = codes.copy()
    codes3[52] = 0x7F
    y3, _ = oracle.gemv(codes3, scales, rows, cols, I, lv, x)
    assert y3[1] == y[1] - 0.25 * x[40] and y3[0] == y[0]
    # an outlier replaces the decoded value: flat index 64 + 3 gets 10.0 (bf16 bits 0x4120)
    y4, _ = oracle.gemv(codes, scales, rows, cols, I, lv, x, idx=np.array([67]), val=np.array([0x4120], np.uint16))
    assert y4[1] == y[1] + (10.0 - 0.5) * x[3]


def test_gemv_is_the_library_matvec_of_the_dequantised_matrix():
    """Against numpy's matvec of the separately dequantised (Eq. 3) and restored (Sec. 3.3) matrix:
    the only difference is the fp32 rounding of scale * level, 2^-24 relative per term."""
    rng = np.random.default_rng(5)
    rows, cols, I = 24, 256, 64
    w = workloads.gaussian(rows * cols, 0.02, seed=91).numpy()
    w[rng.integers(0, w.size, 40)] *= 12.0
    lv = TAB6[:, 2].astype(np.float32)  # BOF4 (MSE), Tab. 6
    clean, idx, val, k = oracle.opq_split(w, I, oracle.opq_threshold(0.95, I))
    assert 0 < k == idx.size
    codes, scales = oracle.quantize(clean, I, oracle.NORM_ABS, lv)
    x = rng.standard_normal(cols).astype(np.float32)
    y, mag = oracle.gemv(codes, scales, rows, cols, I, lv, x, idx, val)
    W = oracle.opq_restore(oracle.dequantize(codes, scales, I, lv), idx, val).reshape(rows, cols).astype(np.float64)
    ref = W @ x.astype(np.float64)
    assert np.all(np.abs(y - ref) <= 2.0 ** -23 * mag)
    assert np.abs(y - ref).max() > 0 or np.array_equal(y, ref)
    # and it is close to the unquantised product: the quantisation error is small, not absent
    exact = w.reshape(rows, cols).astype(np.float64) @ x.astype(np.float64)
    assert 0 < np.abs(y - exact).max() < 0.25 * np.abs(exact).max()
    # a transposed operand or a dropped outlier list is caught
    y_no, _ = oracle.gemv(codes, scales, rows, cols, I, lv, x)
    assert np.abs(y_no - ref).max() > 100 * 2.0 ** -23 * mag.max()


# --------------------------------------------------------------------------- ragged last block


def test_ragged_last_block_is_a_block_of_its_own():
    """A tensor that does not end on a block boundary: the last block is quantised by its own
    maximum.  Zero padding changes no maximum, so its codes must equal those of the zero-padded
    block; only a half-filled last byte differs (zero low nibble instead of the code of 0)."""
    rng = np.random.default_rng(11)
    I, tail = 64, 37
    lv = TAB6[:, 4].astype(np.float32)
    w = (rng.standard_normal(3 * I + tail) * 0.02).astype(np.float32)
    for norm in (ABS, SGN):
        codes, scales = oracle.quantize(w, I, norm, lv)
        assert codes.size == (w.size + 1) // 2 and scales.size == 4
        head_c, head_s = oracle.quantize(w[:3 * I], I, norm, lv)
        assert np.array_equal(codes[:3 * I // 2], head_c) and np.array_equal(scales[:3], head_s)
        padded = np.concatenate([w[3 * I:], np.zeros(I - tail, np.float32)])
        pc, ps = oracle.quantize(padded, I, norm, lv)
        assert scales[3] == ps[0] == oracle.block_constants(w[3 * I:], tail, norm)[0]
        assert np.array_equal(codes[96:96 + tail // 2], pc[:tail // 2])
        assert codes[96 + tail // 2] == (pc[tail // 2] & 0xF0)          # element 36 high, nothing low
        deq = oracle.dequantize(codes, scales, I, lv, n=w.size)
        assert deq.size == w.size
        assert np.array_equal(deq[3 * I:], oracle.dequantize(pc, ps, I, lv)[:tail])


def test_ragged_last_block_sigma_and_outliers():
    """sigma of the short block is the corrected sample deviation over ITS elements (numpy's
    ddof = 1), not over a padded block; a one-weight block has no outliers."""
    rng = np.random.default_rng(12)
    I = 64
    for tail in (1, 2, 3, 33, 63):
        w = (rng.standard_normal(2 * I + tail) * 0.02).astype(np.float32)
        w[2 * I] = 0.5                                   # would be an outlier in any longer block
        sig = oracle.block_sigmas(w, I)
        assert sig.size == 3
        if tail == 1:
            assert np.isnan(sig[2])
        else:
            ref = np.std(w[2 * I:].astype(np.float64), ddof=1)
            assert abs(sig[2] - ref) <= 1e-6 * ref
        clean, idx, val, k = oracle.opq_split(w, I, 1.2)
        in_tail = idx[idx >= 2 * I]
        expect = np.nonzero(np.abs(w[2 * I:]) > np.float32(sig[2]) * np.float32(1.2))[0] + 2 * I if tail > 1 else []
        assert np.array_equal(in_tail, np.asarray(expect, dtype=np.int64))
        assert np.all(clean[idx] == 0) and clean.size == w.size
        if tail == 1:
            assert clean[2 * I] == np.float32(0.5)


# --------------------------------------------------------------------------- ragged tensors in the fit


def _by_hand_stats(w, I, norm, lv):
    """E-step statistics written out with numpy from the definitions (Eq. 1/4 block constant,
    Eq. 2 regions, Sec. 3.1 sums), block by block, every tensor cut from its own start."""
    lv = np.asarray(lv, np.float32)
    xi = ((lv[:-1] + lv[1:]) * np.float32(0.5)).astype(np.float32)
    s1, s0, cnt = np.zeros(16), np.zeros(16), np.zeros(16, np.uint64)
    xs, aw, cs = [], [], []
    err2 = err1 = 0.0
    for t in w:
        for o in range(0, t.size, I):
            blk = t[o:o + I]
            k = int(np.argmax(np.abs(blk)))               # first of the largest magnitudes
            m = np.float32(blk[k] if norm == SGN else abs(blk[k]))
            x = (blk / m).astype(np.float32) if m != 0 else np.zeros_like(blk)
            c = (xi[None, :] <= x[:, None]).sum(1)
            md = float(m)
            np.add.at(s1, c, md * md * x.astype(np.float64))
            np.add.at(s0, c, md * md)
            np.add.at(cnt, c, 1)
            d = blk.astype(np.float64) - md * lv[c].astype(np.float64)     # w - m xhat (App. B.3)
            err2 += float(np.sum(d ** 2))
            err1 += float(np.sum(np.abs(d)))
            xs.append(x), aw.append(np.full(blk.size, abs(md))), cs.append(c)
    return s1, s0, cnt, err2, err1, np.concatenate(xs), np.concatenate(aw), np.concatenate(cs)


@pytest.mark.parametrize("norm", [ABS, SGN])
def test_fit_statistics_of_ragged_tensor_lists_by_hand(norm):
    """Tensors whose lengths are not multiples of the block size: the last block of every tensor
    is a block of its own (its own maximum), and blocks never run across two tensors.  Sums,
    counts, errors and weighted medians against the definitions written out in numpy."""
    rng = np.random.default_rng(21)
    I = 32
    lens = [3 * I + 5, 1, 2 * I, I - 1, 4 * I + 17]
    w = [(rng.standard_normal(n) * rng.uniform(0.01, 0.1)).astype(np.float32) for n in lens]
    lv = np.array(workloads.init_levels_7_0_8(), np.float32)
    s1, s0, cnt, err2, err1, x, a, c = _by_hand_stats(w, I, norm, lv)
    st = oracle.em_accumulate_mse(w, I, norm, lv)
    assert np.array_equal(st["count"], cnt) and st["n"] == sum(lens)
    np.testing.assert_allclose(st["s1"], s1, rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(st["s0"], s0, rtol=1e-12)
    np.testing.assert_allclose(st["err_sum"], err2, rtol=1e-12)
    sa = oracle.em_accumulate_mae(w, I, norm, lv)
    assert np.array_equal(sa["count"], cnt)
    np.testing.assert_allclose(sa["err_sum"], err1, rtol=1e-12)
    for l in range(16):
        xs, ws = x[c == l].astype(np.float64), a[c == l]
        if xs.size == 0:
            assert sa["median"][l] == lv[l]
            continue
        np.testing.assert_allclose(sa["wsum"][l], ws.sum(), rtol=1e-12)
        f = lambda v: np.sum(ws * np.abs(xs - v))
        assert f(float(sa["median"][l])) <= min(f(v) for v in xs) * (1 + 1e-12)
        assert sa["median"][l] in x[c == l]


def test_ragged_fit_is_not_the_fit_of_the_concatenation():
    """The planted mistake: cutting the CONCATENATED data into blocks (blocks running across
    tensor boundaries) gives other block constants; and a ragged tensor equals its whole blocks
    plus the short block fitted as a tensor of its own."""
    rng = np.random.default_rng(22)
    I = 64
    a = (rng.standard_normal(5 * I + 9) * 0.02).astype(np.float32)
    b = (rng.standard_normal(3 * I) * 0.05).astype(np.float32)
    lv = TAB6[:, 4].astype(np.float32)
    both = oracle.em_accumulate_mse([a, b], I, SGN, lv)
    parts = [oracle.em_accumulate_mse(t, I, SGN, lv) for t in (a[:5 * I], a[5 * I:], b)]
    assert np.array_equal(both["count"], sum(p["count"] for p in parts))
    np.testing.assert_allclose(both["s1"], sum(p["s1"] for p in parts), rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(both["s0"], sum(p["s0"] for p in parts), rtol=1e-12)
    cat = np.concatenate([a, b])
    pad = np.concatenate([cat, np.zeros(-cat.size % I, np.float32)])
    wrong = oracle.em_accumulate_mse(pad, I, SGN, lv)
    assert abs(wrong["s0"].sum() - both["s0"].sum()) > 1e-6 * both["s0"].sum()
    # a whole fit over the list runs and never increases the error
    for metric in (MSE, MAE):
        cb, log = oracle.fit([a, b], I, SGN, metric, workloads.init_levels_7_0_8(), FIX4S, 6)
        assert np.all(np.diff(log) <= 1e-15) and np.all(np.diff(cb) > 0)


# --------------------------------------------------------------------------- double quantisation


def test_double_quantisation_by_hand_and_bounds():
    """8-bit uniform quantisation of |m| against the maximum of its group of 256 (the reading
    stated in oracle/double_quant.py), with the sign bit the paper asks for under signed
    normalisation (Limitations)."""
    from oracle import double_quant as dq
    # exact arithmetic: g = 255 -> t = 1, q = |m|
    m = np.array([0.0, 1.0, -2.0, 255.0, -17.0, 100.0, 254.0, -3.0, 7.0], np.float32)
    q, g, sign = dq.compress(m, True)
    assert np.array_equal(q, [0, 1, 2, 255, 17, 100, 254, 3, 7]) and g.tolist() == [255.0]
    assert sign.tolist() == [0b10010100, 0b0]                       # blocks 2, 4, 7 negative; block 8 positive
    assert np.array_equal(dq.expand(q, g, sign, m.size), m)
    # halves round to even: a / t = 0.5 -> 0, 1.5 -> 2, 2.5 -> 2
    m = np.array([255.0, 0.5, 1.5, 2.5], np.float32)
    assert dq.compress(m, False)[0].tolist() == [255, 0, 2, 2]
    # random constants over three groups and a ragged fourth: error bound, signs, group maxima
    rng = np.random.default_rng(31)
    B = 3 * 256 + 57
    m = (np.abs(rng.standard_normal(B)) * 0.05 + 0.01).astype(np.float32) * rng.choice([-1.0, 1.0], B).astype(np.float32)
    m[256:512] *= np.float32(40.0)                                   # a group on another scale
    q, g, sign = dq.compress(m, True)
    assert g.size == 4 and sign.size == (B + 7) // 8
    for k in range(4):
        assert g[k] == np.abs(m[k * 256:(k + 1) * 256]).max()        # own maximum, not the neighbour's
    mh = dq.expand(q, g, sign, B)
    assert np.array_equal(np.signbit(mh), np.signbit(m))             # signs exactly
    bound = np.repeat(g, 256)[:B].astype(np.float64) / 510.0
    assert np.all(np.abs(mh.astype(np.float64) - m) <= bound * (1 + 1e-5))
    assert np.abs(mh.astype(np.float64) - m).max() > 0.3 * bound.max()   # and it is a real quantiser
    # fp64 formula round(255 a / g): identical except where fp32 rounding moves a tie
    ref = np.rint(255.0 * np.abs(m).astype(np.float64) / np.repeat(g, 256)[:B])
    assert np.abs(q.astype(np.int64) - ref).max() <= 1 and (q != ref).mean() < 1e-3
    # unsigned: no sign array, magnitudes only; a zero group stays zero
    q0, g0, s0 = dq.compress(np.zeros(300, np.float32), False)
    assert s0 is None and not q0.any() and not g0.any()
    assert not dq.expand(q0, g0, None, 300).any()


def test_double_quantisation_changes_the_block_maximum():
    """With exact constants the element of largest magnitude of a block is reconstructed exactly
    (Sec. 3.1); after double quantisation only the LARGEST constant of a group comes back within
    an fp32 rounding of itself, every other one moves by up to g/510, and with it the block's
    maximum.  The codes stay those formed with the exact constant."""
    from oracle import double_quant as dq
    rng = np.random.default_rng(32)
    I, B = 64, 512
    w = (rng.standard_normal(B * I) * 0.02).astype(np.float32)
    lv = TAB6[:, 4].astype(np.float32)
    codes, m = oracle.quantize(w, I, SGN, lv)
    q, g, sign = dq.compress(m, True)
    mh = dq.expand(q, g, sign, B)
    for k in range(2):
        top = np.argmax(np.abs(m[k * 256:(k + 1) * 256])) + k * 256
        assert q[top] == 255 and abs(float(mh[top]) - float(m[top])) <= 2.0 ** -22 * abs(float(m[top]))
    assert (mh != m).mean() > 0.9
    exact = oracle.dequantize(codes, m, I, lv)
    dq_out = oracle.dequantize(codes, mh, I, lv)
    peak = np.abs(w.reshape(B, I)).argmax(1) + np.arange(B) * I
    assert np.array_equal(exact[peak], w[peak])                      # the property with exact constants
    assert (dq_out[peak] != w[peak]).mean() > 0.9                    # and what double quantisation gives up
    assert np.abs(dq_out - exact).max() <= np.abs(mh - m).max() * (1 + 1e-6)   # |xhat| <= 1


# --------------------------------------------------------------------------- general weight densities


def test_tabulated_model_reproduces_the_gaussian_solver():
    """Eq. 5 / Eq. 7 for a tabulated density, fed a Gaussian table, against the closed Gaussian
    forms (boxed equations of App. B.2): centroids of single regions and a whole Lloyd run."""
    w = np.linspace(0.0, 10.0, 20001)
    tab = theory.TabulatedBlockModel(64, 10.0, np.exp(-0.5 * w * w))     # unnormalised on purpose
    gau = theory.GaussianBlockModel(64)
    for lo, hi in ((-1.0, -0.6), (-0.3, -0.1), (-0.04, 0.05), (0.2, 0.45), (0.6, 0.9)):
        assert abs(tab.mse_centroid(lo, hi) - gau.mse_centroid(lo, hi)) < 2e-7
        assert abs(tab.mae_centroid(lo, hi) - gau.mae_centroid(lo, hi)) < 2e-7
        assert abs(tab.cont_prob(lo, hi) - gau.cont_prob(lo, hi)) < 2e-7
    for signed, mask in ((False, FIX4), (True, FIX4S)):
        for metric in ("mse", "mae"):
            a = theory.lloyd(64, signed, metric, workloads.init_levels_7_0_8(), mask, 5, tab)
            b = theory.lloyd(64, signed, metric, workloads.init_levels_7_0_8(), mask, 5, gau)
            assert np.abs(a - b).max() < 5e-7


@pytest.mark.parametrize("signed,norm,mask", [(False, ABS, FIX4), (True, SGN, FIX4S)])
@pytest.mark.parametrize("metric", ["mse", "mae"])
def test_tabulated_model_agrees_with_data_driven_fit_on_laplace_weights(signed, norm, mask, metric):
    """A density that is not Gaussian: 2^24 Laplace samples.  One data-driven EM step (Eq. 6 /
    Eq. 8) and one theoretical step (Eq. 5 / Eq. 7, p_W tabulated) from the same start agree
    within Monte-Carlo noise, and the Gaussian model does NOT (the general formula is needed)."""
    w = oracle.as_f32(workloads.laplace(1 << 24, 1.0, 321))
    grid = np.linspace(0.0, 40.0, 40001)
    tab = theory.TabulatedBlockModel(64, 40.0, 0.5 * np.exp(-grid))
    start = workloads.init_levels_7_0_8()
    theo = theory.lloyd(64, signed, metric, start, mask, 1, tab)
    lv, _ = oracle.fit(w, 64, norm, MSE if metric == "mse" else MAE, start, mask, 1)
    # the outer regions of the heavy-tailed density hold few samples: the median of region 1
    # (some 1e4 members) moves by a few 1e-4 from sample to sample
    assert np.abs(lv - theo).max() < (4e-4 if metric == "mse" else 1e-3)
    gau = theory.lloyd(64, signed, metric, start, mask, 1, theory.GaussianBlockModel(64, points=4001))
    assert np.abs(lv - gau).max() > 5e-3


# --------------------------------------------------------------------------- batched consumer


def test_batched_product_with_bf16_weights_by_hand_and_against_gemv():
    """gemm_bf16 = the decoded product for several right-hand sides with the dequantised weight
    rounded to bf16.  (i) A 2 x 64 matrix by hand.  (ii) Where scale * level is exact in bf16
    (power-of-two constants, levels with few significant bits) every column equals the pinned
    matrix-vector product `gemv`.  (iii) With generic levels it differs from `gemv` by the bf16
    rounding of the weights (relative 2^-9 at most, and not zero)."""
    I, rows, cols = 32, 2, 64
    lv = ((np.arange(16) - 7.5) / 8.0).astype(np.float32)                 # multiples of 1/16: 5 significant bits
    rng = np.random.default_rng(41)
    c = rng.integers(0, 16, rows * cols).astype(np.uint8)
    codes = ((c[0::2] << 4) | c[1::2]).astype(np.uint8)
    scales = np.array([0.5, -2.0, 1.0, 0.25], np.float32)                 # four blocks of 32
    X = rng.integers(-3, 4, (3, cols)).astype(np.float32)
    Y, mag = oracle.gemm_bf16(codes, scales, rows, cols, I, lv, X)
    W = (lv[c].astype(np.float64) * np.repeat(scales.astype(np.float64), I)).reshape(rows, cols)
    assert np.array_equal(Y, W @ X.astype(np.float64).T)                  # (i): exact small integers / 16
    assert np.array_equal(mag, np.abs(W) @ np.abs(X.astype(np.float64)).T)
    for b in range(3):                                                    # (ii)
        y, m = oracle.gemv(codes, scales, rows, cols, I, lv, X[b])
        assert np.array_equal(Y[:, b], y) and np.array_equal(mag[:, b], m)
    # an outlier replaces exactly one weight: Y moves by (val - W[r, c]) * X[:, c] in its row only
    val = oracle.f32_to_bf16_bits(np.array([3.5], np.float32))
    Yo, _ = oracle.gemm_bf16(codes, scales, rows, cols, I, lv, X, np.array([cols + 5]), val)
    assert np.array_equal(Yo[0], Y[0])
    assert np.array_equal(Yo[1] - Y[1], (3.5 - W[1, 5]) * X[:, 5].astype(np.float64))
    lv2 = TAB6[:, 4].astype(np.float32)                                   # (iii)
    scales2 = np.array([0.0131, -0.0207, 0.0179, 0.0093], np.float32)
    Y2, mag2 = oracle.gemm_bf16(codes, scales2, rows, cols, I, lv2, X)
    for b in range(3):
        y, m = oracle.gemv(codes, scales2, rows, cols, I, lv2, X[b])
        assert np.all(np.abs(Y2[:, b] - y) <= 2.0 ** -9 * m)
        assert np.any(Y2[:, b] != y)
