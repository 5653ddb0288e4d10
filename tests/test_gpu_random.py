"""Randomised parity: every entry point against the oracle on seeded random shapes, block sizes,
dtypes, normalisations, codebooks and scales of the data (a sweep that no hand-picked case
list covers).  Same bars as the other parity tests: bit-exact codes, scales, outlier lists,
dequantised bits, member counts and MAE medians; 1e-5 relative for the fp sums."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def _random_levels(rng):
    """16 distinct ascending levels in [-1, 1] containing -1 or a free lowest level, 0 and 1."""
    inner = np.concatenate([-rng.uniform(0.02, 0.98, 6), rng.uniform(0.02, 0.98, 7)])
    lv = np.concatenate([[-1.0 if rng.random() < 0.5 else -rng.uniform(0.985, 0.999)], inner, [0.0, 1.0]])
    lv = np.unique(lv.astype(np.float32))
    assert lv.size == 16
    return lv


@pytest.mark.parametrize("seed", range(8))
def test_random_cases_match_the_oracle(bof4, seed):
    rng = np.random.default_rng(1000 + seed)
    dev = "cuda:0"
    for _ in range(6):
        I = int(rng.choice([32, 64, 128, 256, 512, 1024, 2048, 4096]))
        nb = int(rng.integers(1, max(2, (1 << 18) // I)))
        n = nb * I
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        norm = int(rng.integers(0, 2))
        lv = _random_levels(rng)
        sigma = float(10 ** rng.uniform(-4, 1))
        w = workloads.gaussian_student_mixture(n, sigma, 0.02, 3, int(rng.integers(1 << 30)), dtype)
        if rng.random() < 0.3:
            w[rng.integers(0, n, max(1, n // 500))] *= 15
        if rng.random() < 0.2:
            k = int(rng.integers(0, nb))
            w[k * I:(k + 1) * I] = 0
        wd = w.to(dev)
        tag = "I=%d blocks=%d %s norm=%d sigma=%.3g" % (I, nb, dtype, norm, sigma)
        codes, scales = bof4.bof4_quantize(wd, I, norm, lv)
        rc, rs = oracle.quantize(w, I, norm, lv)
        assert np.array_equal(codes.cpu().numpy(), rc), tag
        assert np.array_equal(scales.float().cpu().numpy(), rs), tag
        out = bof4.bof4_dequantize(codes, scales, I, lv, bof4.BF16)
        ro = oracle.f32_to_bf16_bits(oracle.dequantize(rc, rs, I, lv))
        assert np.array_equal(out.view(torch.int16).cpu().numpy().view(np.uint16), ro), tag
        tau = float(np.float32(bof4.bof4_opq_threshold(float(rng.uniform(0.8, 0.99)), I)))
        c2, s2, idx, val, cnt = bof4.bof4_quantize_opq(wd, I, norm, lv, tau, n)
        clean, ridx, rval, rk = oracle.opq_split(w, I, tau)
        k = int(cnt.item())
        assert k == rk, tag
        assert np.array_equal(idx[:k].cpu().numpy().astype(np.int64), ridx), tag
        assert np.array_equal(val[:k].view(torch.int16).cpu().numpy().view(np.uint16), rval), tag
        rc2, rs2 = oracle.quantize(clean, I, norm, lv)
        assert np.array_equal(c2.cpu().numpy(), rc2), tag
        assert np.array_equal(s2.float().cpu().numpy(), rs2), tag
        got = bof4.bof4_em_step([wd], I, norm, bof4.METRIC_MSE, lv)
        ref = oracle.em_accumulate_mse(w, I, norm, lv)
        assert np.array_equal(got["count"], ref["count"]), tag
        np.testing.assert_allclose(got["s1"], ref["s1"], rtol=1e-5, atol=1e-5 * np.abs(ref["s1"]).max() + 1e-30)
        np.testing.assert_allclose(got["s0"], ref["s0"], rtol=1e-5)
        np.testing.assert_allclose(got["err_sum"], ref["err_sum"], rtol=1e-5)
        got = bof4.bof4_em_step([wd], I, norm, bof4.METRIC_MAE, lv)
        ref = oracle.em_accumulate_mae(w, I, norm, lv)
        assert np.array_equal(got["count"], ref["count"]), tag
        assert np.array_equal(got["median"], ref["median"]), tag
        np.testing.assert_allclose(got["err_sum"], ref["err_sum"], rtol=1e-5)
        cols = I * int(rng.integers(1, max(2, min(8, nb))))
        if n % cols == 0 and cols <= 32768:
            rows = n // cols
            x = workloads.gaussian(cols, 1.0, 5, torch.bfloat16)
            y = bof4.bof4_gemv(c2, s2, rows, cols, I, lv, x.to(dev), (idx, val, cnt)).cpu().numpy()
            ry, mag = oracle.gemv(rc2, rs2, rows, cols, I, lv, x.float().numpy(), ridx, rval)
            assert np.all(np.abs(y - ry) <= 64 * 2.0 ** -24 * mag + 1e-300), tag
