"""The rule behind the reciprocal fast path of the bf16 kernels, checked on the CPU in IEEE fp32.

The kernels assign a bf16 weight w of a block with constant m to a region by comparing
x~ = RN(w * RN(1/m)) with thresholds lowered by three fp32 steps, instead of comparing the true
quotient RN(w / m) with the thresholds themselves (Sec. 2.1 Eq. 2, Sec. 3.2).  They do so only for
block constants whose 8-bit significand is not marked "near" by an integer test on (threshold,
significand) pairs.  This file restates that test and enumerates every bf16 operand pair (all
significands, both signs, a range of exponents) for several codebooks, including dyadic ones
whose thresholds are hit exactly by quotients and adversarial ones whose thresholds sit a few
steps around quotients: wherever the significand is not marked, both comparisons must count
the same number of thresholds.  numpy's float32 arithmetic is IEEE round-to-nearest-even."""
import numpy as np
import pytest

import workloads

F = np.float32


def thresholds(levels):
    lv = np.asarray(levels, F)
    return ((lv[:-1] + lv[1:]) * F(0.5)).astype(F)


def three_steps_down(xi):
    u = xi.view(np.uint32).astype(np.int64)
    return np.where(u >> 31, u + 3, u - 3).astype(np.uint32).view(F)


def near_mask(xi):
    """bit b-128 set: some quotient a/b * 2^j lies between a quarter of an fp32 step and
    16 * 2^-24 (relative) below a threshold (one unit of P = X b is 1/b of a step of xi)."""
    mask = np.zeros(128, bool)
    for t in xi:
        bits = int(np.asarray(t, F).view(np.uint32))
        xb = bits & 0x7fffffff
        assert 0x12800000 <= xb < 0x7f800000           # |xi| >= 2^-90 and finite (else the path is off)
        X = (xb & 0x7fffff) | 0x800000
        for b in range(128, 256):
            P = X * b
            s = 24 if P >> 31 else 23
            frac = P & ((1 << s) - 1)
            dist = ((1 << s) - frac) & ((1 << s) - 1) if bits >> 31 else frac
            mask[b - 128] |= (4 * dist >= b) and (dist <= (P >> 20))
    return mask


def operand_grid(exps=range(0, -14, -1)):
    """All (w, m): m = b (128..255), w = +-a * 2^j (a = 0..255, j <= 0) -- every bf16 pair up to scale."""
    b = np.arange(128, 256, dtype=np.float64)
    a = np.arange(0, 256, dtype=np.float64)
    ws = np.concatenate([s * a * 2.0 ** j for j in exps for s in (1.0, -1.0)])
    return ws.astype(F), b.astype(F)


def check_codebook(levels, m_signs=(1.0, -1.0), scale=1.0):
    xi = thresholds(levels)
    lo = three_steps_down(xi)
    mask = near_mask(xi)
    ws, bs = operand_grid()
    n_checked = 0
    for sg in m_signs:
        for k, b in enumerate(bs):
            if mask[k]:
                continue
            m = F(sg * b * scale)
            w = (ws * F(scale)).astype(F)
            w = w[np.abs(w) <= abs(m)]
            x = (w / m).astype(F)                       # RN(w / m)
            r = (F(1.0) / m).astype(F)                  # RN(1 / m)
            xt = (w * r).astype(F)                      # x~
            true = (x[:, None] >= xi[None, :]).sum(1)
            fast = (xt[:, None] >= lo[None, :]).sum(1)
            assert np.array_equal(true, fast), (b, sg, w[true != fast][:4])
            n_checked += w.size
    return mask.mean(), n_checked


def test_printed_and_starting_codebooks():
    """The printed BOF4-S codebook (Tab. 6) and the two starting codebooks with rational levels:
    exact threshold hits (e.g. x = 1/16 against the threshold 1/16) are decided like the true
    quotient.  No significand is marked for the printed codebook; the sevenths and fifteenths of
    the starting codebooks mark the significands that are multiples of 7 resp. 3 and 5 wherever
    the fp32 rounding of a threshold leaves a quotient more than a quarter step below it."""
    for lv, most in ((workloads.BOF4S_MSE_I64, 0.0), (workloads.init_levels_7_0_8(), 0.15),
                     (workloads.init_levels_linspace(), 0.5)):
        frac, n = check_codebook(lv)
        assert n > 500_000 * (1.0 - most)
        assert frac <= most


def test_scale_does_not_matter_within_the_safe_range():
    for scale in (2.0 ** -40, 2.0 ** 31):
        check_codebook(workloads.BOF4S_MSE_I64, scale=scale)


def test_adversarial_thresholds_around_quotients():
    """Codebooks whose thresholds are placed 0, 1, 2, 3, 5, 9, 20 fp32 steps above and below
    quotients a/b: the marked significands must cover every disagreement."""
    rng = np.random.default_rng(5)
    for trial in range(12):
        a = rng.integers(1, 256, 15)
        b = rng.integers(128, 256, 15)
        q = np.sort(np.unique((a / b * 2.0 ** rng.integers(-4, 1, 15)) * rng.choice([-1.0, 1.0], 15)))
        q = q[np.abs(q) < 0.999][:15].astype(F)
        if q.size < 15:
            continue
        steps = rng.choice([0, 1, 2, 3, 5, 9, 20, -1, -2, -3, -5, -9, -20], 15)
        bits = q.view(np.uint32).astype(np.int64)
        xi = np.where(bits >> 31, bits - steps, bits + steps).astype(np.uint32).view(F)   # + = upwards
        xi = np.sort(xi)
        if np.any(np.diff(xi) <= 0):
            continue
        # levels whose midpoints are these thresholds do not exist in general: test the rule on the
        # thresholds directly
        lo = three_steps_down(xi)
        mask = near_mask(xi)
        ws, bs = operand_grid(range(0, -8, -1))
        bad_unmarked = 0
        for k, bb in enumerate(bs):
            m = F(bb)
            w = ws[np.abs(ws) <= bb]
            x = (w / m).astype(F)
            xt = (w * (F(1.0) / m).astype(F)).astype(F)
            differ = (x[:, None] >= xi[None, :]).sum(1) != (xt[:, None] >= lo[None, :]).sum(1)
            if differ.any():
                assert mask[k], (trial, bb)
            bad_unmarked += int(differ.any() and not mask[k])
        assert bad_unmarked == 0
        assert mask.mean() < 0.6


def test_without_the_marking_the_fast_comparison_is_wrong_somewhere():
    """The planted mistake: ignoring the marks (or not lowering the thresholds) does produce wrong
    regions for some operand pair, so the two devices of the rule are both needed."""
    xi = thresholds(workloads.init_levels_7_0_8())
    ws, bs = operand_grid(range(0, -8, -1))
    wrong_plain = 0
    for bb in bs:
        m = F(bb)
        w = ws[np.abs(ws) <= bb]
        x = (w / m).astype(F)
        xt = (w * (F(1.0) / m).astype(F)).astype(F)
        wrong_plain += int(((x[:, None] >= xi[None, :]).sum(1) != (xt[:, None] >= xi[None, :]).sum(1)).sum())
    assert wrong_plain > 0      # x~ against the unlowered thresholds misplaces exact hits
    # a threshold three steps above a quotient 200/173: lowered, it sits right on x~'s uncertainty
    q = F(200.0) / F(173.0) * F(0.25)
    t = (q.view(np.uint32) + np.uint32(2)).view(F)
    xi2 = np.sort(np.append(xi[np.abs(xi - t) > 1e-3], t)).astype(F)[:15]
    assert near_mask(xi2)[173 - 128]
