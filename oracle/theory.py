"""Theoretical (data-free) centroid rules, by quadrature: unit-variance Gaussian weights
(GaussianBlockModel) and any tabulated symmetric density (TabulatedBlockModel).

TEST INFRASTRUCTURE ONLY.  Used to pin the data-driven oracle against the paper's claim that
the Monte-Carlo centroid and the analytical centroid are equivalent (Sec. 3.2, App. B.2, App. C).

Notation (App. B.1): g, G = pdf / cdf of N(0,1); M = absolute block maximum with
p_M(m) = 2 I (2G(m)-1)^(I-1) g(m); given M = m the other I-1 normalised weights are i.i.d.
with continuous cdf F_cont(x | m) = (G(m x) - G(-m)) / (2G(m) - 1) on (-1, 1).

Readings of garbled formulas:
 * the boxed Gaussian MSE centroid (last equation of "Simplified Solution for Gaussian Network
   Weights") has lost the leading minus sign that the two equations before it carry; the
   sign is restored here (without it every centroid would have the wrong sign);
 * the boxed MAE condition (last equation of "MAE Optimization", App. B.2) is read with the
   conditional cdf of its derivation, F(xh | m, X in R) = (F(xh|m) - F(xi_lo|m)) / [F]_lo^hi,
   i.e. the term F(xi_lo | m) that the printed box drops is kept.
"""
from __future__ import annotations

import numpy as np
from scipy.special import ndtr

_SQRT2PI = np.sqrt(2.0 * np.pi)


def _g(x):
    return np.exp(-0.5 * x * x) / _SQRT2PI


class GaussianBlockModel:
    """Quadrature grid over the block maximum m in (0, m_max] for block size I."""

    def __init__(self, I: int, m_max: float = 10.0, points: int = 20001):
        self.I = I
        self.m = np.linspace(0.0, m_max, points)[1:]
        self.dm = self.m[1] - self.m[0]
        G = ndtr(self.m)
        # (2G-1)^(I-2) g(m): common factor of every integrand below
        self.core = np.power(2.0 * G - 1.0, I - 2) * _g(self.m)

    def _int(self, f):
        # trapezoid; every integrand vanishes at m = 0
        return (f.sum() - 0.5 * f[-1]) * self.dm

    # -- MSE centroid of a region (lo, hi) inside (-1, 1): boxed Gaussian solution, sign fixed
    def mse_centroid(self, lo: float, hi: float) -> float:
        m = self.m
        num = -self._int(m * (_g(m * hi) - _g(m * lo)) * self.core)
        den = self._int(m * m * (ndtr(m * hi) - ndtr(m * lo)) * self.core)
        return num / den

    # -- MAE centroid: weighted median of the re-weighted density, by bisection
    def _mae_mass(self, lo: float, x: float) -> float:
        m = self.m
        return self._int(m * (ndtr(m * x) - ndtr(m * lo)) * self.core)

    def mae_centroid(self, lo: float, hi: float) -> float:
        half = 0.5 * self._mae_mass(lo, hi)
        a, b = lo, hi
        for _ in range(60):
            c = 0.5 * (a + b)
            if self._mae_mass(lo, c) < half:
                a = c
            else:
                b = c
        return 0.5 * (a + b)

    # -- probability of the continuous part falling into (lo, hi): P[lo < X < hi | |X| < 1]
    def cont_prob(self, lo: float, hi: float) -> float:
        m = self.m
        return 2.0 * self.I * self._int((ndtr(m * hi) - ndtr(m * lo)) * self.core)


class TabulatedBlockModel:
    """The same centroid rules for ANY symmetric zero-mean weight density (Sec. 3.2 Eq. 5 and
    Eq. 7 with App. B.1 / B.2: the cdf of X given M = m, the density of M, the conditional
    expectation of X for fixed m), the density given as samples p_W(w_j) on the uniform grid
    w_j = j * w_max / (len(pdf) - 1), j >= 0.

    With F_W(w) = 1/2 + Fc(w), Fc(w) = INT_0^w p_W (odd), and H(w) = INT_0^w u p_W(u) du (even), the
    density of M is 2I (2 Fc(m))^(I-1) p_W(m), the cdf of X given m on (-1, 1) is
    (F_W(m x) - F_W(-m)) / (2 Fc(m)), and INT_R m x p_W(m x) dx = [H(m x)]_R / m, so that
        MSE centroid = INT m [H(m x)]_lo^hi c(m) dm / INT m^2 [Fc(m x)]_lo^hi c(m) dm,
        MAE centroid = the x with INT m [Fc(m x)]_lo^x c(m) dm = 1/2 INT m [Fc(m x)]_lo^hi c(m) dm,
    c(m) = (2 Fc(m))^(I-2) p_W(m): the Gaussian formulas with G -> F_W and -g -> H.

    Numerics: the samples are scaled to total mass 1 on [-w_max, w_max]; Fc and H are cumulative
    trapezoid sums on the grid, evaluated between nodes by linear interpolation; the integrals
    over m use the trapezoid rule on the same grid (w_max must cover the block maximum's range).
    """

    def __init__(self, I: int, w_max: float, pdf):
        p = np.asarray(pdf, dtype=np.float64)
        self.I = I
        self.m = np.linspace(0.0, w_max, p.size)
        self.dm = self.m[1] - self.m[0]
        half = (p.sum() - 0.5 * (p[0] + p[-1])) * self.dm
        p = p / (2.0 * half)
        self.p = p
        self.Fc = np.concatenate(([0.0], np.cumsum(0.5 * (p[1:] + p[:-1]) * self.dm)))
        up = self.m * p
        self.H = np.concatenate(([0.0], np.cumsum(0.5 * (up[1:] + up[:-1]) * self.dm)))
        self.core = np.power(2.0 * self.Fc, I - 2) * p

    def _Fc(self, w):
        return np.sign(w) * np.interp(np.abs(w), self.m, self.Fc)

    def _H(self, w):
        return np.interp(np.abs(w), self.m, self.H)

    def _int(self, f):
        return (f.sum() - 0.5 * (f[0] + f[-1])) * self.dm

    def mse_centroid(self, lo: float, hi: float) -> float:
        m = self.m
        num = self._int(m * (self._H(m * hi) - self._H(m * lo)) * self.core)
        den = self._int(m * m * (self._Fc(m * hi) - self._Fc(m * lo)) * self.core)
        return num / den

    def _mae_mass(self, lo: float, x: float) -> float:
        m = self.m
        return self._int(m * (self._Fc(m * x) - self._Fc(m * lo)) * self.core)

    mae_centroid = GaussianBlockModel.mae_centroid

    def cont_prob(self, lo: float, hi: float) -> float:
        m = self.m
        return 2.0 * self.I * self._int((self._Fc(m * hi) - self._Fc(m * lo)) * self.core)


def lloyd(I: int, signed: bool, metric: str, levels0, fixed_mask: int, iters: int,
          model=None) -> np.ndarray:
    """Lloyd iteration with the theoretical centroid for every free level.

    Thresholds are midpoints.  Free levels must own a region inside [-1, 1): the outermost
    levels are either fixed (absolute normalisation: -1 and 1; signed: 1) or, for the
    leftmost level under signed normalisation, use lo = -1 (no point mass there, App. B.2).
    """
    mdl = model or GaussianBlockModel(I)
    lv = np.array(levels0, dtype=np.float64)
    cen = mdl.mse_centroid if metric == "mse" else mdl.mae_centroid
    for _ in range(iters):
        xi = 0.5 * (lv[:-1] + lv[1:])
        new = lv.copy()
        for l in range(16):
            if (fixed_mask >> l) & 1:
                continue
            lo = xi[l - 1] if l > 0 else -1.0
            hi = xi[l] if l < 15 else 1.0
            if l == 0:
                assert signed, "leftmost level carries a point mass under absolute normalisation"
            assert l < 15, "rightmost level carries a point mass; it must be fixed"
            new[l] = cen(max(lo, -1.0), min(hi, 1.0))
        lv = new
    return lv


def region_probabilities(levels, I: int, signed: bool,
                         model: GaussianBlockModel | None = None) -> np.ndarray:
    """P[X in R_l] under the cdf of the normalised weights (App. B.1, last two equations):
    the continuous part carries (I-1)/I; the mass 1/I sits at +1 (signed) or is split
    between -1 and +1 (absolute)."""
    mdl = model or GaussianBlockModel(I)
    lv = np.asarray(levels, dtype=np.float64)
    xi = np.concatenate(([-1.0], 0.5 * (lv[:-1] + lv[1:]), [1.0]))
    p = np.array([mdl.cont_prob(xi[l], xi[l + 1]) for l in range(16)]) * (I - 1) / I
    if signed:
        p[15] += 1.0 / I
    else:
        p[0] += 0.5 / I
        p[15] += 0.5 / I
    return p
