"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module only draws random numbers and lays out shapes. It contains none of the
quantisation arithmetic (no block maxima, no normalisation, no level search), so both the CPU
oracle and the CUDA library can be fed from it without sharing any of the method's code.

Every generator is deterministic in its seed. The shapes follow the public transformer
architectures whose weight matrices the paper quantises (Sec. 4, "Quantized Models"); the
values follow the near-Gaussian weight distribution the paper assumes (Sec. 4, "Evaluated
Quantization Methods"; Appendix E.1), with heavy-tailed or injected outliers where a workload
exercises the outlier-preserving path (Sec. 3.3).
"""
from __future__ import annotations

import math
from typing import Iterator, List, Tuple

import torch

# ----------------------------------------------------------------------------------------
# Small generic generators (CPU or CUDA, decided by `device`)
# ----------------------------------------------------------------------------------------


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gaussian(n: int, sigma: float, seed: int, dtype=torch.float32, device="cpu") -> torch.Tensor:
    """n i.i.d. N(0, sigma^2) samples, drawn in fp32 and rounded (RN) to `dtype`."""
    x = torch.randn(n, generator=_gen(seed, device), device=device, dtype=torch.float32)
    x.mul_(sigma)
    return x.to(dtype)


def laplace(n: int, b: float, seed: int, dtype=torch.float32, device="cpu") -> torch.Tensor:
    """n samples of the Laplace density exp(-|w| / b) / (2 b) (inverse-cdf method)."""
    u = torch.rand(n, generator=_gen(seed, device), dtype=torch.float64, device=device) - 0.5
    w = -b * torch.sign(u) * torch.log1p(-2.0 * u.abs())
    return w.to(dtype)


def gaussian_student_mixture(n: int, sigma: float, frac_t: float, nu: int, seed: int,
                             dtype=torch.bfloat16, device="cpu") -> torch.Tensor:
    """(1-frac_t) N(0, sigma^2) + frac_t * sigma * Student-t(nu).

    The t variate is z / sqrt(chi2_nu / nu) with chi2_nu a sum of nu squared normals.
    """
    g = _gen(seed, device)
    base = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    pick = torch.rand(n, generator=g, device=device) < frac_t
    k = int(pick.sum().item())
    if k:
        z = torch.randn(k, generator=g, device=device, dtype=torch.float32)
        chi2 = torch.randn(k, nu, generator=g, device=device, dtype=torch.float32).pow_(2).sum(1)
        base[pick] = z / torch.sqrt(chi2 / nu)
    base.mul_(sigma)
    return base.to(dtype)


def inject_outliers(w: torch.Tensor, sigma: float, rate: float, lo: float, hi: float,
                    seed: int) -> torch.Tensor:
    """Replace about `rate` of the entries, at seeded uniform positions, by +-U[lo,hi]*sigma."""
    n = w.numel()
    k = int(round(n * rate))
    if k == 0:
        return w
    g = _gen(seed, w.device)
    pos = torch.randint(0, n, (k,), generator=g, device=w.device)
    mag = (torch.rand(k, generator=g, device=w.device) * (hi - lo) + lo) * sigma
    sgn = torch.randint(0, 2, (k,), generator=g, device=w.device).float() * 2 - 1
    flat = w.view(-1)
    flat[pos] = (mag * sgn).to(w.dtype)
    return w


# ----------------------------------------------------------------------------------------
# The five workload configurations
# ----------------------------------------------------------------------------------------

C1_N = 1 << 20
C2_N = 1 << 26


def config1(device="cpu") -> torch.Tensor:
    """2^20 fp32 weights, N(0, 0.02^2), seed 0."""
    return gaussian(C1_N, 0.02, 0, torch.float32, device)


def config2(n: int = C2_N, device="cpu") -> torch.Tensor:
    """bf16 weights: 99 % N(0, 0.02^2) + 1 % 0.02 * Student-t(nu=4), seed 1."""
    return gaussian_student_mixture(n, 0.02, 0.01, 4, 1, torch.bfloat16, device)


def llama7b_shapes() -> List[Tuple[int, int]]:
    """32 layers x {4 x 4096x4096, 3 x 4096x11008}: 224 matrices, 6,476,005,376 weights."""
    layer = [(4096, 4096)] * 4 + [(4096, 11008)] * 3
    return layer * 32


def llama3_8b_shapes() -> List[Tuple[int, int]]:
    """32 layers x {4096x4096, 1024x4096 x2, 4096x4096, 14336x4096 x2, 4096x14336}."""
    layer = [(4096, 4096), (1024, 4096), (1024, 4096), (4096, 4096),
             (14336, 4096), (14336, 4096), (4096, 14336)]
    return layer * 32


def llama70b_layer_shapes() -> List[Tuple[int, int]]:
    """One of the 80 layers: {8192x8192, 1024x8192 x2, 8192x8192, 28672x8192 x2, 8192x28672}."""
    return [(8192, 8192), (1024, 8192), (1024, 8192), (8192, 8192),
            (28672, 8192), (28672, 8192), (8192, 28672)]


def config3_sigmas() -> List[float]:
    """Per-matrix sigma ~ U[0.01, 0.04] for the 224 matrices, drawn first from seed 2."""
    g = _gen(2, "cpu")
    u = torch.rand(len(llama7b_shapes()), generator=g, dtype=torch.float64)
    return (0.01 + 0.03 * u).tolist()


def config3_matrices(device="cpu", row_divisor: int = 1,
                     layers: int = 32) -> Iterator[Tuple[int, torch.Tensor]]:
    """Yield (index, flattened bf16 matrix) for the fitting sweep.

    `row_divisor` > 1 keeps the first rows/row_divisor rows of every matrix (the reduced set
    used where the CPU oracle must finish in seconds); `layers` < 32 keeps the first layers.
    Each matrix has its own seed 2_000_000 + index, so any subset reproduces the same bits.
    """
    sig = config3_sigmas()
    for i, (r, c) in enumerate(llama7b_shapes()[: layers * 7]):
        rows = max(1, r // row_divisor)
        yield i, gaussian(rows * c, sig[i], 2_000_000 + i, torch.bfloat16, device)


def config4_matrices(device="cpu", row_divisor: int = 1,
                     layers: int = 32) -> Iterator[Tuple[int, torch.Tensor]]:
    """Yield (index, flattened bf16 matrix), N(0, 0.02^2), per-matrix seed 3_000_000 + index."""
    for i, (r, c) in enumerate(llama3_8b_shapes()[: layers * 7]):
        rows = max(1, r // row_divisor)
        yield i, gaussian(rows * c, 0.02, 3_000_000 + i, torch.bfloat16, device)


def config5_layer(layer: int, device="cpu", row_divisor: int = 1) -> List[torch.Tensor]:
    """The seven bf16 matrices of one 70B-shaped layer: N(0, 0.015^2) with 0.01 % of the
    entries replaced by +-(10..40) sigma outliers. Seeds 4_000_000 + 16*layer + j."""
    out = []
    for j, (r, c) in enumerate(llama70b_layer_shapes()):
        rows = max(1, r // row_divisor)
        s = 4_000_000 + 16 * layer + j
        w = gaussian(rows * c, 0.015, s, torch.bfloat16, device)
        out.append(inject_outliers(w, 0.015, 1e-4, 10.0, 40.0, s + 8))
    return out


# ----------------------------------------------------------------------------------------
# Initial codebooks (inputs to the fit; both sides receive the same 16 floats)
# ----------------------------------------------------------------------------------------


def init_levels_7_0_8() -> List[float]:
    """7 evenly spaced negative levels from -1, the level 0, 8 evenly spaced positive levels
    up to 1: the 7 / zero / 8 split of the paper's printed codebooks (Tab. 6)."""
    neg = [-1.0 + k / 7.0 for k in range(7)]
    pos = [k / 8.0 for k in range(1, 9)]
    return neg + [0.0] + pos


def init_levels_linspace() -> List[float]:
    """16 evenly spaced levels in [-1, 1] with index 7 overwritten by 0."""
    lv = [(-1.0 + 2.0 * k / 15.0) for k in range(16)]
    lv[7] = 0.0
    return lv


# The printed BOF4-S (MSE) codebook for block size 64 (Tab. 6): the levels the quantise /
# dequantise throughput runs use (an input, like the starting codebooks above).
BOF4S_MSE_I64 = [-0.8568463921546936, -0.6692874431610107, -0.5235266089439392, -0.4004882574081421,
                 -0.2910638153553009, -0.1900092959403992, -0.0938529595732689, 0.0,
                 0.0887671709060669, 0.1794802695512772, 0.2743096053600311, 0.3760197460651398,
                 0.4886530041694641, 0.6188603639602661, 0.7791395783424377, 1.0]

FIXED_BOF4 = (1 << 0) | (1 << 7) | (1 << 15)   # levels -1, 0, 1 (absolute normalisation)
FIXED_BOF4S = (1 << 7) | (1 << 15)             # levels 0, 1 (signed normalisation)
