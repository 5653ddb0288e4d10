"""ctypes front-end of the CPU oracle (``bof4_oracle.c``) and the theoretical solver.

TEST INFRASTRUCTURE ONLY: the plain, slow definition of what the CUDA library must compute.
Nothing in the product package imports this module, and this module imports nothing from
the product package.  Inputs are CPU torch tensors or numpy arrays; bf16 inputs are widened
to fp32 (exact) before they reach the C code.

Parity pins: the C functions as listed in ``bof4_oracle.c``; ``gemv`` (fp64 numpy, the plain
definition of the decoded matrix-vector product) by hand-built closed forms and numpy's matvec
of the separately dequantised and restored matrix; ``gemm_bf16`` by a hand-built case, by its
columns equalling ``gemv`` wherever the products of Eq. 3 are exact in bf16, and by the size of
the bf16 rounding where they are not (tests/test_oracle_pins.py).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

try:  # torch is only used to accept bf16 tensors
    import torch
except Exception:  # pragma: no cover
    torch = None

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bof4_oracle.c")
_LIB = os.path.join(_HERE, "libbof4_oracle.so")
_lib = None

METRIC_MSE, METRIC_MAE = 0, 1
METRIC_MSE_NORMDOM, METRIC_MAE_NORMDOM = 2, 3  # App. D: errors of the normalised weights
NORM_ABS, NORM_SIGNED = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with strict IEEE flags.  Building the checker is not using it."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
           "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.orc_opq_split.restype = ctypes.c_int64
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


# --------------------------------------------------------------------------- marshalling


def as_f32(w) -> np.ndarray:
    """Flattened, contiguous fp32 numpy view/copy of a tensor (bf16 widened exactly)."""
    if torch is not None and isinstance(w, torch.Tensor):
        w = w.detach().cpu().reshape(-1)
        if w.dtype != torch.float32:
            w = w.float()
        return np.ascontiguousarray(w.numpy())
    a = np.ascontiguousarray(np.asarray(w).reshape(-1))
    assert a.dtype == np.float32, a.dtype
    return a


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _levels(xhat) -> np.ndarray:
    a = np.ascontiguousarray(np.asarray(xhat, dtype=np.float32).reshape(-1))
    assert a.shape == (16,)
    return a.copy()


def _check(n: int, I: int, ragged: bool = False):
    """Whole blocks only, unless the function takes a shorter last block (ragged)."""
    if I <= 0 or (n % I and not ragged):
        raise ValueError("n must be a multiple of the block size")


def _blocks(n: int, I: int) -> int:
    return (n + I - 1) // I


# --------------------------------------------------------------------------- functions


def thresholds(xhat) -> np.ndarray:
    lv = _levels(xhat)
    xi = np.empty(15, np.float32)
    _load().orc_thresholds(_p(lv), _p(xi))
    return xi


def block_constants(w, I: int, norm: int) -> np.ndarray:
    a = as_f32(w)
    _check(a.size, I, ragged=True)
    m = np.empty(_blocks(a.size, I), np.float32)
    _load().orc_block_constants(_p(a), ctypes.c_int64(a.size), I, norm, _p(m))
    return m


def quantize(w, I: int, norm: int, xhat) -> Tuple[np.ndarray, np.ndarray]:
    """-> (codes uint8 [n/2], scales fp32 [n/I])."""
    a = as_f32(w)
    _check(a.size, I, ragged=True)
    lv = _levels(xhat)
    codes = np.empty((a.size + 1) // 2, np.uint8)
    scales = np.empty(_blocks(a.size, I), np.float32)
    _load().orc_quantize(_p(a), ctypes.c_int64(a.size), I, norm, _p(lv), _p(codes), _p(scales))
    return codes, scales


def dequantize(codes: np.ndarray, scales: np.ndarray, I: int, xhat, n: Optional[int] = None) -> np.ndarray:
    """-> fp32 products m * xhat(code), before any rounding to the output type.  `n` = number of
    weights when it is not twice the number of code bytes (an odd count)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.float32)
    n = codes.size * 2 if n is None else int(n)
    assert (n + 1) // 2 == codes.size
    _check(n, I, ragged=True)
    assert scales.size == _blocks(n, I)
    lv = _levels(xhat)
    out = np.empty(n, np.float32)
    _load().orc_dequantize(_p(codes), _p(scales), ctypes.c_int64(n), I, _p(lv), _p(out))
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.size, np.uint16)
    _load().orc_f32_to_bf16(_p(x), ctypes.c_int64(x.size), _p(out))
    return out.reshape(x.shape)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.uint16)
    out = np.empty(h.size, np.float32)
    _load().orc_bf16_to_f32(_p(h), ctypes.c_int64(h.size), _p(out))
    return out.reshape(h.shape)


def _segments(w):
    """A tensor or a list of tensors -> (concatenated fp32 data, int64 lengths).  Every tensor is
    cut into blocks from its own start; a length that is not a multiple of the block size ends
    in a shorter block."""
    ws = list(w) if isinstance(w, (list, tuple)) else [w]
    parts = [as_f32(t) for t in ws]
    seg = np.array([p.size for p in parts], np.int64)
    data = np.ascontiguousarray(np.concatenate(parts)) if len(parts) != 1 else parts[0]
    return data, seg


def em_accumulate_mse(w, I: int, norm: int, xhat, normdom: bool = False):
    """-> dict(s1[16] f64, s0[16] f64, count[16] u64, err_sum f64, n).  normdom: App. D variant.
    `w`: a tensor or a list of tensors (ragged lengths allowed)."""
    a, seg = _segments(w)
    _check(a.size, I, ragged=True)
    lv = _levels(xhat)
    s1 = np.zeros(16, np.float64)
    s0 = np.zeros(16, np.float64)
    cnt = np.zeros(16, np.uint64)
    err = ctypes.c_double(0.0)
    _load().orc_em_accumulate_mse_seg(_p(a), _p(seg), int(seg.size), I, norm, _p(lv), int(bool(normdom)), _p(s1),
                                      _p(s0), _p(cnt), ctypes.byref(err))
    return dict(s1=s1, s0=s0, count=cnt, err_sum=err.value, n=a.size)


def em_accumulate_mae(w, I: int, norm: int, xhat, normdom: bool = False):
    """-> dict(median[16] f32, wsum[16] f64, count[16] u64, err_sum f64, n).  normdom: App. D variant."""
    a, seg = _segments(w)
    _check(a.size, I, ragged=True)
    lv = _levels(xhat)
    med = np.zeros(16, np.float32)
    ws = np.zeros(16, np.float64)
    cnt = np.zeros(16, np.uint64)
    err = ctypes.c_double(0.0)
    _load().orc_em_accumulate_mae_seg(_p(a), _p(seg), int(seg.size), I, norm, _p(lv), int(bool(normdom)), _p(med),
                                      _p(ws), _p(cnt), ctypes.byref(err))
    return dict(median=med, wsum=ws, count=cnt, err_sum=err.value, n=a.size)


def fit(w, I: int, norm: int, metric: int, xhat, fixed_mask: int, iters: int):
    """-> (levels fp32[16], err_log f64[iters])."""
    a, seg = _segments(w)
    _check(a.size, I, ragged=True)
    lv = _levels(xhat)
    log = np.zeros(max(iters, 1), np.float64)
    _load().orc_fit_seg(_p(a), _p(seg), int(seg.size), I, norm, metric, _p(lv),
                        ctypes.c_uint32(fixed_mask), iters, _p(log))
    return lv, log[:iters]


def quant_error(w, I: int, norm: int, xhat) -> Tuple[float, float]:
    """-> (MSE, MAE) of the block-wise quantiser with levels xhat on w."""
    a = as_f32(w)
    _check(a.size, I)
    lv = _levels(xhat)
    mse, mae = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _load().orc_quant_error(_p(a), ctypes.c_int64(a.size), I, norm, _p(lv),
                            ctypes.byref(mse), ctypes.byref(mae))
    return mse.value, mae.value


def block_sigmas(w, I: int) -> np.ndarray:
    a = as_f32(w)
    _check(a.size, I, ragged=True)
    s = np.empty(_blocks(a.size, I), np.float32)
    _load().orc_block_sigmas(_p(a), ctypes.c_int64(a.size), I, _p(s))
    return s


def opq_split(w, I: int, tau: float, capacity: Optional[int] = None):
    """-> (w_clean fp32[n], idx int64[k], val bf16-bits uint16[k], n_out)."""
    a = as_f32(w)
    _check(a.size, I, ragged=True)
    cap = a.size if capacity is None else int(capacity)
    clean = np.empty(a.size, np.float32)
    idx = np.empty(max(cap, 1), np.int64)
    val = np.empty(max(cap, 1), np.uint16)
    k = _load().orc_opq_split(_p(a), ctypes.c_int64(a.size), I, ctypes.c_float(tau),
                              _p(clean), _p(idx), _p(val), ctypes.c_int64(cap))
    kk = min(k, cap)
    return clean, idx[:kk].copy(), val[:kk].copy(), int(k)


def opq_restore(out: np.ndarray, idx: np.ndarray, val: np.ndarray) -> np.ndarray:
    out = np.ascontiguousarray(out, dtype=np.float32)
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    val = np.ascontiguousarray(val, dtype=np.uint16)
    _load().orc_opq_restore(_p(out), _p(idx), _p(val), ctypes.c_int64(idx.size))
    return out


def opq_threshold(q: float, I: int) -> float:
    """tau = F_M^{-1}(q) for unit-variance Gaussian weights: F_M(m) = (2 G(m) - 1)^I
    (App. B.1, CDF of the absolute block maximum), hence G(tau) = (1 + q^(1/I)) / 2."""
    from scipy.special import ndtri
    return float(ndtri((1.0 + q ** (1.0 / I)) / 2.0))


def gemv(codes: np.ndarray, scales: np.ndarray, rows: int, cols: int, I: int, xhat, x,
         idx: Optional[np.ndarray] = None, val: Optional[np.ndarray] = None):
    """y = W x in fp64 for the decoded matrix (Eq. 3; with OPQ the stored outliers replace the
    decoded values, Sec. 3.3): W[r, c] = scale[block] * xhat[code] exactly (a product of two fp32
    numbers is exact in fp64), W.flat[idx] = val.  Also returns sum_c |W[r, c] x[c]|, the scale
    of the rounding error any fp32 evaluation of the same sum may show.
    -> (y fp64 [rows], mag fp64 [rows])."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    scales = np.ascontiguousarray(scales, dtype=np.float32).reshape(-1)
    n = rows * cols
    assert codes.size * 2 == n and cols % I == 0 and scales.size == n // I
    lv = _levels(xhat).astype(np.float64)
    c = np.empty(n, np.uint8)
    c[0::2] = codes >> 4
    c[1::2] = codes & 15
    W = lv[c] * np.repeat(scales.astype(np.float64), I)
    if idx is not None and len(idx):
        W[np.asarray(idx, dtype=np.int64)] = bf16_bits_to_f32(np.asarray(val, dtype=np.uint16)).astype(np.float64)
    W = W.reshape(rows, cols)
    xv = np.asarray(x, dtype=np.float64).reshape(-1)
    assert xv.size == cols
    return W @ xv, np.abs(W) @ np.abs(xv)


def gemm_bf16(codes: np.ndarray, scales: np.ndarray, rows: int, cols: int, I: int, xhat, X,
              idx: Optional[np.ndarray] = None, val: Optional[np.ndarray] = None):
    """Y = W X^T in fp64 for a batch of right-hand sides X [n_rhs, cols], the decoded weight being
    the dequantised value ROUNDED TO bf16 (Eq. 3 followed by round-to-nearest-even, i.e. what
    `dequantize` returns as bf16): the operand precision of the batched tensor-core consumer.  With
    OPQ the stored bf16 outlier values replace the decoded ones (W.flat[idx] = val).
    Also returns sum_c |W[r, c] X[b, c]|.  -> (Y fp64 [rows, n_rhs], mag fp64 [rows, n_rhs])."""
    w32 = dequantize(codes, scales, I, xhat, n=rows * cols)              # fp32 products of Eq. 3
    W = bf16_bits_to_f32(f32_to_bf16_bits(w32)).astype(np.float64)
    if idx is not None and len(idx):                                    # OPQ: the stored values (Sec. 3.3)
        W[np.asarray(idx, dtype=np.int64)] = bf16_bits_to_f32(np.asarray(val, dtype=np.uint16)).astype(np.float64)
    W = W.reshape(rows, cols)
    Xd = np.asarray(X, dtype=np.float64).reshape(-1, cols)
    return W @ Xd.T, np.abs(W) @ np.abs(Xd).T
