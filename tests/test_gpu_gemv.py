"""y = W_q x with the 4-bit matrix decoded on the fly (Eq. 3 fused into the matrix-vector product,
outliers of Sec. 3.3 as a sparse correction) against the oracle's fp64 definition.

Tolerance: the kernel sums in fp32.  A lane adds 16 packed products per accumulator half, joins
the halves, scales, then a 5-step butterfly and at most 32 stripes follow, and the correction
kernel adds a few terms more: fewer than 64 roundings, each at most 2^-24 of the sum of the
absolute terms, which the oracle returns beside y."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

TOL = 64 * 2.0 ** -24


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def _levels(signed):
    lv = np.sort(np.concatenate([-np.linspace(1, 0, 8, endpoint=False) ** 1.3, [0.0], np.linspace(0, 1, 8)[1:] ** 1.2]))
    if signed:
        lv = np.sort(np.concatenate([-0.86 * np.linspace(1, 0, 7, endpoint=False), [0.0], np.linspace(0, 1, 9)[1:]]))
    assert lv.size == 16
    return lv.astype(np.float32)


def _matrix(rows, cols, dtype, seed, outlier_rate=2e-3):
    w = workloads.gaussian(rows * cols, 0.02, seed=seed, dtype=torch.float32)
    w = workloads.inject_outliers(w, 0.02, outlier_rate, 6.0, 20.0, seed=seed + 1)
    return w.to(dtype)


def _oracle_in_row_chunks(codes, scales, rows, cols, I, lv, x, o_idx, o_val):
    """Rows are independent, so the fp64 oracle runs on a few million weights at a time."""
    step = max(1, (1 << 23) // cols)
    ys, mags = [], []
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        ii = vv = None
        if o_idx is not None:
            sel = (o_idx.astype(np.int64) // cols >= r0) & (o_idx.astype(np.int64) // cols < r1)
            ii, vv = o_idx[sel].astype(np.int64) - r0 * cols, o_val[sel]
        y, m = oracle.gemv(codes[r0 * cols // 2:r1 * cols // 2], scales[r0 * cols // I:r1 * cols // I], r1 - r0,
                           cols, I, lv, x, ii, vv)
        ys.append(y)
        mags.append(m)
    return np.concatenate(ys), np.concatenate(mags)


def _check(bof4, rows, cols, I, w_dtype, x_dtype, signed, opq, seed, capacity=None):
    dev = "cuda:0"
    lv = _levels(signed)
    norm = bof4.NORM_SIGNED if signed else bof4.NORM_ABS
    w = _matrix(rows, cols, w_dtype, seed)
    x = workloads.gaussian(cols, 1.0, seed=seed + 7, dtype=torch.float32).to(x_dtype)
    wd, xd = w.to(dev), x.to(dev)
    if opq:
        tau = bof4.bof4_opq_threshold(0.95, I)
        cap = capacity if capacity is not None else max(rows * cols // 16, 64)
        codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(wd, I, norm, lv, tau, cap)
        outl = (idx, val, cnt)
        k = min(int(cnt.item()), cap)
        assert k > 0 or rows * cols < (1 << 16)
        o_idx = idx[:k].cpu().numpy()
        o_val = val[:k].view(torch.int16).cpu().numpy().view(np.uint16)
    else:
        codes, scales = bof4.bof4_quantize(wd, I, norm, lv)
        outl, o_idx, o_val = None, None, None
    y = bof4.bof4_gemv(codes, scales, rows, cols, I, lv, xd, outl)
    y2 = bof4.bof4_gemv(codes, scales, rows, cols, I, lv, xd, outl)
    torch.cuda.synchronize()
    assert y.dtype == torch.float32 and y.shape == (rows,)
    assert torch.equal(y, y2), "the summation order is fixed: two calls must agree bit for bit"
    ref, mag = _oracle_in_row_chunks(codes.cpu().numpy(), scales.float().cpu().numpy(), rows, cols, I, lv,
                                     x.float().numpy(), o_idx, o_val)
    err = np.abs(y.cpu().numpy().astype(np.float64) - ref)
    assert np.all(err <= TOL * mag + 1e-300), (err / np.maximum(mag, 1e-300)).max()
    return err, mag


SHAPES = [(3, 32, 32), (64, 1024, 64), (37, 4096, 64), (100, 2144, 32), (16, 11008, 64), (21, 8192, 128),
          (9, 28672, 64), (6, 32768, 4096), (13, 17408, 1024)]


@pytest.mark.parametrize("rows,cols,I", SHAPES)
@pytest.mark.parametrize("opq", [False, True])
def test_gemv_matches_the_oracle(bof4, rows, cols, I, opq):
    _check(bof4, rows, cols, I, torch.bfloat16, torch.bfloat16, False, opq, seed=1000 + rows)


@pytest.mark.parametrize("w_dtype,x_dtype", [(torch.float32, torch.float32), (torch.float32, torch.bfloat16),
                                             (torch.bfloat16, torch.float32)])
@pytest.mark.parametrize("signed", [False, True])
def test_gemv_dtypes_and_normalisations(bof4, w_dtype, x_dtype, signed):
    _check(bof4, 50, 3072, 64, w_dtype, x_dtype, signed, True, seed=77)


def test_gemv_uses_only_the_outliers_that_fit(bof4):
    """capacity below the number found: the first `capacity` entries are applied, as in decoding."""
    _check(bof4, 40, 2048, 64, torch.bfloat16, torch.bfloat16, False, True, seed=5, capacity=96)


def test_gemv_many_rows_several_batches_per_cta(bof4):
    """More row batches than resident CTAs, so a CTA loops and both partial-sum buffers are reused."""
    _check(bof4, 148 * 8 * 8 * 2 + 5, 4096, 64, torch.bfloat16, torch.bfloat16, False, True, seed=9)


def test_gemv_full_size_sampled_rows(bof4):
    """8192 x 8192 (the square projection of the 70B shapes, App. E.1) in the timed launch
    configuration; the oracle computes 48 sampled rows."""
    dev = "cuda:0"
    rows = cols = 8192
    I = 64
    lv = _levels(False)
    w = _matrix(rows, cols, torch.bfloat16, seed=31).to(dev)
    x = workloads.gaussian(cols, 1.0, seed=33, dtype=torch.float32).to(torch.bfloat16)
    tau = bof4.bof4_opq_threshold(0.95, I)
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(w, I, bof4.NORM_ABS, lv, tau, rows * cols // 64)
    k = int(cnt.item())
    assert 0 < k <= idx.numel()
    y = bof4.bof4_gemv(codes, scales, rows, cols, I, lv, x.to(dev), (idx, val, cnt)).cpu().numpy()
    idx_h = idx[:k].cpu().numpy().astype(np.int64)
    val_h = val[:k].view(torch.int16).cpu().numpy().view(np.uint16)
    codes_h = codes.cpu().numpy().reshape(rows, cols // 2)
    scales_h = scales.float().cpu().numpy().reshape(rows, cols // I)
    rng = np.random.default_rng(2)
    for r in np.concatenate([[0, rows - 1], rng.integers(0, rows, 46)]):
        sel = (idx_h // cols) == r
        ref, mag = oracle.gemv(codes_h[r], scales_h[r], 1, cols, I, lv, x.float().numpy(),
                               idx_h[sel] - r * cols, val_h[sel])
        assert abs(float(y[r]) - ref[0]) <= TOL * mag[0]


def test_gemv_degenerate_shapes_and_errors(bof4):
    dev = "cuda:0"
    lv = _levels(False)
    x = torch.ones(64, dtype=torch.bfloat16, device=dev)
    empty_c = torch.empty(0, dtype=torch.uint8, device=dev)
    empty_s = torch.empty(0, dtype=torch.bfloat16, device=dev)
    assert bof4.bof4_gemv(empty_c, empty_s, 0, 64, 32, lv, x).numel() == 0
    y = bof4.bof4_gemv(empty_c, empty_s, 5, 0, 32, lv, x[:0], out=torch.full((5,), 3.0, device=dev))
    assert torch.equal(y.cpu(), torch.zeros(5))
    codes = torch.zeros(64 * 48 // 2, dtype=torch.uint8, device=dev)
    scales = torch.ones(64 * 48 // 32, dtype=torch.bfloat16, device=dev)
    with pytest.raises(bof4.Bof4Error) as e:  # 48 columns are not a multiple of the block size
        bof4.bof4_gemv(codes, scales, 64, 48, 32, lv, x[:48])
    assert e.value.code == -2
    big = torch.zeros(32800 // 2, dtype=torch.uint8, device=dev)
    with pytest.raises(bof4.Bof4Error) as e:  # wider than the 32 stripes of one CTA
        bof4.bof4_gemv(big, torch.ones(32800 // 32, dtype=torch.bfloat16, device=dev), 1, 32800, 32, lv,
                       torch.ones(32800, dtype=torch.bfloat16, device=dev))
    assert e.value.code == -2
    xx = torch.ones(72, dtype=torch.bfloat16, device=dev)
    with pytest.raises(bof4.Bof4Error) as e:  # x must be 16-byte aligned (vector loads)
        bof4.bof4_gemv(torch.zeros(4 * 64 // 2, dtype=torch.uint8, device=dev),
                       torch.ones(4 * 64 // 32, dtype=torch.bfloat16, device=dev), 4, 64, 32, lv, xx[3:67])
    assert e.value.code == -1
    # all-zero blocks: scale 0, y = 0 exactly
    z = torch.zeros(4 * 64, dtype=torch.bfloat16, device=dev)
    c, s = bof4.bof4_quantize(z, 32, bof4.NORM_ABS, lv)
    assert torch.equal(bof4.bof4_gemv(c, s, 4, 64, 32, lv, x).cpu(), torch.zeros(4))
