"""bof4_gemm_tc: the batched decode-side consumer on the tensor cores (tcgen05.mma, accumulator in
tensor memory) against oracle.gemm_bf16.  Integer-valued cases must be exact whatever the
hardware's summation order (every partial sum is representable), which pins the operand layout
(swizzle, descriptors, nibble order, scale lookup) bit for bit; generic cases must stay within
2^-14 of sum |w x|."""
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


def _exact_case(rows, cols, n_rhs, I, seed):
    """Codes at random, power-of-two constants of both signs, levels multiples of 1/16, X small
    integers: all products are multiples of 2^-8 below 4 in magnitude, so sums of up to 2^14 of them need
    at most 24 bits and are exact in fp32 in whatever order they are taken."""
    rng = np.random.default_rng(seed)
    lv = ((np.arange(16) - 7.5) / 8.0).astype(np.float32)
    c = rng.integers(0, 16, rows * cols).astype(np.uint8)
    codes = ((c[0::2] << 4) | c[1::2]).astype(np.uint8)
    scales = (2.0 ** rng.integers(-4, 2, rows * cols // I) * rng.choice([-1.0, 1.0], rows * cols // I)).astype(np.float32)
    X = rng.integers(-2, 3, (n_rhs, cols)).astype(np.float32)
    return lv, codes, scales, X


@pytest.mark.parametrize("rows,cols,n_rhs,I", [(128, 64, 16, 64), (128, 128, 16, 32), (128, 192, 32, 64),
                                               (256, 1024, 64, 128), (384, 4096, 48, 64), (128, 8192, 64, 4096)])
@pytest.mark.parametrize("scale_dtype", [torch.bfloat16, torch.float32])
def test_integer_valued_products_are_exact(bof4, rows, cols, n_rhs, I, scale_dtype):
    lv, codes, scales, X = _exact_case(rows, cols, n_rhs, I, rows + cols + n_rhs)
    y, status = bof4.bof4_gemm_tc(torch.from_numpy(codes).cuda(), torch.from_numpy(scales).to(scale_dtype).cuda(),
                                  rows, cols, I, lv, torch.from_numpy(X).to(torch.bfloat16).cuda())
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref, _ = oracle.gemm_bf16(codes, scales, rows, cols, I, lv, X)
    assert np.array_equal(y.cpu().numpy().astype(np.float64), ref)
    # without the K split (one CTA per 128 rows) the same, bit for bit
    y1, status1 = bof4.bof4_gemm_tc(torch.from_numpy(codes).cuda(), torch.from_numpy(scales).to(scale_dtype).cuda(),
                                    rows, cols, I, lv, torch.from_numpy(X).to(torch.bfloat16).cuda(), split=False)
    assert int(status1.item()) == 0 and torch.equal(y, y1)


def test_random_shapes_are_exact(bof4):
    """Seeded random shapes (row tiles, k-blocks that do and do not divide by the split factors,
    every batch size and block size the entry point takes), integer-valued: bit for bit."""
    rng = np.random.default_rng(2026)
    for trial in range(24):
        rows = 128 * int(rng.integers(1, 9))
        I = int(rng.choice([32, 64, 128, 256, 1024]))
        cols = max(I, 64) * int(rng.integers(1, 1 + 16384 // max(I, 64)))   # <= 2^14: partial sums stay exact
        n_rhs = int(rng.choice([16, 32, 48, 64]))
        lv, codes, scales, X = _exact_case(rows, cols, n_rhs, I, 1000 + trial)
        sd = torch.bfloat16 if trial % 2 else torch.float32
        y, status = bof4.bof4_gemm_tc(torch.from_numpy(codes).cuda(), torch.from_numpy(scales).to(sd).cuda(),
                                      rows, cols, I, lv, torch.from_numpy(X).to(torch.bfloat16).cuda(),
                                      split=bool(trial % 3))
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref, _ = oracle.gemm_bf16(codes, scales, rows, cols, I, lv, X)
        assert np.array_equal(y.cpu().numpy().astype(np.float64), ref), (rows, cols, n_rhs, I)


@pytest.mark.parametrize("rows,cols,n_rhs", [(256, 4096, 16), (512, 8192, 64), (128, 14336, 32)])
@pytest.mark.parametrize("norm", [0, 1])
def test_quantised_matrix_times_batch(bof4, rows, cols, n_rhs, norm):
    I = 64
    lv = np.array(workloads.BOF4S_MSE_I64, np.float32)
    w = workloads.gaussian_student_mixture(rows * cols, 0.02, 0.02, 3, 5 + n_rhs, torch.bfloat16)
    codes, scales = bof4.bof4_quantize(w.cuda(), I, norm, lv)
    x = workloads.gaussian(n_rhs * cols, 1.0, 6, torch.bfloat16).reshape(n_rhs, cols)
    y, status = bof4.bof4_gemm_tc(codes, scales, rows, cols, I, lv, x.cuda())
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref, mag = oracle.gemm_bf16(codes.cpu().numpy(), scales.float().cpu().numpy(), rows, cols, I, lv, x.float().numpy())
    err = np.abs(y.cpu().numpy().astype(np.float64) - ref)
    assert np.all(err <= 2.0 ** -14 * mag + 1e-30), float((err / mag).max())
    # the operand is what bof4_dequantize writes: the same product through torch on that tensor agrees as well
    wd = bof4.bof4_dequantize(codes, scales, I, lv, bof4.BF16).view(rows, cols)
    yt = (wd.double() @ x.cuda().double().T).cpu().numpy()
    assert np.all(np.abs(yt - ref) <= 1e-12 * mag)


@pytest.mark.parametrize("rows,cols,n_rhs", [(256, 4096, 16), (384, 8192, 64)])
def test_with_outlier_list(bof4, rows, cols, n_rhs):
    """OPQ quantisation, then the batched product with the outlier list: the stored values replace
    the decoded weights (Sec. 3.3).  Also a list that is cut off by its capacity."""
    I = 64
    lv = np.array(workloads.BOF4S_MSE_I64, np.float32)
    w = workloads.inject_outliers(workloads.gaussian(rows * cols, 0.02, 9, torch.bfloat16), 0.02, 3e-4, 10.0, 40.0, 10)
    tau = float(np.float32(bof4.bof4_opq_threshold(0.95, I)))
    cap = rows * cols // 64
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(w.cuda(), I, 1, lv, tau, cap)
    k = bof4.bof4_outlier_count(cnt, cap)
    assert k > rows
    x = workloads.gaussian(n_rhs * cols, 1.0, 11, torch.bfloat16).reshape(n_rhs, cols)
    idx_h = idx[:k].cpu().numpy().astype(np.int64)
    val_h = val[:k].view(torch.int16).cpu().numpy().view(np.uint16)
    for use in (k, k // 2):
        y, status = bof4.bof4_gemm_tc(codes, scales, rows, cols, I, lv, x.cuda(), outliers=(idx[:use], val[:use], cnt))
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref, mag = oracle.gemm_bf16(codes.cpu().numpy(), scales.float().cpu().numpy(), rows, cols, I, lv,
                                    x.float().numpy(), idx_h[:use], val_h[:use])
        err = np.abs(y.cpu().numpy().astype(np.float64) - ref)
        assert np.all(err <= 2.0 ** -14 * mag + 1e-30), float((err / mag).max())
    plain, _ = bof4.bof4_gemm_tc(codes, scales, rows, cols, I, lv, x.cuda())
    assert not torch.equal(plain, y)


def test_gemm_tc_argument_errors(bof4):
    lv = np.array(workloads.BOF4S_MSE_I64, np.float32)
    codes = torch.zeros(128 * 64 // 2, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(128, dtype=torch.bfloat16, device="cuda")
    for rows, cols, n in ((100, 64, 16), (128, 96, 16), (128, 64, 8), (128, 64, 24), (128, 64, 80)):
        x = torch.zeros(n, cols, dtype=torch.bfloat16, device="cuda")
        c = torch.zeros(rows * cols // 2, dtype=torch.uint8, device="cuda")
        with pytest.raises(bof4.Bof4Error):
            bof4.bof4_gemm_tc(c, scales, rows, cols, 32 if cols % 64 else 64, lv, x)
