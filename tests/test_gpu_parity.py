"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Codes, packed bytes, scales, outlier lists and dequantised values must agree
bit for bit; EM statistics, fitted levels and the error log within 1e-5 relative."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

RTOL = 1e-5  # tolerance of the fitted codebook and the per-iteration error

LV_BOF4S = np.array([-0.8568463921546936, -0.6692874431610107, -0.5235266089439392,
                     -0.4004882574081421, -0.2910638153553009, -0.1900092959403992,
                     -0.0938529595732689, 0.0, 0.0887671709060669, 0.1794802695512772,
                     0.2743096053600311, 0.3760197460651398, 0.4886530041694641,
                     0.6188603639602661, 0.7791395783424377, 1.0], np.float32)  # Tab. 6, BOF4-S (MSE)
LV_INIT = np.array(workloads.init_levels_7_0_8(), np.float32)


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def bits16(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def scales_f32(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy()


def make_weights(n, dtype, seed, kind="mix"):
    if kind == "mix":
        w = workloads.gaussian_student_mixture(n, 0.02, 0.01, 4, seed, dtype)
    else:
        w = workloads.gaussian(n, 0.02, seed, dtype)
    return w


def special_blocks(w: torch.Tensor, I: int) -> torch.Tensor:
    """Plants the degenerate cases: an all-zero block, a block of negative zeros, a tie of
    +max / -max (the lower index must win), a constant block, exact threshold hits."""
    w = w.clone()
    B = w.numel() // I
    if B >= 6:
        w[0:I] = 0.0
        w[I:2 * I] = -0.0
        blk = w[2 * I:3 * I]
        m = blk.abs().max() * 2
        blk[5] = -m
        blk[I - 3] = m
        w[3 * I:4 * I] = 0.0123
        blk = w[4 * I:5 * I]
        blk[:] = 0.0
        blk[0] = 1.0
        # values that land exactly on thresholds of LV_BOF4S (m = 1): midpoints in fp32
        xi = oracle.thresholds(LV_BOF4S)
        k = min(15, I - 1)
        blk[1:1 + k] = torch.from_numpy(xi[:k].copy()).to(w.dtype)
    return w


# --------------------------------------------------------------------------- quantise / dequantise


@pytest.mark.parametrize("I", [32, 64, 128, 256])
@pytest.mark.parametrize("norm", [0, 1])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_quantize_dequantize_bit_exact(bof4, I, norm, dtype):
    # several CTA rows, both unrolled iterations, and a ragged tail (not a multiple of 2048)
    n = 256 * 37 * 8 + 3 * I
    w = special_blocks(make_weights(n, dtype, 11 + I + norm), I)
    wd = w.cuda()
    codes, scales = bof4.bof4_quantize(wd, I, norm, LV_BOF4S)
    rc, rs = oracle.quantize(w, I, norm, LV_BOF4S)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(scales_f32(scales).view(np.uint32), rs.view(np.uint32))  # incl. sign of zero
    for out_dt, out_code in ((torch.bfloat16, bof4.BF16), (torch.float32, bof4.F32)):
        out = bof4.bof4_dequantize(codes, scales, I, LV_BOF4S, out_code)
        ref = oracle.dequantize(rc, rs, I, LV_BOF4S)
        if out_dt == torch.bfloat16:
            assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(ref))
        else:
            assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))


def test_quantize_bf16_weights_with_fp32_scales(bof4):
    I, n = 64, 64 * 1000
    w = make_weights(n, torch.bfloat16, 5)
    codes, scales = bof4.bof4_quantize(w.cuda(), I, 1, LV_BOF4S, scale_dtype=bof4.F32)
    rc, rs = oracle.quantize(w, I, 1, LV_BOF4S)
    assert scales.dtype == torch.float32
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(scales.cpu().numpy(), rs)


@pytest.mark.parametrize("n_blocks", [0, 1, 2, 31, 33])
def test_quantize_tiny_and_empty(bof4, n_blocks):
    I = 32
    w = make_weights(max(n_blocks * I, 1), torch.bfloat16, 3)[: n_blocks * I]
    codes, scales = bof4.bof4_quantize(w.cuda(), I, 1, LV_BOF4S)
    out = bof4.bof4_dequantize(codes, scales, I, LV_BOF4S, bof4.BF16)
    torch.cuda.synchronize()
    if n_blocks == 0:
        assert codes.numel() == 0 and out.numel() == 0
        return
    rc, rs = oracle.quantize(w, I, 1, LV_BOF4S)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(scales_f32(scales), rs)
    assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(oracle.dequantize(rc, rs, I, LV_BOF4S)))


def test_block_maximum_survives_the_round_trip(bof4):
    """The element of largest magnitude is reconstructed exactly (levels +-1 / 1 fixed)."""
    I, n = 64, 64 * 4096
    w = make_weights(n, torch.bfloat16, 21)
    wd = w.cuda()
    for norm, lv in ((1, LV_BOF4S), (0, np.concatenate(([-1.0], LV_BOF4S[1:])).astype(np.float32))):
        codes, scales = bof4.bof4_quantize(wd, I, norm, lv)
        out = bof4.bof4_dequantize(codes, scales, I, lv, bof4.BF16).cpu().float().view(-1, I)
        wb = w.float().view(-1, I)
        j = wb.abs().argmax(dim=1, keepdim=True)
        assert torch.equal(out.gather(1, j), wb.gather(1, j))


# --------------------------------------------------------------------------- OPQ


def _opq_reference(w, I, norm, lv, tau):
    clean, ridx, rval, rk = oracle.opq_split(w, I, tau)
    rc, rs = oracle.quantize(clean, I, norm, lv)
    rout = oracle.opq_restore(oracle.dequantize(rc, rs, I, lv), ridx, rval)
    return clean, ridx, rval, rk, rc, rs, rout


@pytest.mark.parametrize("I", [32, 64, 128, 256])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_opq_quantize_dequantize_bit_exact(bof4, I, dtype):
    n = 256 * 8 * 9 + 5 * 256
    n -= n % I
    w = make_weights(n, dtype, 100 + I, kind="gauss")
    w = workloads.inject_outliers(w, 0.02, 2e-3, 10.0, 40.0, 7)
    w = special_blocks(w, I)          # the constant block has sigma = 0: all of it is outliers
    # a dense burst: more than 8 outliers inside one 256-element tile (staging overflow path)
    w[256 * 20: 256 * 20 + 40] = torch.tensor([(-1.0) ** k * (3.0 + k) for k in range(40)]).to(dtype)
    tau = float(np.float32(bof4.bof4_opq_threshold(0.95, I)))
    wd = w.cuda()
    clean, ridx, rval, rk, rc, rs, rout = _opq_reference(w, I, 1, LV_BOF4S, tau)
    assert rk > 60
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(wd, I, 1, LV_BOF4S, tau, n)
    out = bof4.bof4_dequantize(codes, scales, I, LV_BOF4S, bof4.BF16, (idx, val, cnt))
    k = int(cnt.item())
    assert k == rk
    assert np.array_equal(idx[:k].cpu().numpy().astype(np.int64), ridx)
    assert np.array_equal(bits16(val[:k]), rval)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(scales_f32(scales), rs)
    assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(rout))
    # the split alone: cleaned copy and the same list
    c2, idx2, val2, cnt2 = bof4.opq_split(wd, I, tau, n)
    assert int(cnt2.item()) == rk
    assert np.array_equal(idx2[:k].cpu().numpy().astype(np.int64), ridx)
    assert np.array_equal(bits16(val2[:k]), rval)
    assert np.array_equal(c2.float().cpu().numpy().view(np.uint32), clean.view(np.uint32))


def test_opq_capacity_overflow_reports_true_count(bof4):
    I, n = 64, 64 * 2048
    w = workloads.inject_outliers(make_weights(n, torch.bfloat16, 9, "gauss"), 0.02, 5e-3, 10, 40, 3)
    tau = float(np.float32(bof4.bof4_opq_threshold(0.95, I)))
    _, ridx, rval, rk = oracle.opq_split(w, I, tau)
    cap = rk // 2
    guard = 16
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(w.cuda(), I, 1, LV_BOF4S, tau, cap + guard)
    # hand the library a shorter capacity than the buffers: the tail must stay untouched
    idx.fill_(-7)
    val.fill_(0)
    out = (codes, scales, idx, val, cnt)
    import ctypes
    from paper_2505_06653_b200 import binding as b
    wsp = torch.empty(b.bof4_workspace_bytes(b.OP_OPQ, n, I), dtype=torch.uint8, device="cuda")
    wd = w.cuda()
    cb = torch.tensor(LV_BOF4S, device="cuda")
    rc = b.lib().bof4_quantize_opq(wd.data_ptr(), b.BF16, n, I, 1, cb.data_ptr(), tau, codes.data_ptr(),
                                   scales.data_ptr(), b.BF16, idx.data_ptr(), val.data_ptr(), cap,
                                   cnt.data_ptr(), wsp.data_ptr(), wsp.numel(), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert int(cnt.item()) == rk
    assert np.array_equal(idx[:cap].cpu().numpy().astype(np.int64), ridx[:cap])
    assert np.all(idx[cap:].cpu().numpy() == -7)
    # the two-call pattern: the synchronising count check turns the overflow into an error that
    # names the capacity that would have sufficed; with that capacity the same check passes
    host = ctypes.c_int64(-1)
    rc = b.lib().bof4_outlier_count(cnt.data_ptr(), cap, ctypes.byref(host), None)
    assert rc == -5 and host.value == rk
    assert str(rk).encode() in b.lib().bof4_last_error()
    with pytest.raises(b.Bof4Error) as ei:
        b.bof4_outlier_count(cnt, cap)
    assert ei.value.code == -5
    assert b.bof4_outlier_count(cnt, rk) == rk
    # capacity 0: only the count
    cnt.zero_()
    rc = b.lib().bof4_quantize_opq(wd.data_ptr(), b.BF16, n, I, 1, cb.data_ptr(), tau, codes.data_ptr(),
                                   scales.data_ptr(), b.BF16, None, None, 0, cnt.data_ptr(),
                                   wsp.data_ptr(), wsp.numel(), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert int(cnt.item()) == rk


def test_opq_no_outliers_and_empty(bof4):
    I = 64
    w = torch.zeros(64 * 40, dtype=torch.bfloat16)
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(w.cuda(), I, 1, LV_BOF4S, 3.35, 16)
    assert int(cnt.item()) == 0
    e = torch.zeros(0, dtype=torch.bfloat16, device="cuda")
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(e, I, 1, LV_BOF4S, 3.35, 16)
    assert int(cnt.item()) == 0


# --------------------------------------------------------------------------- EM, MSE


def _check_stats(got, ref):
    assert got["n"] == ref["n"]
    assert np.array_equal(got["count"], ref["count"])          # integer work: exact
    np.testing.assert_allclose(got["s1"], ref["s1"], rtol=RTOL, atol=1e-12 * np.abs(ref["s1"]).max())
    np.testing.assert_allclose(got["s0"], ref["s0"], rtol=RTOL)
    np.testing.assert_allclose(got["err_sum"], ref["err_sum"], rtol=RTOL)


@pytest.mark.parametrize("I", [32, 64, 128, 256])
@pytest.mark.parametrize("norm", [0, 1])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_em_step_mse_matches_oracle(bof4, I, norm, dtype):
    n = 2048 * 21 + 5 * 256
    n -= n % I
    w = special_blocks(make_weights(n, dtype, 40 + I), I)
    got = bof4.bof4_em_step([w.cuda()], I, norm, bof4.METRIC_MSE, LV_INIT)
    ref = oracle.em_accumulate_mse(w, I, norm, LV_INIT)
    _check_stats(got, ref)


def test_em_step_mse_many_tensors_equals_concatenation(bof4):
    """More tensors than one launch's table holds, of ragged sizes, incl. an empty one."""
    I = 64
    sizes = [64 * (1 + (7 * k) % 50) for k in range(70)] + [0, 2048 * 3]
    ws = [make_weights(max(s, 1), torch.bfloat16, 500 + k)[:s] for k, s in enumerate(sizes)]
    got = bof4.bof4_em_step([w.cuda() for w in ws], I, 1, bof4.METRIC_MSE, LV_BOF4S)
    ref = oracle.em_accumulate_mse(torch.cat(ws), I, 1, LV_BOF4S)
    _check_stats(got, ref)


def test_em_step_is_bit_reproducible(bof4):
    I, n = 64, 1 << 20
    wd = make_weights(n, torch.bfloat16, 77).cuda()
    a = bof4.bof4_em_step([wd], I, 1, bof4.METRIC_MSE, LV_INIT)
    b = bof4.bof4_em_step([wd], I, 1, bof4.METRIC_MSE, LV_INIT)
    for k in ("s1", "s0", "count"):
        assert np.array_equal(a[k], b[k])
    assert a["err_sum"] == b["err_sum"]


@pytest.mark.parametrize("norm,mask,dtype", [(0, workloads.FIXED_BOF4, torch.float32),
                                             (1, workloads.FIXED_BOF4S, torch.bfloat16)])
def test_fit_mse_matches_oracle(bof4, norm, mask, dtype):
    I, n, iters = 64, 1 << 18, 12
    w = make_weights(n, dtype, 60 + norm)
    cb, log = bof4.bof4_fit_codebook([w.cuda()], I, norm, bof4.METRIC_MSE, LV_INIT, mask, iters)
    rcb, rlog = oracle.fit(w, I, norm, oracle.METRIC_MSE, LV_INIT, mask, iters)
    cb = cb.cpu().numpy()
    np.testing.assert_allclose(cb, rcb, rtol=RTOL, atol=1e-7)
    np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=RTOL)
    for l in range(16):
        if (mask >> l) & 1:
            assert cb[l] == LV_INIT[l]          # fixed levels: exact
    assert np.all(np.diff(log.cpu().numpy()) <= 1e-12 * rlog[0])


def test_fit_zero_iterations_and_empty_input(bof4):
    I = 64
    w = make_weights(64 * 8, torch.bfloat16, 1).cuda()
    cb, log = bof4.bof4_fit_codebook([w], I, 1, bof4.METRIC_MSE, LV_INIT, 0, 0)
    assert np.array_equal(cb.cpu().numpy(), LV_INIT) and log.numel() == 0
    e = torch.zeros(0, dtype=torch.bfloat16, device="cuda")
    cb, log = bof4.bof4_fit_codebook([e], I, 1, bof4.METRIC_MSE, LV_INIT, 0, 2)
    assert np.array_equal(cb.cpu().numpy(), LV_INIT)
    assert np.all(log.cpu().numpy() == 0)


# --------------------------------------------------------------------------- EM, MAE


def _check_mae_stats(got, ref, levels_in):
    assert got["n"] == ref["n"]
    assert np.array_equal(got["count"], ref["count"])
    np.testing.assert_allclose(got["s0"], ref["wsum"], rtol=RTOL)
    np.testing.assert_allclose(got["err_sum"], ref["err_sum"], rtol=RTOL)
    # the median is a sample of the data: it must be the same sample, not merely a close one
    assert np.array_equal(got["median"], ref["median"])


@pytest.mark.parametrize("I", [32, 64, 128, 256])
@pytest.mark.parametrize("norm", [0, 1])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_em_step_mae_matches_oracle(bof4, I, norm, dtype):
    n = 8192 * 5 + 7 * 512
    n -= n % I
    w = special_blocks(make_weights(n, dtype, 140 + I), I)
    got = bof4.bof4_em_step([w.cuda()], I, norm, bof4.METRIC_MAE, LV_INIT)
    ref = oracle.em_accumulate_mae(w, I, norm, LV_INIT)
    _check_mae_stats(got, ref, LV_INIT)


def test_em_step_mae_exact_half_ties(bof4):
    """Equal block constants: cumulative weights hit exactly half of the total for every region
    with an even member count; the lower of the two middle samples must be returned."""
    I, nb = 64, 512
    g = torch.Generator().manual_seed(5)
    w = (torch.rand(nb, I, generator=g) * 2 - 1) * 0.999
    w[:, 0] = 1.0                                  # every block has m = 1
    w = w.reshape(-1).to(torch.bfloat16)
    got = bof4.bof4_em_step([w.cuda()], I, 0, bof4.METRIC_MAE, LV_INIT)
    ref = oracle.em_accumulate_mae(w, I, 0, LV_INIT)
    assert (ref["count"] % 2 == 0).any()
    _check_mae_stats(got, ref, LV_INIT)


def test_em_step_mae_many_tensors(bof4):
    I = 64
    sizes = [64 * (1 + (5 * k) % 40) for k in range(70)] + [0, 8192 * 2]
    ws = [make_weights(max(s, 1), torch.bfloat16, 900 + k)[:s] for k, s in enumerate(sizes)]
    got = bof4.bof4_em_step([w.cuda() for w in ws], I, 1, bof4.METRIC_MAE, LV_BOF4S)
    ref = oracle.em_accumulate_mae(torch.cat(ws), I, 1, LV_BOF4S)
    _check_mae_stats(got, ref, LV_BOF4S)


@pytest.mark.parametrize("norm,mask,dtype", [(0, workloads.FIXED_BOF4, torch.float32),
                                             (1, workloads.FIXED_BOF4S, torch.bfloat16)])
def test_fit_mae_matches_oracle(bof4, norm, mask, dtype):
    I, n, iters = 64, 1 << 17, 8
    w = make_weights(n, dtype, 160 + norm)
    cb, log = bof4.bof4_fit_codebook([w.cuda()], I, norm, bof4.METRIC_MAE, LV_INIT, mask, iters)
    rcb, rlog = oracle.fit(w, I, norm, oracle.METRIC_MAE, LV_INIT, mask, iters)
    cb = cb.cpu().numpy()
    np.testing.assert_allclose(cb, rcb, rtol=RTOL, atol=1e-7)
    np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=RTOL)
    for l in range(16):
        if (mask >> l) & 1:
            assert cb[l] == LV_INIT[l]


def test_fit_mae_is_bit_reproducible(bof4):
    I, n = 64, 1 << 20
    wd = make_weights(n, torch.bfloat16, 78).cuda()
    a, la = bof4.bof4_fit_codebook([wd], I, 1, bof4.METRIC_MAE, LV_INIT, workloads.FIXED_BOF4S, 3)
    b, lb = bof4.bof4_fit_codebook([wd], I, 1, bof4.METRIC_MAE, LV_INIT, workloads.FIXED_BOF4S, 3)
    assert torch.equal(a, b) and torch.equal(la, lb)


def test_non_finite_weights_do_not_disturb_other_blocks(bof4):
    """NaN / infinite weights are outside the contract, but they must neither fault nor change
    the result of any block that holds only finite numbers (rows with a non-finite block take
    the comparison-only search instead of the table)."""
    I, n = 64, 8192 * 3
    w = make_weights(n, torch.bfloat16, 33)
    bad_blocks = [3, 40, 41, 200]
    w[3 * I + 5] = float("nan")
    w[40 * I] = float("inf")
    w[41 * I + 63] = float("-inf")
    w[200 * I + 1] = float("nan")
    w[200 * I + 2] = float("inf")
    wd = w.cuda()
    codes, scales = bof4.bof4_quantize(wd, I, 1, LV_BOF4S)
    out = bof4.bof4_dequantize(codes, scales, I, LV_BOF4S, bof4.BF16)
    st = bof4.bof4_em_step([wd], I, 1, bof4.METRIC_MSE, LV_BOF4S)
    torch.cuda.synchronize()
    clean = w.clone()
    for b in bad_blocks:
        clean[b * I:(b + 1) * I] = 0.0
    rc, rs = oracle.quantize(clean, I, 1, LV_BOF4S)
    keep = np.ones(n // I, bool)
    keep[bad_blocks] = False
    assert np.array_equal(codes.cpu().numpy().reshape(-1, I // 2)[keep], rc.reshape(-1, I // 2)[keep])
    assert np.array_equal(scales_f32(scales)[keep], rs[keep])
    assert st["n"] == n


def test_fit_into_caller_buffers(bof4):
    """`out=` makes the binding write levels and error log into the caller's tensors."""
    I, n = 64, 1 << 16
    w = make_weights(n, torch.bfloat16, 88).cuda()
    lv, log = bof4.bof4_fit_codebook([w], I, 1, bof4.METRIC_MSE, LV_INIT, workloads.FIXED_BOF4S, 3)
    cb = torch.empty(16, dtype=torch.float32, device="cuda")
    lg = torch.full((5,), -1.0, dtype=torch.float64, device="cuda")
    lv2, log2 = bof4.bof4_fit_codebook([w], I, 1, bof4.METRIC_MSE, LV_INIT, workloads.FIXED_BOF4S, 3, out=(cb, lg))
    assert lv2.data_ptr() == cb.data_ptr() and log2.numel() == 3
    assert torch.equal(lv, cb) and torch.equal(log, lg[:3]) and float(lg[3]) == -1.0
    with pytest.raises(ValueError):
        bof4.bof4_fit_codebook([w], I, 1, bof4.METRIC_MSE, LV_INIT, 0, 3, out=(cb, lg[:2]))


def test_mae_candidate_list_overflow_takes_the_later_data_passes(bof4):
    """Two million normalised weights within one first-digit bin of a free level (four distinct
    values around 0.5): the candidate list of that level overflows, so the third and fourth data
    passes, which carry their own selection and the level update, have to finish the median."""
    I, nb = 32, 1 << 16
    g = torch.Generator().manual_seed(77)
    k = torch.randint(0, 4, (nb, I), generator=g).float()
    x = 0.5 + k * 2.0 ** -13
    x[:, 0] = 1.0                                            # the block maximum
    x[:, 1] = -(0.25 + torch.randint(0, 64, (nb,), generator=g).float() * 2.0 ** -9)  # some spread elsewhere
    scale = 2.0 ** (torch.arange(nb) % 5 - 2).float()        # block constants 1/4 ... 4: unequal weights
    w = (x * scale[:, None]).reshape(-1).contiguous()        # exact in fp32
    ref = oracle.em_accumulate_mae(w, I, 1, LV_INIT)
    assert ref["count"][11] > 65536 * 16                     # level 0.5 holds the 2 M samples
    got = bof4.bof4_em_step([w.cuda()], I, 1, bof4.METRIC_MAE, LV_INIT)
    _check_mae_stats(got, ref, LV_INIT)
    # the same through the fit entry point: one iteration moves level 11 to that median
    lv, log = bof4.bof4_fit_codebook([w.cuda()], I, 1, bof4.METRIC_MAE, LV_INIT, 0, 1)
    assert lv.cpu().numpy()[11] == ref["median"][11]


def test_mae_with_the_smallest_workspace_collects_candidates_one_pass_later(bof4):
    """The candidate lists of the median selection live in the workspace and grow with the size
    asked for; with the smallest workspace the library accepts, a region's candidates do not fit
    after the first pass of 2^26 weights, one more data pass runs before they are collected, and
    the medians must still be the oracle's, bit for bit (the other tests use the default size)."""
    from paper_2505_06653_b200 import binding as b
    I, n = 64, (1 << 26) + (1 << 16)
    w = workloads.gaussian_student_mixture(n, 0.02, 0.01, 4, 302, torch.bfloat16)
    ref = oracle.em_accumulate_mae(w, I, 1, LV_INIT)
    small = b.bof4_workspace_bytes(b.OP_EM, 0, I, b.METRIC_MAE)
    assert small < b.bof4_workspace_bytes(b.OP_EM, n, I, b.METRIC_MAE)
    wd = w.cuda()
    for nbytes in (small, None):
        ws = None if nbytes is None else torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        got = bof4.bof4_em_step([wd], I, 1, bof4.METRIC_MAE, LV_INIT, workspace=ws)
        _check_mae_stats(got, ref, LV_INIT)


# --------------------------------------------------------------------------- blocks wider than a warp


WIDE = [512, 1024, 2048, 4096]


def wide_special(w, I):
    """Plants, at warp-crossing positions of wide blocks: a tie of +max / -max whose first
    occurrence sits in a later warp than ... the other sign (lower index must win), an all-zero
    block and a constant block."""
    w = w.clone()
    B = w.numel() // I
    assert B >= 5
    w[0:I] = 0.0
    blk = w[I:2 * I]
    m = blk.abs().max() * 2
    blk[I - 7] = m          # last warp of the block
    blk[I // 2 + 3] = -m    # an earlier warp: the negative one comes first
    blk = w[2 * I:3 * I]
    m = blk.abs().max() * 2
    blk[5] = m              # first warp
    blk[I - 1] = -m
    w[3 * I:4 * I] = 0.0123
    return w


@pytest.mark.parametrize("I", WIDE)
@pytest.mark.parametrize("norm", [0, 1])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_wide_blocks_quantize_dequantize_bit_exact(bof4, I, norm, dtype):
    n = 8192 * 5 + 4096 * 3     # several CTA rows and a partial one
    w = wide_special(make_weights(n, dtype, 400 + I + norm), I)
    codes, scales = bof4.bof4_quantize(w.cuda(), I, norm, LV_BOF4S)
    out = bof4.bof4_dequantize(codes, scales, I, LV_BOF4S, bof4.BF16)
    rc, rs = oracle.quantize(w, I, norm, LV_BOF4S)
    assert np.array_equal(scales_f32(scales).view(np.uint32), rs.view(np.uint32))
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(oracle.dequantize(rc, rs, I, LV_BOF4S)))


@pytest.mark.parametrize("I", WIDE)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_wide_blocks_opq_bit_exact(bof4, I, dtype):
    n = 8192 * 6 + 4096
    w = workloads.inject_outliers(make_weights(n, dtype, 500 + I, "gauss"), 0.02, 2e-3, 10.0, 40.0, 17)
    w = wide_special(w, I)
    w[8192 * 2 + 100: 8192 * 2 + 140] = torch.tensor([(-1.0) ** k * (3.0 + k) for k in range(40)]).to(dtype)
    tau = float(np.float32(bof4.bof4_opq_threshold(0.95, I)))
    clean, ridx, rval, rk, rc, rs, rout = _opq_reference(w, I, 1, LV_BOF4S, tau)
    codes, scales, idx, val, cnt = bof4.bof4_quantize_opq(w.cuda(), I, 1, LV_BOF4S, tau, n)
    out = bof4.bof4_dequantize(codes, scales, I, LV_BOF4S, bof4.BF16, (idx, val, cnt))
    k = int(cnt.item())
    assert k == rk and rk > 40
    assert np.array_equal(idx[:k].cpu().numpy().astype(np.int64), ridx)
    assert np.array_equal(bits16(val[:k]), rval)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(scales_f32(scales), rs)
    assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(rout))
    c2, idx2, val2, cnt2 = bof4.opq_split(w.cuda(), I, tau, n)
    assert int(cnt2.item()) == rk
    assert np.array_equal(c2.float().cpu().numpy().view(np.uint32), clean.view(np.uint32))


@pytest.mark.parametrize("I", WIDE)
@pytest.mark.parametrize("norm", [0, 1])
def test_wide_blocks_em_steps_match_oracle(bof4, I, norm):
    n = 16384 * 3 + 8192
    w = wide_special(make_weights(n, torch.bfloat16, 600 + I), I)
    wd = w.cuda()
    _check_stats(bof4.bof4_em_step([wd], I, norm, bof4.METRIC_MSE, LV_INIT),
                 oracle.em_accumulate_mse(w, I, norm, LV_INIT))
    _check_mae_stats(bof4.bof4_em_step([wd], I, norm, bof4.METRIC_MAE, LV_INIT),
                     oracle.em_accumulate_mae(w, I, norm, LV_INIT), LV_INIT)
    mask = workloads.FIXED_BOF4S if norm else workloads.FIXED_BOF4
    cb, log = bof4.bof4_fit_codebook([wd], I, norm, bof4.METRIC_MSE, LV_INIT, mask, 4)
    rcb, rlog = oracle.fit(w, I, norm, oracle.METRIC_MSE, LV_INIT, mask, 4)
    np.testing.assert_allclose(cb.cpu().numpy(), rcb, rtol=RTOL, atol=1e-7)
    np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=RTOL)


# --------------------------------------------------------------------------- App. D variants


@pytest.mark.parametrize("I", [64, 256, 2048])
@pytest.mark.parametrize("norm", [0, 1])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_normalised_domain_steps_match_oracle(bof4, I, norm, dtype):
    """Textbook Lloyd on the normalised weights (unit sample weights, errors on x)."""
    n = 16384 * 2 + 4096
    # blocks of very different scale, so that the weighting matters
    g = torch.Generator().manual_seed(700 + I)
    scale = torch.rand(n // I, 1, generator=g) * 3 + 0.01
    w = (torch.randn(n // I, I, generator=g) * scale).reshape(-1).to(dtype)
    wd = w.cuda()
    got = bof4.bof4_em_step([wd], I, norm, bof4.METRIC_MSE_NORMALIZED, LV_INIT)
    ref = oracle.em_accumulate_mse(w, I, norm, LV_INIT, normdom=True)
    _check_stats(got, ref)
    assert np.array_equal(got["s0"], ref["count"].astype(np.float64))   # unit weights: exact
    got = bof4.bof4_em_step([wd], I, norm, bof4.METRIC_MAE_NORMALIZED, LV_INIT)
    ref = oracle.em_accumulate_mae(w, I, norm, LV_INIT, normdom=True)
    _check_mae_stats(got, ref, LV_INIT)
    mask = workloads.FIXED_BOF4S if norm else workloads.FIXED_BOF4
    for metric in (bof4.METRIC_MSE_NORMALIZED, bof4.METRIC_MAE_NORMALIZED):
        cb, log = bof4.bof4_fit_codebook([wd], I, norm, metric, LV_INIT, mask, 3)
        rcb, rlog = oracle.fit(w, I, norm, metric, LV_INIT, mask, 3)
        np.testing.assert_allclose(cb.cpu().numpy(), rcb, rtol=RTOL, atol=1e-7)
        np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=RTOL)


def test_calls_follow_the_callers_stream(bof4):
    """Everything is enqueued on the stream handed in (here: torch's current stream, a side
    stream), in order, without touching the default stream's work."""
    I, n = 64, 8192 * 4
    w = make_weights(n, torch.bfloat16, 55)
    side = torch.cuda.Stream()
    wd = w.cuda()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        cb, log = bof4.bof4_fit_codebook([wd], I, 1, bof4.METRIC_MSE, LV_INIT, workloads.FIXED_BOF4S, 3,
                                         sync=False)
        codes, scales = bof4.bof4_quantize(wd, I, 1, cb)          # consumes the fitted levels in order
        out = bof4.bof4_dequantize(codes, scales, I, cb, bof4.BF16)
    side.synchronize()
    rcb, _ = oracle.fit(w, I, 1, oracle.METRIC_MSE, LV_INIT, workloads.FIXED_BOF4S, 3)
    cbh = cb.cpu().numpy()
    np.testing.assert_allclose(cbh, rcb, rtol=RTOL, atol=1e-7)
    rc, rs = oracle.quantize(w, I, 1, cbh)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert np.array_equal(bits16(out), oracle.f32_to_bf16_bits(oracle.dequantize(rc, rs, I, cbh)))
