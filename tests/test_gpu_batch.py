"""bof4_quantize_batch / bof4_dequantize_batch: many tensors in few launches, their rows dealt over
one grid.  Every tensor's codes, constants and dequantised values must be the oracle's, bit for
bit, whatever its place in the list (the CTA that starts a tensor rotates with the rows before it)."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

LV = np.array(workloads.BOF4S_MSE_I64, np.float32)


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _tensors(sizes, dtype, seed):
    out = []
    for k, n in enumerate(sizes):
        w = workloads.gaussian_student_mixture(max(n, 1), 0.02, 0.02, 3, seed + k, dtype)[:n].clone()
        if n > 70:
            w[64:128] = 0.0                        # an all-zero block
        out.append(w.contiguous())
    return out


SIZE_SETS = [
    [16384 * 3, 16384, 64, 16384 * 2 + 64 * 5, 0, 16384 * 300 + 4096, 128],             # whole rows, partial rows, empty
    [16384 * 7 + 37, 31, 64 * 3 + 1, 16384 * 296 + 16384 * 5, 100],                      # ragged tails
    [4096 * (k + 1) for k in range(70)],                                                 # more than one launch's table
]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("norm", [0, 1])
@pytest.mark.parametrize("I", [64, 32, 256, 2048])
def test_batch_equals_the_oracle_per_tensor(bof4, dtype, norm, I):
    for s, sizes in enumerate(SIZE_SETS):
        if dtype == torch.float32 and s == 0 and I != 64:
            continue                                # fp32 goes through the single-tensor path: one set is enough
        ws = _tensors(sizes, dtype, 800 + 10 * s)
        live = [w for w in ws if w.numel() > 0]
        codes, scales = bof4.bof4_quantize_batch([w.cuda() for w in live], I, norm, LV)
        for w, c, sc in zip(live, codes, scales):
            rc, rs = oracle.quantize(w, I, norm, LV)
            assert np.array_equal(c.cpu().numpy(), rc), (sizes, w.numel())
            assert np.array_equal(sc.float().cpu().numpy().view(np.uint32), rs.view(np.uint32)), (sizes, w.numel())
        for out_dtype in (bof4.BF16, bof4.F32):
            outs = bof4.bof4_dequantize_batch(codes, scales, [w.numel() for w in live], I, LV, out_dtype)
            for w, c, sc, o in zip(live, codes, scales, outs):
                ref = oracle.dequantize(c.cpu().numpy(), sc.float().cpu().numpy(), I, LV, n=w.numel())
                if out_dtype == bof4.BF16:
                    assert np.array_equal(_bits(o), oracle.f32_to_bf16_bits(ref)), (sizes, w.numel())
                else:
                    assert np.array_equal(o.cpu().numpy().view(np.uint32), ref.view(np.uint32)), (sizes, w.numel())


def test_batch_matches_single_calls_on_model_shapes(bof4):
    """One layer of the 8B-shaped set (seven matrices, 2.2e8 weights): identical to the single calls."""
    mats = [m.cuda() for _, m in workloads.config4_matrices(layers=1)]
    codes, scales = bof4.bof4_quantize_batch(mats, 64, 1, LV)
    outs = bof4.bof4_dequantize_batch(codes, scales, [m.numel() for m in mats], 64, LV, bof4.BF16)
    for m, c, sc, o in zip(mats, codes, scales, outs):
        c1, s1 = bof4.bof4_quantize(m, 64, 1, LV)
        assert torch.equal(c, c1) and torch.equal(sc.view(torch.int16), s1.view(torch.int16))
        o1 = bof4.bof4_dequantize(c1, s1, 64, LV, bof4.BF16)
        assert torch.equal(o.view(torch.int16), o1.view(torch.int16))
    # and the first matrix against the oracle on sampled blocks
    w = mats[0].cpu().reshape(-1)
    rc, rs = oracle.quantize(w[:1 << 22], 64, 1, LV)
    assert np.array_equal(codes[0][:1 << 21].cpu().numpy(), rc)


def test_batch_argument_errors(bof4):
    w = torch.zeros(128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bof4.Bof4Error):
        bof4.bof4_quantize_batch([w], 48, 0, LV)
    with pytest.raises(ValueError):
        bof4.bof4_quantize_batch([w], 64, 0, LV, out=([torch.zeros(3, dtype=torch.uint8, device="cuda")],
                                                      [torch.zeros(2, dtype=torch.bfloat16, device="cuda")]))
