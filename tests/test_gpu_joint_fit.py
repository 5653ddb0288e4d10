"""Joint fit over shards (bof4_em_step per shard, records gathered, bof4_m_step): the ranks of a
multi-GPU run are emulated here as consecutive calls on one GPU.  The result must be the oracle's
fit over the list of shards, and the single-call fit over the same list."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu

LV0 = np.array(workloads.init_levels_7_0_8(), np.float32)


@pytest.fixture(scope="module")
def bof4():
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_06653_b200 as m
    assert torch.cuda.is_available()
    return m


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("norm,mask", [(0, workloads.FIXED_BOF4), (1, workloads.FIXED_BOF4S)])
@pytest.mark.parametrize("metric", [0, 2])
def test_joint_fit_over_three_shards(bof4, dtype, norm, mask, metric):
    from paper_2505_06653_b200 import binding as b
    I, iters = 64, 6
    shards = [workloads.gaussian_student_mixture(n, 0.02 * (k + 1), 0.02, 3, 70 + k, dtype)
              for k, n in enumerate([1 << 20, (1 << 19) + 64 * 3 + 5, 3 * (1 << 18)])]
    dev = [s.cuda() for s in shards]
    cb = torch.tensor(LV0, device="cuda")
    log = torch.zeros(iters, dtype=torch.float64, device="cuda")
    for t in range(iters):
        recs = torch.cat([b.em_step_record([d], I, norm, metric, cb) for d in dev])   # "all-gather" in rank order
        b.bof4_m_step(recs, metric, cb, mask, log[t:t + 1])
    rcb, rlog = oracle.fit(shards, I, norm, metric, LV0, mask, iters)
    np.testing.assert_allclose(cb.cpu().numpy(), rcb, rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(log.cpu().numpy(), rlog, rtol=1e-5)
    one, one_log = bof4.bof4_fit_codebook(dev, I, norm, metric, LV0, mask, iters)
    np.testing.assert_allclose(cb.cpu().numpy(), one.cpu().numpy(), rtol=1e-6, atol=1e-8)
    # without a process group the joint driver is the same loop over the local shard list
    j, jlog = bof4.bof4_fit_codebook_joint(dev, I, norm, metric, LV0, mask, iters)
    np.testing.assert_allclose(j.cpu().numpy(), rcb, rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(jlog.cpu().numpy(), rlog, rtol=1e-5)


def test_m_step_refuses_medians(bof4):
    from paper_2505_06653_b200 import binding as b
    w = workloads.gaussian(1 << 16, 0.02, 3, torch.bfloat16).cuda()
    cb = torch.tensor(LV0, device="cuda")
    rec = b.em_step_record([w], 64, 1, bof4.METRIC_MAE, cb)
    with pytest.raises(bof4.Bof4Error):
        b.bof4_m_step(rec, bof4.METRIC_MAE, cb, workloads.FIXED_BOF4S)
