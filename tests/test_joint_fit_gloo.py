"""The exchange of a joint fit over several GPUs: every rank contributes one bof4_em_stats record
per iteration, gathered in rank order.  Two gloo ranks on CPU exercise that plumbing
(`binding.gather_records`) with records made by the oracle on each rank's shard: the gathered
records, summed in rank order, must be the oracle's statistics of the union of the shards
(Sec. 3.2, Eq. 6: sums over shards add)."""
import ctypes
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
I = 64


def _shard(rank):
    sys.path.insert(0, ROOT)
    import workloads
    return workloads.gaussian((3 + rank) * 4096 + 17 * rank, 0.02 * (1 + rank), 40 + rank, torch.bfloat16)


def _record(st):
    from paper_2505_06653_b200 import binding
    rec = binding.EmStats()
    for l in range(16):
        rec.s1[l], rec.s0[l], rec.count[l] = float(st["s1"][l]), float(st["s0"][l]), int(st["count"][l])
    rec.err_sum, rec.n_total = float(st["err_sum"]), int(st["n"])
    return torch.frombuffer(bytearray(bytes(rec)), dtype=torch.uint8).clone()


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import oracle
    import workloads
    from paper_2505_06653_b200 import binding
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lv = np.array(workloads.BOF4S_MSE_I64, np.float32)
        st = oracle.em_accumulate_mse(_shard(rank), I, 1, lv)
        got = binding.gather_records(_record(st))
        out.put((rank, got.numpy().tobytes()))
    finally:
        dist.destroy_process_group()


def test_records_are_gathered_in_rank_order_and_add_up_to_the_union():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    sys.path.insert(0, ROOT)
    import oracle
    import workloads
    from paper_2505_06653_b200 import binding
    assert res[0] == res[1]                                   # every rank holds the same records
    size = ctypes.sizeof(binding.EmStats)
    recs = [binding.EmStats.from_buffer_copy(res[0][k * size:(k + 1) * size]) for k in range(2)]
    shards = [_shard(0), _shard(1)]
    assert [r.n_total for r in recs] == [s.numel() for s in shards]    # rank order
    lv = np.array(workloads.BOF4S_MSE_I64, np.float32)
    union = oracle.em_accumulate_mse(shards, I, 1, lv)        # a list: blocks never span two shards
    s1 = np.array(recs[0].s1) + np.array(recs[1].s1)
    s0 = np.array(recs[0].s0) + np.array(recs[1].s0)
    np.testing.assert_allclose(s1, union["s1"], rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(s0, union["s0"], rtol=1e-12)
    assert np.array_equal(np.array(recs[0].count) + np.array(recs[1].count), union["count"].astype(np.int64))
    assert abs(recs[0].err_sum + recs[1].err_sum - union["err_sum"]) <= 1e-12 * union["err_sum"]


def test_without_a_process_group_the_record_stands_alone():
    sys.path.insert(0, ROOT)
    from paper_2505_06653_b200 import binding
    t = torch.arange(ctypes.sizeof(binding.EmStats), dtype=torch.uint8)
    assert binding.gather_records(t) is t
