"""The multi-GPU leg of bench.py shards by giving every rank its own problem and reduces only
timings.  That host logic is exercised here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.rank_env() == (rank, rank, world)
        seed = bench.workload_seed_offset(rank)
        # rank 1 is the slower one in both timings
        total_ms, e2e_ms = bench.max_over_ranks([10.0 + 5.0 * rank, 100.0 - 30.0 * rank], dist, "cpu")
        dist.barrier()
        ref = None
        if rank != 0:
            class A:  # the reference arm does no work off rank 0
                steps, warmup, gpus = 1, 0, world
            ref = bench.run_reference(A)
        out.put((rank, seed, total_ms, e2e_ms, ref))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_without_a_collective_on_the_data():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    (r0, s0, t0, e0, _), (r1, s1, t1, e1, ref1) = res
    assert (r0, r1) == (0, 1) and s0 != s1          # independent problems
    assert t0 == t1 == 15.0 and e0 == e1 == 100.0   # max over ranks, seen by every rank
    assert ref1 is None


def test_whole_job_value_and_single_process_reduction():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None, "cpu") == [1.5, 2.5]
    # 2 ranks x 2^26 weights in 1 ms = 134.2 Gweights/s
    assert abs(bench.whole_job_gweights_per_s(2, 1 << 26, 1.0) - 134.217728) < 1e-9
