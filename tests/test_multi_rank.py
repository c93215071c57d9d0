"""The N > 1 path of bench.py on CPU: two gloo ranks.  The path does not shard (replicas only), so what
the ranks share is the timing protocol: barrier, maximum over ranks, whole-job throughput."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # each rank "measures" a different time: the job is as slow as the slowest replica
    local = [0.010 * (rank + 1), 0.5 - 0.1 * rank]
    dist.barrier()
    merged = bench.max_over_ranks(local)
    value = bench.whole_job_value(100, world, merged[0])
    seeds = [None] * world
    dist.all_gather_object(seeds, bench.replica_seed(7, rank))
    out.put((rank, merged, value, seeds))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_the_job_value():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, merged, value, seeds in results:
        assert merged == [0.020, 0.5]                      # max over ranks, element-wise
        assert abs(value - 2 * 100 / 0.020) < 1e-6         # both replicas' steps over the slowest time
        assert seeds == [7, 1007]                          # independent replicas: distinct seeded inputs


def test_single_process_is_the_identity():
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_value(10, 1, 2.0) == 5.0
