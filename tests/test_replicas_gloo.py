"""The multi-GPU mode of the benchmark is N independent replicas (sequences are independent,
the path has no exchange step): the only cross-rank logic is "time of the slowest rank" and
"sum of the sequences".  Checked here with two gloo ranks on CPU."""
import os
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, results):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + rank, 3.0 - rank]          # rank 1 is slower on the first, faster on the second
        got = bench.max_over_ranks(mine)
        value = bench.aggregate_throughput(world, 32, 5, got[0] * 1e-3)
        results.put((rank, got, value))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_work():
    ctx = mp.get_context("spawn")
    results = ctx.Queue()
    port = 29000 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, results)) for r in range(2)]
    for p in procs:
        p.start()
    out = [results.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in out:
        assert got == [11.0, 3.0]
        assert abs(value - 2 * 32 * 5 / 11.0e-3) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.aggregate_throughput(1, 32, 10, 0.5) == 640.0
