"""Host-side logic of bench.py's N > 1 path (independent replicas, one per GPU): the step time of
the job is the maximum over ranks and the value is the aggregate.  Run here as two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                 # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, world, dist, "cpu")
    out.put((rank, ms, bench.aggregate_value(ms, world)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_aggregate_rate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in res:
        assert ms == 15.0                          # max over ranks
        assert abs(value - 2 * 1e3 / 15.0) < 1e-9   # two replicas, each one step per 15 ms


def test_single_rank_is_a_pass_through():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1, None, "cpu") == 7.5
    assert bench.aggregate_value(20.0, 1) == 50.0
