"""The benchmark's multi-rank bookkeeping on CPU (gloo, two ranks): replicas only, so the ranks exchange
nothing but their timings; the slowest rank sets the step time and the job's rate counts every rank's work."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 50.0 - 5 * rank]                  # rank 1 is slower on the first, faster on the second
    red = bench.max_over_ranks(mine)
    dist.barrier()
    out.put((rank, red, bench.whole_job_rate(world, 1000, 4, red[0])))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, red, rate in got:
        assert red == [11.0, 50.0]
        assert abs(rate - 2 * 1000 * 4 / 11e-3) < 1e-6


def test_single_process_is_the_identity():
    import bench
    assert bench.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert bench.whole_job_rate(1, 10, 2, 1000.0) == 20.0
