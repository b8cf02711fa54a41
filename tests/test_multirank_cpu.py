"""The N > 1 path of the benchmark on the CPU: the step shards by request with no data-path
collective (replicas), so what ranks exchange is only timing.  Two gloo ranks check the max-over-ranks
reduction and the whole-job rate bench.py prints."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, world, rank)
    ms = [10.0, 40.0] if rank == 0 else [12.5, 30.0]      # rank 1 is slower on the first, rank 0 on the second
    red = bench.reduce_max_over_ranks(ms, world, "cpu")
    dist.barrier()
    if rank == 0:
        out.put((red, bench.whole_job_value(544, world, red[0])))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    red, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert red == [12.5, 40.0]
    assert abs(value - 2 * 544 / 12.5e-3) < 1e-6


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_over_ranks([3.0, 4.0], 1, "cpu") == [3.0, 4.0]
    assert bench.whole_job_value(100, 1, 10.0) == 100 / 10e-3
