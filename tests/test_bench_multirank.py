"""The multi-GPU leg of bench.py is "replicas only": ranks exchange nothing but a barrier and
the maximum of their times.  That host logic is checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    secs = 0.5 + 0.25 * rank                     # rank 1 is the slow one
    dist.barrier()
    secs_max, value = bench.whole_job(secs, 1000, world, dist, "cpu")
    out.put((rank, secs_max, value))
    dist.barrier()
    dist.destroy_process_group()


def test_whole_job_is_all_units_over_the_slowest_rank():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, secs_max, value in got:
        assert secs_max == 0.75                          # the max over ranks, on every rank
        assert value == 2 * 1000 / 0.75                  # whole-job units over that time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.whole_job(0.5, 100, 1) == (0.5, 200.0)
