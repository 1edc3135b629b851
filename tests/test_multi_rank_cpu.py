"""The only multi-rank logic of the benchmark (replicas, no data-path exchange): the slowest rank's time
decides, the value is the work of all ranks over that time.  Two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 5.0 - rank, 7.0]                      # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine, world, "cpu")
    rate = bench.whole_job_rate(per_gpu_units=16 * 256, world=world, ms=got[0])
    dist.barrier()
    if rank == 0:
        out.put((got, rate))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    world, port = 2, 29517
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got, rate = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [11.0, 5.0, 7.0]
    assert abs(rate - 2 * 16 * 256 / 11e-3) < 1e-6


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2], 1, "cpu") == [1.5, 2.0]
    assert bench.whole_job_rate(100, 1, 50.0) == 2000.0
