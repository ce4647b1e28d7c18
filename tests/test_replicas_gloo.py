"""The N > 1 path of the benchmark is N independent replicas with no data-path
collective; the only cross-rank step is the max-over-ranks of the timed
seconds (whole-job throughput = all ranks' tokens / the slowest rank's time).
Two gloo ranks on the CPU run that step and the throughput arithmetic."""
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
    mine = [0.010 * (rank + 1), 0.5 - 0.1 * rank]          # rank 1 is slower on the first, rank 0 on the second
    got = bench.max_over_ranks(mine, "cpu", world)
    dist.barrier()
    if rank == 0:
        out.put(got)
    dist.destroy_process_group()


def test_max_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert abs(got[0] - 0.020) < 1e-12 and abs(got[1] - 0.5) < 1e-12
    # whole-job throughput of two replicas of 32 tokens x 10 steps over the slowest rank's time
    assert abs(2 * 32 * 10 / got[0] - 32000.0) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu", 1) == [1.5, 2.5]
