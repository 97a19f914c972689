"""The multi-GPU form of the benchmark is N independent replicas (the path has no exchange between
GPUs): what the ranks share is a barrier and the maximum of their step times.  Two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 70.0 + 5.0 * rank                                   # this replica's time for the block of steps
    slowest = bench.max_over_ranks(mine)
    dist.barrier()
    out[rank] = (slowest, bench.replica_throughput(318_000_000, world, slowest / 1000.0))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_sum_of_the_work():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        port = 29500 + os.getpid() % 2000
        procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        assert out[0] == out[1]
        slowest, gbs = out[0]
        assert slowest == 75.0
        assert abs(gbs - 2 * 318_000_000 / 75e-6 / 1e9) < 1e-6


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.replica_throughput(10**9, 1, 1.0) == 1000.0
