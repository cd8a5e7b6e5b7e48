"""The multi-GPU form of the benchmark is N independent replicas (the path does not shard and has no
collective): each rank times its own steps, the job's time is the slowest rank's, and the value is
the units all ranks processed over that time.  Checked with two gloo processes on the CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 if rank == 0 else 25.0          # ms over 5 steps on this rank
    total = bench.max_over_ranks(mine, dist, "cpu")
    dist.barrier()
    out[rank] = (total, bench.replica_throughput(256, 5, world, total))
    dist.destroy_process_group()


def test_replicas_time_is_the_slowest_rank_and_value_is_the_aggregate():
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    for rank in (0, 1):
        total, value = out[rank]
        assert total == 25.0
        assert abs(value - 256 * 5 * 2 / 0.025) < 1e-6


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.replica_throughput(10, 4, 1, 2.0) == 10 * 4 / 0.002
