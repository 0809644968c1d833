"""The N > 1 path of bench.py is "replicas only": no data-path collective, only the timing is combined (the slowest
rank's time, whole-job throughput = world_size x units / that).  Two gloo ranks on the CPU exercise that combination."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [0.010 * (rank + 1), 0.5 - 0.1 * rank]          # rank 1 is slower on the first, rank 0 on the second
    dist.barrier()
    got = bench.slowest_rank(torch, dist, mine, "cpu")
    out[rank] = got
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_ranks_time():
    import bench
    assert bench.slowest_rank(torch, None, [0.25, 1.5], "cpu") == [0.25, 1.5]       # one rank: its own times
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29517, out), nprocs=world, join=True)
        assert out[0] == out[1] == [0.020, 0.5]
    units = 1000.0
    assert world * units / 0.020 == 100000.0                 # the whole-job value bench.py prints for N replicas
