"""Host-side logic of the multi-GPU bench path, run as two gloo ranks on the CPU: the path does not
shard (independent replicas, no data-path collective), so all the ranks share is the timing:
the slowest rank's time, and a whole-job throughput of world x one replica's work."""
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
    got = bench.max_over_ranks([1.0 + rank, 10.0 - rank, 5.0])
    out[rank] = (got, bench.replica_throughput(100.0, got[0], world))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_replica_throughput_two_gloo_ranks():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        got, thr = res[rank]
        assert got == [2.0, 10.0, 5.0]                     # element-wise max, the same on every rank
        assert thr == 2 * 100.0 / (2.0 * 1e-3)             # two replicas, paced by the slower one


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert bench.replica_throughput(10.0, 2.0, 1) == 5000.0
