"""Host-side logic of the multi-GPU benchmark path (independent replicas, slowest rank decides),
run as two gloo ranks on the CPU."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [100.0 + 10 * rank, 5.0 - rank, 7.0]                 # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine)
    dist.barrier()
    q.put((rank, got, bench.replica_throughput(256, world, got[0] / 1e3)))
    dist.destroy_process_group()


def test_max_over_ranks_and_replica_throughput_two_ranks():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in res:
        assert got == [110.0, 5.0, 7.0]                          # every rank sees the slowest time
        assert value == pytest.approx(2 * 256 / 0.110)           # two replicas' tokens over the slowest time


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.replica_throughput(100, 1, 0.5) == 200.0
