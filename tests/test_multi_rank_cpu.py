"""The N>1 path of the benchmark is 'independent replicas, time = max over ranks'.  Its host
logic is exercised here with two gloo ranks on CPU (no GPU, no data-path collective)."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 2.0 if rank == 0 else 5.0           # rank 1 is the slow one
    value, ms = bench.aggregate_throughput(1.0e6, local_ms, world)
    out[rank] = (value, ms, bench.max_over_ranks(float(rank)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregate_uses_the_slowest_rank():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        value, ms, mx = res[rank]
        assert ms == 5.0                            # max over ranks, same on every rank
        assert abs(value - 2 * 1.0e6 / 5.0e-3) < 1e-3
        assert mx == 1.0


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25) == 3.25
    v, ms = bench.aggregate_throughput(10.0, 2.0, 1)
    assert ms == 2.0 and v == 10.0 / 2e-3
