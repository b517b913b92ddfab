"""N > 1 path of the benchmark on CPU: two gloo ranks act as independent replicas; the aggregate is
the sum of units over ranks divided by the slowest rank's time (weak scaling, no data-path exchange)."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    assert bench.dist_env() == (rank, rank, world)
    ms_local = 2.0 + rank          # rank 1 is the slow one
    units_local = 256.0
    dist.barrier()
    ms, units = bench.aggregate_over_ranks(ms_local, units_local)
    out[rank] = (ms, units)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_as_independent_replicas():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        ms, units = out[rank]
        assert ms == 3.0 and units == 512.0   # max time, summed units: value = 512 / 3 ms on every rank


def test_single_process_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(1.5, 7.0) == (1.5, 7.0)
