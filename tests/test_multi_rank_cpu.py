"""The N > 1 path of bench.py on CPU: two gloo ranks, independent replicas, timings reduced with a
max over ranks and the whole-job throughput computed from the slowest rank (weak scaling)."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank r "measures" different times; every rank must end up with the maximum of each
    mine = [10.0 + rank, 20.0 - rank, 5.0 * (rank + 1)]
    red = bench.reduce_over_ranks(mine, dist, torch.device("cpu"))
    value = bench.job_throughput_gbs(1_000_000, 100, world, red[0])
    dist.barrier()
    out[rank] = (red, value)
    dist.destroy_process_group()


def test_two_ranks_reduce_timings_with_max_and_sum_the_work():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        results = dict(out)
    assert set(results) == {0, 1}
    for rank in range(world):
        red, value = results[rank]
        assert red == [11.0, 20.0, 10.0]
        # 2 ranks x 100 steps x 1e6 bytes over 11 ms
        assert abs(value - 2 * 100 * 1_000_000 / 11e-3 / 1e9) < 1e-9


def test_single_process_path_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks([1.5, 2.5], None, torch.device("cpu")) == [1.5, 2.5]
    assert bench.job_throughput_gbs(4_000_000_000, 10, 1, 10_000.0) == 4.0
