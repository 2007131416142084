"""N > 1 runs independent replicas: only the timing is reduced (max over ranks) and the throughput
summed.  Checked here with two gloo ranks on CPU."""
import os
import socket
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 + 5.0 * rank                       # rank 1 is slower
    worst = bench.reduce_max(dist, mine, device="cpu")
    dist.barrier()
    out[rank] = (worst, bench.aggregate_value(world, 512 * 2**20, worst))
    dist.destroy_process_group()


def test_two_rank_aggregation():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1]
    worst, value = out[0]
    assert worst == 15.0
    assert abs(value - 2 * 512 * 2**20 / 15e-3 / 1e9) < 1e-9


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(None, 3.5) == 3.5
    assert abs(bench.aggregate_value(1, 10**9, 1.0) - 1000.0) < 1e-9
