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


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` without WORLD_SIZE re-executes itself under torch.distributed.run; with
    the CPU stand-in for the timed body the printed line must come from two ranks: n_gpus 2, the slower
    rank's time, both ranks' bytes."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--standin", "--steps", "5"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                      # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["steps"] == 5
    assert abs(line["ms_per_step"] - 15.0 / 5) < 1e-9          # max over ranks (10 ms and 15 ms)
    assert abs(line["value"] - 2 * (512 << 20) / (3.0e-3) / 1e9) < 1e-2
