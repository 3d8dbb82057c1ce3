"""The N > 1 path on CPU: two gloo ranks aggregate their replica timings the way bench.py does."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2401_14021_b200 import replicas
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.world() == (rank, world)
        replicas.barrier()
        # rank r answered 8 * (r + 1) queries; its device-resident region took 10 + r ms, its
        # end-to-end region 20 - r ms
        times, total = replicas.aggregate([10.0 + rank, 20.0 - rank], 8 * (rank + 1))
        qps = replicas.throughput([10.0 + rank, 20.0 - rank], 8 * (rank + 1))
        out.put((rank, times, total, qps))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_max_time_sum_queries():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, times, total, qps in results:
        assert times == [11.0, 20.0]              # slowest rank of each region
        assert total == 8 + 16
        assert abs(qps[0] - 24 / 11e-3) < 1e-6 and abs(qps[1] - 24 / 20e-3) < 1e-6


def test_single_process_passes_through():
    sys.path.insert(0, ROOT)
    from paper_2401_14021_b200 import replicas
    assert replicas.world() == (0, 1)
    assert replicas.aggregate([3.0], 5) == ([3.0], 5)
    assert replicas.throughput([2.0], 4) == [2000.0]
