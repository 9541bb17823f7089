"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, max-over-ranks timing and the aggregate
throughput of independent replicas (the path has no exchange step, so there is no collective in
the data path to test)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r measured (r + 1) ms for the device-timed steps and (10 - r) ms end to end
    total_ms, e2e_ms = bench.reduce_max_over_ranks([rank + 1.0, 10.0 - rank], torch.device("cpu"), world)
    dist.barrier()
    q.put((rank, total_ms, e2e_ms, bench.aggregate_throughput(50_000_000, world, total_ms)))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_and_sum_the_replicas():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, _free_port() if r < 0 else PORT, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total_ms, e2e_ms, value in got:
        assert total_ms == 2.0 and e2e_ms == 10.0          # slowest rank decides, on every rank
        assert value == pytest.approx(2 * 50e6 / 2e-3 / 1e9)


PORT = _free_port()
