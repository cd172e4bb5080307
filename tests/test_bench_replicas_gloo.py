"""The multi-GPU mode of bench.py is "replicas only": ranks share nothing but a barrier and the
max-over-ranks of their timings.  That host logic is exercised here with two gloo ranks on CPU."""
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
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 2.0 + rank            # rank 1 is the slow replica
    dist.barrier()
    slow = bench.max_over_ranks(mine, world, device="cpu")
    value = bench.aggregate_throughput(world, 32, 10, 1.0, slow)
    out.put((rank, slow, value))
    dist.destroy_process_group()


def test_two_replicas_report_max_time_and_whole_job_throughput():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slow, value in res:
        assert slow == 3.0                               # every rank sees the slowest replica's time
        assert abs(value - 2 * 32 * 10 / 3.0) < 1e-9     # whole-job units / max time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25, 1) == 1.25
    assert bench.aggregate_throughput(1, 32, 10, 1.0, 2.0) == 160.0
