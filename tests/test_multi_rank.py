"""The multi-process path of the benchmark (one independent problem per rank, barrier, maximum of
the ranks' times, whole-job throughput) on two CPU ranks over gloo."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seconds = 0.5 + 0.25 * rank                       # rank 1 is the slower one
        agg = bench.aggregate_over_ranks(seconds, units_per_rank=1000.0, dist=dist, device="cpu")
        out.put((rank, agg))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_whole_job_throughput_at_the_slowest_ranks_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank in range(world):
        seconds, value = results[rank]
        assert abs(seconds - 0.75) < 1e-9                 # the maximum over the ranks
        assert abs(value - 2 * 1000.0 / 0.75) < 1e-6      # all ranks' units over that time


def test_single_rank_needs_no_process_group():
    import bench
    seconds, value = bench.aggregate_over_ranks(0.5, units_per_rank=10.0, dist=None, device="cpu")
    assert seconds == 0.5 and value == 20.0
