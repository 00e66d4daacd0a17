"""The N > 1 part of the benchmark protocol on CPU: two gloo ranks, max-over-ranks timing, aggregate value.

The path itself does not shard (P workers are simulated inside one SF buffer), so bench.py --gpus N
runs N independent replicas; the only cross-rank logic is the timing reduction tested here.
"""
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
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms, e2e = bench.max_over_ranks([10.0 + rank, 40.0 - 5 * rank])
    dist.barrier()
    out.put((rank, ms, e2e, bench.whole_job_throughput(4096, 20, ms, world)))
    dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_sum_the_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, value in res:
        assert ms == 11.0 and e2e == 40.0               # slowest rank decides, on every rank
        assert abs(value - 2 * 4096 * 20 / 11e-3) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.5]) == [3.0, 4.5]
    assert bench.whole_job_throughput(100, 10, 500.0, 1) == 2000.0
