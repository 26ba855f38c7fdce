"""The N > 1 path of bench.py on CPU: two gloo ranks shard the requests, time different durations, and agree
on the max-over-ranks time and the whole-job throughput."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2209_13443_b200 import replicas


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    first, count = replicas.rank_requests(rank, world, 64)
    my_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    dist.barrier()
    mx = replicas.max_over_ranks(my_ms, dist, "cpu")
    q.put((rank, first, count, mx, replicas.job_throughput(world, 64, 20, mx)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_over_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [0, 64] and all(r[2] == 64 for r in res)          # disjoint, contiguous, complete
    assert all(r[3] == 15.0 for r in res)                                          # everyone sees the slowest rank
    assert all(abs(r[4] - 2 * 64 * 20 / 0.015) < 1e-6 for r in res)               # whole-job samples/s


def test_single_process_needs_no_process_group():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.rank_requests(0, 1, 8) == (0, 8)
