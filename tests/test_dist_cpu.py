"""The multi-rank plumbing of the benchmark (independent replicas, max-over-ranks timing) on two gloo ranks."""
import os
import socket

import torch.multiprocessing as mp

from paper_2605_11354_b200 import dist as pdist


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def worker(rank, world, port, results):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, lr, w = pdist.init(backend="gloo")
    assert (r, lr, w) == (rank, rank, world)
    pdist.barrier()
    local_seconds = 1.0 + rank  # rank 1 is the slow one
    worst = pdist.max_over_ranks(local_seconds)
    rate, worst2 = pdist.aggregate_throughput(10.0, local_seconds)
    results.put((rank, worst, rate, worst2))
    pdist.barrier()
    pdist.shutdown()


def test_two_rank_replicas_use_the_slowest_rank_time():
    ctx = mp.get_context("spawn")
    results = ctx.Queue()
    port = free_port()
    procs = [ctx.Process(target=worker, args=(r, 2, port, results)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(results.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, worst, rate, worst2 in got:
        assert worst == 2.0 and worst2 == 2.0
        assert rate == 20.0 / 2.0  # both ranks' units over the slowest rank's time


def test_single_process_defaults():
    for key in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(key, None)
    assert pdist.env_world() == (0, 0, 1)
    assert pdist.max_over_ranks(3.5) == 3.5
    assert pdist.aggregate_throughput(8.0, 2.0) == (4.0, 2.0)
