"""The N > 1 benchmark path (independent replicas, max-over-ranks timing) on two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_13285_b200 import multirank


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    info = multirank.rank_info(os.environ)
    multirank.barrier(dist)
    # rank r "measures" (10 + r) ms per step and 1.5 ms decode time, and streams (r + 1) * 100 bytes
    times, work = multirank.reduce_times_and_work([10.0 + rank, 1.5 - 0.25 * rank], (rank + 1) * 100.0, dist)
    multirank.barrier(dist)
    out.put((info["rank"], info["world"], times, work))
    dist.destroy_process_group()


def test_two_replicas_max_time_and_summed_work():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, w, times, work in got:
        assert w == 2
        assert times == [11.0, 1.5]          # slowest rank sets each time
        assert work == 300.0                 # replicas' work adds up
    assert multirank.job_throughput(300.0, 11.0) == 300.0 / 0.011


def test_single_rank_needs_no_process_group():
    times, work = multirank.reduce_times_and_work([3.0], 7.0, None)
    assert times == [3.0] and work == 7.0
    assert multirank.rank_info({}) == {"rank": 0, "local_rank": 0, "world": 1}
