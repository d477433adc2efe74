"""The N > 1 host logic (replicas, no data-path collective) on CPU with the gloo backend, world size 2."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2308_14711_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        elapsed = [12.5, 20.0][rank]                       # rank 1 is the slow one
        mx = replicas.max_over_ranks(elapsed, dist)
        value = replicas.whole_job_throughput(1000, 10, world, mx)
        lo, hi = replicas.token_shard(1001, rank, world)
        dist.barrier()
        out.put((rank, mx, value, lo, hi))
    finally:
        dist.destroy_process_group()


def test_two_replicas_take_the_slowest_rank_and_add_up_tokens():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, mx, value, lo, hi in res:
        assert mx == 20.0
        assert abs(value - 2 * 1000 * 10 / 20e-3) < 1e-6
    assert (res[0][3], res[0][4], res[1][3], res[1][4]) == (0, 501, 501, 1001)


def test_single_process_needs_no_group():
    assert replicas.max_over_ranks(3.0, None) == 3.0
    assert replicas.whole_job_throughput(50432, 4, 1, 2.0) == 50432 * 4 / 2e-3
    assert [replicas.token_shard(10, r, 3) for r in range(3)] == [(0, 4), (4, 7), (7, 10)]
