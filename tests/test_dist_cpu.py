"""The N > 1 plumbing of the benchmark, exercised with two gloo ranks on the CPU."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2503_01483_b200 import dist_util


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist = dist_util.init("gloo")
    dist_util.barrier(dist)
    layers = dist_util.layers_of_rank(5, rank, world)
    # rank r "processes" 1000 units per layer in (1 + r) seconds
    value, t = dist_util.whole_job_throughput(dist, 1000.0 * len(layers), 1.0 + rank)
    mx = dist_util.max_over_ranks(dist, 10.0 * (rank + 1))
    out.put((rank, layers, value, t, mx))
    dist_util.barrier(dist)
    dist_util.finalize(dist)


def test_two_gloo_ranks_aggregate_like_the_benchmark():
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == [0, 1, 2] and res[1][1] == [3, 4]           # every layer owned exactly once
    for _, _, value, t, mx in res:
        assert t == 2.0 and value == pytest.approx(5000.0 / 2.0)   # all units / slowest rank
        assert mx == 20.0


def test_single_rank_is_a_no_op():
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert dist_util.init("gloo") is None
    assert dist_util.max_over_ranks(None, 3.5) == 3.5
    assert dist_util.layers_of_rank(7, 0, 1) == list(range(7))
    assert sorted(sum((dist_util.layers_of_rank(80, r, 8) for r in range(8)), [])) == list(range(80))
