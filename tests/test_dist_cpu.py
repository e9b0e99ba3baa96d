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


class _OracleCtx:
    """Stands in for the library's Context on the CPU: fit_sharded with the library's sequence of reductions per
    step (the loss, then dR, each already weighted by this shard's share of the rows), computed by the float64
    oracle and summed through the very hook the GPU path hands to kt_fit_sharded."""

    def fit_sharded(self, X, R, rows_total, reduce, steps, lr, history=False):
        from oracle import kurtail_oracle as ko
        w = X.shape[0] / float(rows_total)
        losses = []
        for _ in range(steps):
            L, dR = ko.loss_grad(X.numpy(), R.numpy())
            loss_t = torch.tensor([L * w], dtype=torch.float64)
            dR_t = torch.from_numpy(dR * w).contiguous()
            if reduce is not None:
                assert reduce(loss_t.data_ptr(), 1, 2, None) == 0
                assert reduce(dR_t.data_ptr(), dR_t.numel(), 2, None) == 0
            Rn, _, _ = ko.orth_step(R.numpy(), dR_t.numpy(), lr)
            R.copy_(torch.from_numpy(Rn))
            losses.append(float(loss_t.item()))
        return dict(loss_history=losses)


def _problem():
    g = torch.Generator().manual_seed(5)
    X = torch.randn((48, 8), generator=g, dtype=torch.float64)
    X[:, 3] *= 25.0
    return X, torch.eye(8, dtype=torch.float64)


def _shard_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist = dist_util.init("gloo")
    X, R = _problem()
    rows = [slice(0, 16), slice(16, 48)][rank]          # unequal shards: the weights matter
    losses = dist_util.fit_row_sharded(_OracleCtx(), X[rows], R, 5, 1e-2, dist, X.shape[0])
    out.put((rank, losses, R.numpy().tolist()))
    dist_util.barrier(dist)
    dist_util.finalize(dist)


def test_row_sharded_fit_equals_the_full_batch_fit():
    import numpy as np
    from oracle import kurtail_oracle as ko
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    X, R0 = _problem()
    R_ref, losses_ref = ko.fit(X.numpy(), R0.numpy(), 5, 1e-2)
    assert res[0][2] == res[1][2]                                    # replicas bit-identical
    assert np.abs(np.array(res[0][2]) - R_ref).max() < 1e-12
    assert np.allclose(res[0][1], losses_ref, rtol=1e-12) and res[0][1] == res[1][1]
    # one rank alone: the plain loop
    X, R = _problem()
    assert np.allclose(dist_util.fit_row_sharded(_OracleCtx(), X, R, 5, 1e-2, None, X.shape[0]), losses_ref, rtol=1e-12)


def _hook_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist = dist_util.init("gloo")
    hook = dist_util.all_reduce_hook(dist, "cpu")
    a = torch.full((6,), float(rank + 1), dtype=torch.float32)
    b = torch.tensor([0.5 + rank], dtype=torch.float64)
    for _ in range(2):                                   # the second call reuses the cached view of the buffer
        assert hook(a.data_ptr(), a.numel(), 1, None) == 0
    assert hook(b.data_ptr(), 1, 2, None) == 0
    out.put((rank, a.tolist(), b.tolist()))
    dist_util.barrier(dist)
    dist_util.finalize(dist)


def test_all_reduce_hook_sums_raw_buffers_in_place():
    # the hook receives what kt_fit_sharded hands it: an address, a count and a type code (1 float32, 2 float64)
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_hook_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # first reduction: 1 + 2 = 3 on both ranks; second: 3 + 3 = 6
    assert res[0][1] == res[1][1] == [6.0] * 6
    assert res[0][2] == res[1][2] == [2.0]
    assert dist_util.all_reduce_hook(None, "cpu") is None
