"""Plumbing for bench.py at N > 1: one process per GPU.

Two ways to use several GPUs.  Layers are independent problems (each has its own rotation): sharded over
ranks they exchange no data on the compute path, and the process group is used only for the start barrier,
for the maximum of the per-rank times and for summing the work done.  One rotation over many tokens is the
other: the rows of X are sharded (`fit_row_sharded`), every rank computes the loss and gradient of its rows,
and one sum all-reduce per step of dR (d x d float32) and of the loss makes the step identical on all ranks.
Works with NCCL (GPU) and gloo (CPU tests).
"""
from __future__ import annotations

import os

import torch


def env_rank():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend, device=None):
    """Initialises the default process group from the torchrun environment (no-op at world size 1)."""
    rank, _, world = env_rank()
    if world == 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kw = {}
        if backend == "nccl" and device is not None:
            kw["device_id"] = torch.device(device)
        dist.init_process_group(backend, **kw)
    return dist


def barrier(dist):
    if dist is not None:
        dist.barrier()


def max_over_ranks(dist, value, device="cpu"):
    """Largest `value` (a float) over all ranks."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(dist, value, device="cpu"):
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def layers_of_rank(n_layers, rank, world):
    """Contiguous block of layer indices owned by `rank` (sizes differ by at most one)."""
    base, extra = divmod(n_layers, world)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


def whole_job_throughput(dist, units_this_rank, seconds_this_rank, device="cpu"):
    """Units processed by all ranks divided by the slowest rank's time."""
    total = sum_over_ranks(dist, units_this_rank, device)
    t = max_over_ranks(dist, seconds_this_rank, device)
    return total / t, t


def fit_row_sharded(ctx, X_local, R, steps, lr, dist, rows_total):
    """`steps` x (loss and gradient of this rank's rows; all-reduce; step on the orthogonal group).

    The loss is a mean over all `rows_total` tokens (per-token mode), so the full-batch gradient is the sum over
    ranks of (rows of the rank / rows_total) x the rank's own gradient: one SUM all-reduce of dR and one of the
    loss per step.  Every rank then takes the same step from the same dR, so the replicas of R stay bit-identical
    without ever being exchanged.  `ctx` needs loss_grad(X, R) -> (loss, dR) and orth_step(R, dR, lr) (the
    library's Context); returns the per-step full-batch losses."""
    w = float(X_local.shape[0]) / float(rows_total)
    losses = []
    for _ in range(steps):
        loss, dR = ctx.loss_grad(X_local, R)
        dR.mul_(w)
        lt = torch.tensor([loss * w], dtype=torch.float64, device=dR.device)
        if dist is not None:
            dist.all_reduce(dR, op=dist.ReduceOp.SUM)
            dist.all_reduce(lt, op=dist.ReduceOp.SUM)
        ctx.orth_step(R, dR, lr)
        losses.append(float(lt.item()))
    return losses


def finalize(dist):
    if dist is not None and dist.is_initialized():
        dist.destroy_process_group()
