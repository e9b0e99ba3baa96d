"""Plumbing for bench.py at N > 1: one process per GPU.

Two ways to use several GPUs.  Layers are independent problems (each has its own rotation): sharded over
ranks they exchange no data on the compute path, and the process group is used only for the start barrier,
for the maximum of the per-rank times and for summing the work done.  One rotation over many tokens is the
other: the rows of X are sharded (`fit_row_sharded` -> kt_fit_sharded), every rank computes the loss and gradient of
its rows, and the library calls back, while it enqueues a step, for one sum all-reduce of dR (d x d float32) and of
the loss, which makes the step identical on all ranks.
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


class _DeviceBuffer:
    """A raw device pointer dressed up for torch.as_tensor (no copy)."""

    def __init__(self, ptr, count, typestr):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (ptr, False), "version": 2}


def all_reduce_hook(dist, device):
    """The `reduce` callable of Context.fit_sharded: an in-place SUM all-reduce, through torch.distributed, of the
    buffer the library hands over (NCCL for device memory: the collective is ordered after the work already enqueued
    on torch's current stream, which must be the context's stream, and nothing waits on the host; gloo for the CPU
    tests).  Returns None when there is one process only."""
    if dist is None:
        return None
    import ctypes as C
    dev = torch.device(device)
    views = {}

    def reduce(ptr, count, dtype, stream):
        key = (ptr, count, dtype)
        t = views.get(key)
        if t is None:
            if dev.type == "cuda":
                t = torch.as_tensor(_DeviceBuffer(ptr, count, "<f4" if dtype == 1 else "<f8"), device=dev)
            else:
                ctype = C.c_float if dtype == 1 else C.c_double
                t = torch.frombuffer((ctype * count).from_address(ptr),
                                     dtype=torch.float32 if dtype == 1 else torch.float64)
            views[key] = t
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return 0

    return reduce


def fit_row_sharded(ctx, X_local, R, steps, lr, dist, rows_total):
    """One rotation over a batch whose rows are spread over the ranks: `ctx.fit_sharded` (kt_fit_sharded) on this
    rank's rows with the all-reduce hook above.  The loss is a mean over all `rows_total` tokens; per step the
    library sums the loss and dR (d x d float32) over the ranks -- and, for the whole-layer loss, the batch's mean
    and central sums -- on its stream, without a host round trip, and every rank then takes the same step, so the
    replicas of R stay bit-identical without ever being exchanged.  Returns the per-step losses of the whole batch."""
    rep = ctx.fit_sharded(X_local, R, rows_total, all_reduce_hook(dist, R.device), steps, lr, history=True)
    return rep["loss_history"]


def finalize(dist):
    if dist is not None and dist.is_initialized():
        dist.destroy_process_group()
