"""Layer-wise sweep with a checkpoint after every layer.

The paper stores the captured activations per layer and optimises one rotation
at a time (Section 3, "Training Cost"); a sweep over 80 layers is therefore a
sequence of independent fits, and an interrupted one can go on where it stopped.
This harness writes, after each finished layer, the layer's rotation (float32)
and loss history, and the index of the next layer, into a directory:

    <dir>/layer_0007.npz   R (d x d float32), loss_history (float64), report fields
    <dir>/state.json       {"next_layer": 8, "layers": 80, "steps": 50, "lr": 0.01}

Resuming = reading state.json, loading the rotations of the finished layers and
fitting from `next_layer` on.  Files are written to a temporary name and renamed,
so a crash in the middle of a write leaves the previous state intact.  All
arithmetic stays in the library (`ctx.fit`); this file only sequences and stores.
"""
from __future__ import annotations

import json
import os

import numpy as np
import torch


def _state_path(path):
    return os.path.join(path, "state.json")


def _layer_path(path, l):
    return os.path.join(path, "layer_%04d.npz" % l)


def _atomic(write, final):
    tmp = final + ".tmp"
    write(tmp)
    os.replace(tmp, final)


def read_state(path):
    """The checkpoint's state dict, or None when there is no (complete) checkpoint."""
    try:
        with open(_state_path(path)) as f:
            return json.load(f)
    except (OSError, ValueError):
        return None


def fit_layers_checkpointed(ctx, Xs, Rs, steps, lr, path, stop_after=None):
    """Fits Rs[l] on Xs[l] for every layer, in order, with a checkpoint in directory `path` after each layer.

    If `path` holds a checkpoint of a sweep with the same number of layers, steps and lr, the rotations of its
    finished layers are loaded into Rs and the sweep continues at its next layer; otherwise it starts at layer 0.
    `stop_after` = k ends the call after k layers have been fitted in this call (how the tests interrupt a sweep).
    Returns a list with one dict per layer finished so far: loss_history, loss_first, loss_last, orth_err."""
    os.makedirs(path, exist_ok=True)
    L = len(Xs)
    st = read_state(path)
    first = 0
    if st and st.get("layers") == L and st.get("steps") == steps and st.get("lr") == lr:
        first = int(st["next_layer"])
    reports = []
    for l in range(first):
        with np.load(_layer_path(path, l)) as z:
            Rs[l].copy_(torch.from_numpy(z["R"]).to(Rs[l].device))
            reports.append(dict(loss_history=z["loss_history"].tolist(), loss_first=float(z["loss_first"]),
                                loss_last=float(z["loss_last"]), orth_err=float(z["orth_err"]), resumed=True))
    done_here = 0
    for l in range(first, L):
        if stop_after is not None and done_here >= stop_after:
            break
        rep = ctx.fit(Xs[l], Rs[l], steps, lr, history=True)
        R_host = Rs[l].detach().cpu().numpy()
        _atomic(lambda tmp: _savez(tmp, R=R_host, loss_history=np.asarray(rep["loss_history"], dtype=np.float64),
                                   loss_first=rep["loss_first"], loss_last=rep["loss_last"],
                                   orth_err=rep["orth_err"]), _layer_path(path, l))
        _atomic(lambda tmp: _dump(tmp, dict(next_layer=l + 1, layers=L, steps=steps, lr=lr)), _state_path(path))
        reports.append(dict(loss_history=rep["loss_history"], loss_first=rep["loss_first"],
                            loss_last=rep["loss_last"], orth_err=rep["orth_err"], resumed=False))
        done_here += 1
    return reports


def _savez(tmp, **arrays):
    with open(tmp, "wb") as f:
        np.savez(f, **arrays)


def _dump(tmp, obj):
    with open(tmp, "w") as f:
        json.dump(obj, f)
