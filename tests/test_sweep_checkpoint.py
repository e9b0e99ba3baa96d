"""The layer-wise sweep's checkpoint/resume harness (Section 3, "Training Cost": one rotation at a time)."""
import json
import os

import numpy as np
import pytest
import torch

from paper_2503_01483_b200 import sweep


class _FakeCtx:
    """Counts the fits and moves R deterministically, so the host-side sequencing can be checked without a GPU."""

    def __init__(self):
        self.fitted = []

    def fit(self, X, R, steps, lr, history=False):
        self.fitted.append(int(X[0, 0].item()))
        losses = []
        for k in range(steps):
            R.mul_(1.0 - lr).add_(X[:R.shape[0], :R.shape[1]] * lr)
            losses.append(float(R.sum().item()))
        return dict(loss_history=losses, loss_first=losses[0], loss_last=losses[-1], orth_err=0.0)


def _problem(L=5, d=4):
    Xs = [torch.full((d, d), float(l)) + torch.arange(d * d, dtype=torch.float32).reshape(d, d) / 100 for l in range(L)]
    Rs = [torch.eye(d) for _ in range(L)]
    return Xs, Rs


def test_interrupted_sweep_resumes_where_it_stopped(tmp_path):
    Xs, Rs_full = _problem()
    full = sweep.fit_layers_checkpointed(_FakeCtx(), Xs, Rs_full, 3, 0.25, str(tmp_path / "a"))
    assert len(full) == 5 and not any(r["resumed"] for r in full)

    Xs, Rs = _problem()
    c1 = _FakeCtx()
    part = sweep.fit_layers_checkpointed(c1, Xs, Rs, 3, 0.25, str(tmp_path / "b"), stop_after=2)
    assert c1.fitted == [0, 1] and len(part) == 2
    assert sweep.read_state(str(tmp_path / "b"))["next_layer"] == 2
    # a new process: rotations start from scratch, the finished ones come back from the files
    Xs, Rs = _problem()
    c2 = _FakeCtx()
    rest = sweep.fit_layers_checkpointed(c2, Xs, Rs, 3, 0.25, str(tmp_path / "b"))
    assert c2.fitted == [2, 3, 4]
    assert [r["resumed"] for r in rest] == [True, True, False, False, False]
    for a, b in zip(Rs, Rs_full):
        assert torch.equal(a, b)
    assert [r["loss_history"] for r in rest] == [r["loss_history"] for r in full]
    # a finished sweep has nothing left to do
    c3 = _FakeCtx()
    again = sweep.fit_layers_checkpointed(c3, Xs, Rs, 3, 0.25, str(tmp_path / "b"))
    assert c3.fitted == [] and all(r["resumed"] for r in again)


def test_checkpoint_of_another_sweep_is_not_resumed(tmp_path):
    Xs, Rs = _problem()
    sweep.fit_layers_checkpointed(_FakeCtx(), Xs, Rs, 3, 0.25, str(tmp_path), stop_after=3)
    Xs, Rs = _problem()
    c = _FakeCtx()
    sweep.fit_layers_checkpointed(c, Xs, Rs, 4, 0.25, str(tmp_path), stop_after=1)      # other step count: from layer 0
    assert c.fitted == [0]
    # a torn state file (a crash while writing never leaves one, but a foreign file may be there) means no checkpoint
    with open(os.path.join(str(tmp_path), "state.json"), "w") as f:
        f.write("{not json")
    assert sweep.read_state(str(tmp_path)) is None
    # leftovers of an interrupted write are ignored
    assert not [n for n in os.listdir(str(tmp_path)) if n.endswith(".tmp")]


@pytest.mark.gpu
def test_gpu_sweep_resume_is_bit_identical(tmp_path):
    from paper_2503_01483_b200 import kurtail, synth
    dev = "cuda:0"
    ctx = kurtail.Context(dev)
    Xs = [synth.activations(1000, 256, "student_t", 2.5, 4, 200.0, seed=1000 + l, device=dev) for l in range(4)]
    Ra = [ctx.init_rotation(256, "hadamard") for _ in Xs]
    ref = ctx.fit_layers(Xs, Ra, 5, 1e-2)
    Rb = [ctx.init_rotation(256, "hadamard") for _ in Xs]
    sweep.fit_layers_checkpointed(ctx, Xs, Rb, 5, 1e-2, str(tmp_path), stop_after=1)
    assert json.load(open(os.path.join(str(tmp_path), "state.json")))["next_layer"] == 1
    Rc = [ctx.init_rotation(256, "hadamard") for _ in Xs]
    reps = sweep.fit_layers_checkpointed(ctx, Xs, Rc, 5, 1e-2, str(tmp_path))
    assert [r["resumed"] for r in reps] == [True, False, False, False]
    for a, c in zip(Ra, Rc):
        assert torch.equal(a, c)
    assert [r["loss_last"] for r in reps] == [r["loss_last"] for r in ref]
    assert np.isfinite([r["orth_err"] for r in reps]).all()
    ctx.close()
