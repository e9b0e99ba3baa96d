"""Cayley Adam on the GPU (kt_adam_step, kt_fit with optimizer = 1) against the float64 oracle's
cayley_adam_step, teacher-forced: every GPU step starts from the state the oracle is given."""
import numpy as np
import pytest
import torch

from oracle import kurtail_oracle as ko
from paper_2503_01483_b200 import kurtail, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def f64(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def make_x(N, d, seed):
    return synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=4, outlier_scale=50.0, seed=seed,
                             dtype=torch.bfloat16, device=DEV)


@pytest.fixture(scope="module")
def ctx():
    c = kurtail.Context(DEV)
    yield c
    c.close()


@pytest.mark.parametrize("d,lr", [(128, 1e-2), (256, 1e-2), (1024, 1e-2), (512, 5e-2)])
def test_adam_steps_match_oracle_teacher_forced(ctx, d, lr):
    X = make_x(1024, d, seed=91)
    R = synth.random_orthogonal(d, seed=11, device=DEV).contiguous()
    M = torch.zeros((d, d), dtype=torch.float32, device=DEV)
    state = dict(v=0.0, step=0)
    for it in range(4):
        _, dR = ctx.loss_grad(X, R)
        R0, dR0 = f64(R), f64(dR)
        ost = dict(M=f64(M), v=state["v"], k=state["step"])
        ref = ko.cayley_adam_step(R0, dR0, ost, lr, beta1=0.9, beta2=0.99, adam_eps=1e-8, iters=2, q=0.5, eps=1e-8,
                                  polish_thresh=1e-5)
        ctx.adam_step(R, dR, M, state, lr)
        assert state["step"] == ost["k"] == it + 1
        assert state["v"] == pytest.approx(ost["v"], rel=1e-6)
        # momentum: bf16 M in the product M R^T and bf16 W in W R (2^-9 relative each, random)
        assert np.linalg.norm(f64(M) - ost["M"]) <= 1e-2 * np.linalg.norm(ost["M"])
        upd = np.abs(ref - R0).max()
        assert np.abs(f64(R) - ref).max() <= 2e-2 * upd + 3e-7, it
        assert ko.orthogonality_error(f64(R)) <= 2e-5


def test_adam_momentum_stays_in_the_tangent_space(ctx):
    # after a step M = r W R with W skew: M R^T is skew
    d = 256
    X = make_x(512, d, seed=92)
    R = synth.random_orthogonal(d, seed=12, device=DEV).contiguous()
    M = torch.zeros((d, d), dtype=torch.float32, device=DEV)
    state = dict(v=0.0, step=0)
    Rprev = R.clone()
    _, dR = ctx.loss_grad(X, R)
    ctx.adam_step(R, dR, M, state, 1e-2)
    A = f64(M) @ f64(Rprev).T
    assert np.abs(A + A.T).max() <= 1e-5 * np.abs(A).max()


def test_adam_zero_gradient_keeps_r(ctx):
    d = 256
    R = synth.random_orthogonal(d, seed=13, device=DEV).contiguous()
    M = torch.zeros((d, d), dtype=torch.float32, device=DEV)
    state = dict(v=0.0, step=0)
    Rn = ctx.adam_step(R.clone(), torch.zeros_like(R), M, state, 1e-2)
    assert np.abs(f64(Rn) - f64(R)).max() <= 2e-7
    assert state["step"] == 1 and state["v"] == 0.0
    assert float(M.abs().max()) == 0.0


@pytest.mark.parametrize("d", [128, 256, 1024])
def test_fit_adam_equals_composed_calls(d):
    c = kurtail.Context(DEV, optimizer=1, guard_every=1)
    X = make_x(1500, d, seed=93)
    Ra = c.init_rotation(d, "hadamard")
    Rb = Ra.clone()
    rep = c.fit(X, Ra, 4, 1e-2, history=True)
    M = torch.zeros((d, d), dtype=torch.float32, device=DEV)
    state = dict(v=0.0, step=0)
    losses = []
    for _ in range(4):
        l, dR = c.loss_grad(X, Rb)
        losses.append(l)
        c.adam_step(Rb, dR, M, state, 1e-2)
    assert torch.equal(Ra, Rb)
    assert losses == rep["loss_history"]
    c.close()


def test_fit_adam_descends_and_stays_orthogonal():
    c = kurtail.Context(DEV, optimizer=1)
    X = synth.activations(4096, 512, dist="student_t", nu=3.0, n_outliers=8, outlier_scale=100.0, seed=94,
                          dtype=torch.bfloat16, device=DEV)
    R = c.init_rotation(512, "identity")
    L0 = c.kurtosis_loss(X, R)
    # Adam normalises the direction (||W||_F <= 1): a step moves R by about lr, so lr = 0.05 here
    rep = c.fit(X, R, 100, 5e-2)
    assert rep["steps_done"] == 100
    assert c.kurtosis_loss(X, R) < 0.5 * L0
    assert c.orth_error(R) <= 1e-4 and ko.orthogonality_error(f64(R)) <= 1e-4
    # a second fit on the same context starts from a zero state again: same result from the same start
    R2 = c.init_rotation(512, "identity")
    c.fit(X, R2, 100, 5e-2)
    assert torch.equal(R, R2)
    c.close()


@pytest.mark.parametrize("d", [128, 384, 512])
def test_adam_one_launch_step_is_float32_exact_and_agrees_with_the_tensor_core_path(d):
    # d <= 512: the whole Cayley-Adam step is one cooperative launch with float32 products, so it follows the oracle
    # far more closely than the bf16 tensor-core path, which stays available (small_d_orth = 0) and must agree
    X = make_x(700, d, seed=93)
    R0t = synth.random_orthogonal(d, seed=13, device=DEV).contiguous()
    one = kurtail.Context(DEV)
    gen = kurtail.Context(DEV, small_d_orth=0)
    Ra, Rb = R0t.clone(), R0t.clone()
    Ma = torch.zeros((d, d), dtype=torch.float32, device=DEV)
    Mb = torch.zeros_like(Ma)
    sa, sb = dict(v=0.0, step=0), dict(v=0.0, step=0)
    for it in range(3):
        _, dR = one.loss_grad(X, Ra)
        ost = dict(M=f64(Ma), v=sa["v"], k=sa["step"])
        ref = ko.cayley_adam_step(f64(Ra), f64(dR), ost, 1e-2, beta1=0.9, beta2=0.99, adam_eps=1e-8, iters=2, q=0.5,
                                  eps=1e-8, polish_thresh=1e-5)
        R_in = f64(Ra)
        Rb.copy_(Ra)
        Mb.copy_(Ma)
        sb.update(sa)
        one.adam_step(Ra, dR, Ma, sa, 1e-2)
        gen.adam_step(Rb, dR, Mb, sb, 1e-2)
        upd = np.abs(ref - R_in).max()
        assert sa["step"] == sb["step"] == ost["k"] == it + 1
        # (beta2 reaches the library as a float32: 1 - beta2 differs from the oracle's by 1e-6 of itself)
        assert sa["v"] == pytest.approx(ost["v"], rel=2e-6) and sb["v"] == pytest.approx(ost["v"], rel=2e-6)
        assert np.linalg.norm(f64(Ma) - ost["M"]) <= 2e-5 * np.linalg.norm(ost["M"])
        assert np.abs(f64(Ra) - ref).max() <= 1e-3 * upd + 3e-7
        assert np.abs(f64(Rb) - ref).max() <= 2e-2 * upd + 3e-7
        assert ko.orthogonality_error(f64(Ra)) <= 2e-5
    one.close()
    gen.close()
