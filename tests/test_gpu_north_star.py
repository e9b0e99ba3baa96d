"""The stated tolerances at the stated sizes, on the code paths the benchmark runs.

  * dR against the float64 oracle (relative Frobenius error <= 1e-2) at d = 4096, 8192 and 14336 on ragged row
    slices the oracle can afford (a few hundred rows at full d);
  * one step on the orthogonal group at d = 4096 and d = 8192, in the default configuration (the device chooses
    how many series terms and how many bf16 terms of R to use), against the oracle's stepwise Cayley step;
  * 100 steps of kt_fit on the tensor-core path (d = 1024 and d = 4096, Cayley SGD and Cayley Adam) with
    max|R^T R - I| <= 1e-4 computed in float64 on the host, not by the library's own guard;
  * teacher-forced steps of the default kt_fit at d = 1024;
  * the kurtosis does not depend on the scale of X, and neither do loss and gradient of the library.
"""
import numpy as np
import pytest
import torch

from oracle import kurtail_oracle as ko
from paper_2503_01483_b200 import build, kurtail, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = kurtail.Context(DEV)
    yield c
    c.close()


def f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def rel_fro(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def _gpu_qr(d, seed):
    g = torch.Generator(device=DEV).manual_seed(seed)
    Q, _ = torch.linalg.qr(torch.randn((d, d), device=DEV, generator=g))
    return Q.contiguous()


# ------------------------------------------------------------------ gradient
@pytest.mark.parametrize("workload,rows,init", [("llama2_7b_attn", 1000, "hadamard"),
                                                ("llama3_70b_sweep", 777, "hadamard"),
                                                ("llama3_70b_sweep", 640, "orth"),
                                                ("llama3_8b_down", 300, "orth")])
def test_gradient_matches_oracle_at_full_width(ctx, workload, rows, init):
    kw = dict(layers=1) if workload == "llama3_70b_sweep" else {}
    cfg = synth.config(workload, device=DEV, rows=rows, **kw)
    X = cfg["X"][0] if isinstance(cfg["X"], list) else cfg["X"]
    d = cfg["d"]
    assert tuple(X.shape) == (rows, d)
    R = ctx.init_rotation(d, "hadamard") if init == "hadamard" else _gpu_qr(d, seed=41)
    loss, dR = ctx.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    assert rel_fro(f64(dR), dR_ref) <= 1e-2
    # the mode that never writes Y (a second GEMM pass recomputes it) is held to the same bar, and equals the
    # mode that keeps Y in float32 bit for bit (the default keeps it in float16)
    c2 = kurtail.Context(DEV, backward_mode=1)
    l2, dR2 = c2.loss_grad(X, R)
    c2.close()
    assert l2 == loss
    assert rel_fro(f64(dR2), dR_ref) <= 1e-2
    c3 = kurtail.Context(DEV, backward_mode=2)
    l3, dR3 = c3.loss_grad(X, R)
    c3.close()
    assert l3 == loss and torch.equal(dR3, dR2)


# ------------------------------------------------------- one orthogonal step
@pytest.mark.parametrize("d,lr", [(4096, 1e-2), (4096, 20.0), (8192, 1e-2), (8192, 20.0)])
def test_orth_step_matches_oracle_at_full_width_default_configuration(ctx, d, lr):
    # lr = 1e-2 is the benchmark's regime (alpha ||W||_F ~ 1e-4: the device keeps one series term and one bf16 term
    # of R); lr = 20 makes alpha ||W||_F a few tenths, where every term of the series and the two-term split run
    wl = "llama2_7b_attn" if d == 4096 else "llama3_70b_sweep"
    cfg = synth.config(wl, device=DEV, rows=1024, **(dict(layers=1) if d == 8192 else {}))
    X = cfg["X"][0] if isinstance(cfg["X"], list) else cfg["X"]
    R = ctx.init_rotation(d, "hadamard")
    _, dR = ctx.loss_grad(X, R)
    R0, dR0 = f64(R), f64(dR)
    ref, alpha, wn = ko.orth_step(R0, dR0, lr, iters=2, q=0.5, eps=1e-8, polish_thresh=1e-5)
    Rn = ctx.orth_step(R.clone(), dR, lr)
    upd = np.abs(ref - R0).max()
    err = np.abs(f64(Rn) - ref).max()
    # the update is matched to ~1 % of its own size (W and dR enter as bf16), plus float32 rounding of R's entries
    assert err <= 2e-2 * upd + 4 * 2.0 ** -24 * np.abs(R0).max(), (err, upd, alpha * wn)
    assert rel_fro(f64(Rn) - R0, ref - R0) <= 2e-2 + 2.0 ** -22 * np.linalg.norm(R0) / np.linalg.norm(ref - R0)
    # one polish after the step: at the benchmark's step size R stays orthogonal to float32 accuracy; after a large
    # step (the truncated series leaves ~1e-3, which one Newton-Schulz correction through bf16 factors takes to
    # ~1e-5) well inside the 1e-4 bound
    assert ko.orthogonality_error(f64(Rn)) <= (1e-5 if lr < 1.0 else 5e-5)
    if lr > 1.0:
        assert alpha * wn > 0.1          # the regime this case is meant to cover


# ------------------------------------------------ 100 steps stay orthogonal
@pytest.mark.parametrize("d,optimizer,lr", [(1024, 0, 1e-2), (1024, 1, 1e-2), (4096, 0, 1e-2), (4096, 1, 1e-2),
                                            (4096, 0, 10.0)])
def test_100_steps_on_the_tensor_core_path_stay_orthogonal(d, optimizer, lr):
    c = kurtail.Context(DEV, optimizer=optimizer)
    X = synth.activations(4096 + 77, d, dist="student_t", nu=3.0, n_outliers=16, outlier_scale=100.0, seed=71,
                          dtype=torch.bfloat16, device=DEV)
    R = c.init_rotation(d, "hadamard")
    rep = c.fit(X, R, 100, lr, history=True)
    assert rep["steps_done"] == 100
    # measured on the host in float64, not by the guard that kept it
    assert ko.orthogonality_error(f64(R)) <= 1e-4
    assert rep["orth_err"] <= 1e-4
    h = rep["loss_history"]
    assert np.isfinite(h).all() and min(h[-5:]) < h[0]
    c.close()


# ----------------------------------------------------- teacher-forced steps
def test_default_fit_steps_follow_the_oracle_teacher_forced(ctx):
    # kt_fit itself (adaptive terms, bf16 dR straight from the split-K sum), one step at a time from the GPU's own R_k
    d = 1024
    X = synth.activations(1500, d, dist="student_t", nu=3.0, n_outliers=8, outlier_scale=100.0, seed=72,
                          dtype=torch.bfloat16, device=DEV)
    R = ctx.init_rotation(d, "hadamard")
    for lr in (1e-2, 1e-2, 3.0):
        Rk = f64(R)
        L_ref, dR_ref = ko.loss_grad(f64(X), Rk)
        ref, _, _ = ko.orth_step(Rk, dR_ref, lr, polish_thresh=1e-5)
        rep = ctx.fit(X, R, 1, lr)
        assert abs(rep["loss_first"] - L_ref) <= 1e-3 * abs(L_ref)
        assert np.linalg.norm(f64(R) - ref) <= 2e-2 * np.linalg.norm(ref - Rk) + 2.0 ** -23 * np.linalg.norm(Rk)


# ----------------------------------------------------------- scale freedom
@pytest.mark.parametrize("d,log2_scale", [(128, -40), (128, 30), (256, -12), (1024, 10)])
def test_loss_and_gradient_do_not_depend_on_the_scale_of_x(ctx, d, log2_scale):
    # kappa(s y) = kappa(y): the loss and dL/dR are the same for X and s X.  d = 128 runs the single-pass kernel,
    # which normalises every row by a power of two before taking power sums (2^-40 would otherwise underflow them)
    N = 3000
    X = synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=2, outlier_scale=30.0, seed=73,
                          dtype=torch.bfloat16, device=DEV)
    R = synth.random_orthogonal(d, seed=17, device=DEV).contiguous()
    Xs = (X.float() * 2.0 ** log2_scale).to(torch.bfloat16)          # exact: a power of two
    assert torch.equal(Xs.float() * 2.0 ** -log2_scale, X.float())
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    L_ref_s, dR_ref_s = ko.loss_grad(f64(Xs), f64(R))
    assert L_ref_s == pytest.approx(L_ref, rel=1e-12) and rel_fro(dR_ref_s, dR_ref) <= 1e-12   # the oracle's own
    l0, g0 = ctx.loss_grad(X, R)
    l1, g1 = ctx.loss_grad(Xs, R)
    for l, g in ((l0, g0), (l1, g1)):
        assert abs(l - L_ref) <= 1e-3 * abs(L_ref)
        assert rel_fro(f64(g), dR_ref) <= 1e-2
    if d == 128:
        assert l1 == l0 and torch.equal(g1, g0)       # power-of-two scaling changes no bit of the single-pass kernel
    if abs(log2_scale) <= 12:
        # the three-GEMM path takes its power sums in float32 on the rows as they are: fine for any activations a
        # network produces (row rms between about 1e-8 and 1e8), not for 2^-40
        assert abs(ctx.kurtosis_loss(Xs, R) - L_ref) <= 1e-3 * abs(L_ref)


def test_rmsnorm_makes_the_three_gemm_path_scale_free():
    # with the RMSNorm of the paper's small network behind the rotation (rms_eps = 0) every row is brought to unit
    # mean square in float32 before its moments are taken: X 2^-40 gives the loss and gradient of X
    d, N = 256, 2000
    c = kurtail.Context(DEV, rmsnorm=1, rms_eps=0.0)
    X = synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=4, outlier_scale=50.0, seed=74,
                          dtype=torch.bfloat16, device=DEV)
    X[5] = 0.0                                                     # a zero row: factor 0, contributes nothing
    R = synth.random_orthogonal(d, seed=18, device=DEV).contiguous()
    Xs = (X.float() * 2.0 ** -40).to(torch.bfloat16)
    L_ref, dR_ref = ko.loss_grad(ko.rmsnorm_rows(f64(X), 0.0 + 1e-300), f64(R))
    for x in (X, Xs):
        l, g = c.loss_grad(x, R)
        assert abs(l - L_ref) <= 1e-3 * abs(L_ref)
        assert rel_fro(f64(g), dR_ref) <= 1e-2
    c.close()


# ------------------------------------------- the gradient away from a bf16-exact rotation
@pytest.mark.parametrize("workload,d,rows,steps", [("llama2_7b_attn", 4096, 4096, 3), ("llama2_7b_attn", 4096, 2048, 40),
                                                   ("llama3_70b_sweep", 8192, 2048, 40)])
def test_gradient_at_a_rotation_that_bf16_cannot_hold(workload, d, rows, steps):
    # The Hadamard start is exact in bf16; a few steps later R = H + (updates far below bf16's spacing at 1/sqrt(d)),
    # and a forward pass on bf16(R) would evaluate the gradient at H again: 2e-2 of its norm away from the gradient at
    # R.  The default forward pass keeps R as float16 (three more bits) and must stay inside the 1e-2 tolerance there;
    # the bf16 variant is run beside it to show the case is the hard one.
    kw = dict(layers=1) if workload == "llama3_70b_sweep" else {}
    cfg = synth.config(workload, device=DEV, rows=rows, **kw)
    X = cfg["X"][0] if isinstance(cfg["X"], list) else cfg["X"]
    c = kurtail.Context(DEV)
    R = c.init_rotation(d, "hadamard")
    c.fit(X, R, steps, 1e-2)
    assert float((R - R.to(torch.bfloat16).float()).abs().max()) > 0.0       # not bf16-exact any more
    loss, dR = c.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    err = rel_fro(f64(dR), dR_ref)
    assert err <= 6e-3, err
    c.close()
    b = kurtail.Context(DEV, forward_bf16=1)
    _, dRb = b.loss_grad(X, R)
    assert rel_fro(f64(dRb), dR_ref) > err
    b.close()


def test_full_batch_loss_and_gradient_against_the_oracle_on_every_row():
    # The benchmark's own configuration, nothing sampled: N = 65536 rows at d = 4096, R a few steps away from the
    # Hadamard start (so no longer exact in any 16-bit format), in the launch configuration bench.py times.  The
    # oracle takes the rows in blocks (its loss and gradient are means over tokens: the blocks combine with their
    # row counts as weights) -- about 9 TFLOP in float64 on the host cores.
    cfg = synth.config("llama2_7b_attn", device=DEV)
    X = cfg["X"]
    N, d = X.shape
    assert (N, d) == (65536, 4096)
    c = kurtail.Context(DEV)
    R = c.init_rotation(d, "hadamard")
    c.fit(X, R, 3, 1e-2)
    loss, dR = c.loss_grad(X, R)
    R64 = f64(R)
    L_ref, G_ref = 0.0, np.zeros((d, d))
    for r0 in range(0, N, 8192):
        Xb = f64(X[r0:r0 + 8192])
        l, g = ko.loss_grad(Xb, R64)
        L_ref += l * Xb.shape[0]
        G_ref += g * Xb.shape[0]
    L_ref /= N
    G_ref /= N
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    err = rel_fro(f64(dR), G_ref)
    assert err <= 1e-2, err
    assert ko.orthogonality_error(R64) <= 1e-4
    c.close()
