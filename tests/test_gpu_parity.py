"""GPU parity: the CUDA library, called through its C ABI, against the float64
oracle on the same seeded inputs.

Tolerances (the contract): loss relative 1e-3; dR relative Frobenius 1e-2;
max|R^T R - I| <= 1e-4 after 100 steps; int4 codes bit-exact for identical
float32 Y.  Tighter, arithmetic-derived bounds are used where the two sides see
identical operands (kt_rotate: bf16 operands, float32 accumulation).
"""
import math

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


def bf16_round64(a):
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)


def make_x(N, d, seed=0, dist="student_t", nu=3.0, n_out=4, scale=50.0, dtype=torch.bfloat16):
    return synth.activations(N, d, dist, nu, n_out, scale, seed=seed, dtype=dtype, device=DEV)


def rand_orth(d, seed):
    return synth.random_orthogonal(d, seed=seed, device=DEV).contiguous()


# ------------------------------------------------------------------ the GEMM
@pytest.mark.parametrize("N,d", [(128, 128), (300, 256), (1000, 384), (2048, 256), (128 * 200 + 7, 256),
                                 (513, 1024)])
def test_rotate_matches_exact_product_of_bf16_operands(ctx, N, d):
    X = make_x(N, d, seed=N + d)
    R = rand_orth(d, seed=d).to(torch.bfloat16).float()     # bf16-exact R: both sides see the same operands
    Y = ctx.rotate(X, R)
    ref = f64(X) @ f64(R)
    scale = np.abs(f64(X)) @ np.abs(f64(R))
    err = np.abs(f64(Y) - ref)
    # float32 accumulation of d products: error <= ~ d * 2^-24 * sum|x||r| in the worst case
    assert np.all(err <= 4e-6 * scale + 1e-30), float((err / (scale + 1e-30)).max())


def test_rotate_identity_returns_x(ctx):
    X = make_x(777, 256, seed=5)
    R = ctx.init_rotation(256, "identity")
    Y = ctx.rotate(X, R)
    assert torch.equal(Y, X.float())


def test_rotate_float32_x_is_rounded_to_bf16(ctx):
    X = make_x(640, 256, seed=6, dtype=torch.float32)
    R = rand_orth(256, seed=2).to(torch.bfloat16).float()
    Y = ctx.rotate(X, R)
    ref = bf16_round64(X.cpu().numpy()) @ f64(R)
    assert np.abs(f64(Y) - ref).max() <= 4e-6 * (np.abs(f64(X)) @ np.abs(f64(R))).max()


def test_strided_x(ctx):
    big = make_x(500, 512, seed=7)
    X = big[:, :256]                      # leading dimension 512
    R = rand_orth(256, seed=3)
    assert torch.equal(ctx.rotate(X, R), ctx.rotate(X.contiguous(), R))


# ------------------------------------------------------- moments and the loss
@pytest.mark.parametrize("N,d,init", [(2048, 256, "identity"), (1000, 256, "hadamard"), (700, 1024, "orth"),
                                      (300, 128, "orth"), (1500, 384, "orth")])
def test_row_moments_and_loss(ctx, N, d, init):
    X = make_x(N, d, seed=11 + d)
    R = ctx.init_rotation(d, init) if init != "orth" else rand_orth(d, seed=4)
    mom = f64(ctx.row_moments(X, R))
    Y = ko.rotate(f64(X), f64(R))
    mu, m2, m3, m4 = ko.row_moments(Y)
    rms = np.sqrt(m2 + mu ** 2)
    assert np.all(np.abs(mom[:, 0] - mu) <= 4e-3 * rms)
    assert np.allclose(mom[:, 1], m2, rtol=4e-3)
    assert np.allclose(mom[:, 3], m4, rtol=8e-3)
    assert np.all(np.abs(mom[:, 2] - m3) <= 8e-3 * m2 ** 1.5 * np.maximum(1.0, np.abs(m3) / m2 ** 1.5))
    kap = mom[:, 3] / mom[:, 1] ** 2
    assert np.allclose(kap, ko.kurtosis_rows(Y), rtol=4e-3)
    loss = ctx.kurtosis_loss(X, R)
    ref = ko.kurtosis_loss(f64(X), f64(R))
    assert abs(loss - ref) <= 1e-3 * abs(ref)


def test_tiny_config_loss_identity(ctx):
    cfg = synth.config("tiny", device=DEV)
    X = cfg["X"]                                    # float32 2048 x 256
    R = ctx.init_rotation(256, "identity")
    loss = ctx.kurtosis_loss(X, R)
    ref = ko.kurtosis_loss(f64(X), np.eye(256))     # the oracle sees the float32 X
    assert abs(loss - ref) <= 1e-3 * abs(ref)


def test_moments_of_nearly_constant_rows(ctx):
    # rows = large constant + small noise: raw power sums would cancel catastrophically
    g = torch.Generator(device="cpu").manual_seed(3)
    base = torch.full((256, 256), 64.0) + 0.5 * torch.randn((256, 256), generator=g)
    X = base.to(torch.bfloat16).to(DEV)
    R = ctx.init_rotation(256, "identity")
    mom = f64(ctx.row_moments(X, R))
    mu, m2, m3, m4 = ko.row_moments(f64(X))
    assert np.allclose(mom[:, 0], mu, rtol=1e-6)
    assert np.allclose(mom[:, 1], m2, rtol=1e-4)
    assert np.allclose(mom[:, 3], m4, rtol=1e-4)


def test_degenerate_rows(ctx):
    d = 256
    X = make_x(256, d, seed=21)
    X[3] = 0
    X[10] = 0
    X[10, 0] = 9.0       # one-hot in channel 0 times Hadamard = constant row
    X[11] = 0
    X[11, 5] = 9.0       # one-hot elsewhere: +-a row, kappa = 1
    R = ctx.init_rotation(d, "hadamard")
    mom = f64(ctx.row_moments(X, R))
    assert mom[3, 1] == 0 and mom[10, 1] == 0
    assert mom[11, 3] / mom[11, 1] ** 2 == pytest.approx(1.0, rel=1e-5)
    assert abs(mom[11, 0]) <= 1e-6
    loss = ctx.kurtosis_loss(X, R)
    ref = ko.kurtosis_loss(f64(X), f64(R))
    assert abs(loss - ref) <= 1e-3 * abs(ref)
    _, dR = ctx.loss_grad(X, R)
    assert torch.isfinite(dR).all()


# -------------------------------------------------------------- the gradient
@pytest.mark.parametrize("N,d,init", [(2048, 256, "identity"), (1000, 256, "hadamard"), (900, 1024, "orth"),
                                      (333, 128, "orth"), (4096 + 65, 512, "hadamard")])
def test_loss_grad(ctx, N, d, init):
    X = make_x(N, d, seed=31 + d)
    R = ctx.init_rotation(d, init) if init != "orth" else rand_orth(d, seed=5)
    loss, dR = ctx.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    rel = np.linalg.norm(f64(dR) - dR_ref) / np.linalg.norm(dR_ref)
    assert rel <= 1e-2, rel
    # <R, dR> = tr(Y^T G) = 0 (kappa is scale invariant)
    ip = float((f64(R) * f64(dR)).sum())
    assert abs(ip) <= 2e-2 * float(np.abs(f64(R) * f64(dR)).sum())


@pytest.mark.parametrize("N,d,init", [(2048, 256, "identity"), (900, 1024, "orth"), (128 * 40 + 9, 384, "orth"),
                                      (333, 4096, "hadamard")])
def test_backward_from_stored_y_equals_recomputed_backward(N, d, init):
    # backward_mode 1 recomputes each Y tile in a second GEMM pass, backward_mode 2 keeps Y in float32: same bits,
    # and the recomputing path is held to the oracle like the default one
    X = make_x(N, d, seed=45)
    keep = kurtail.Context(DEV, backward_mode=2)
    reco = kurtail.Context(DEV, backward_mode=1)
    R = rand_orth(d, seed=3) if init == "orth" else keep.init_rotation(d, init)
    la, da = keep.loss_grad(X, R)
    lb, db = reco.loss_grad(X, R)
    assert la == lb and torch.equal(da, db)
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(lb - L_ref) <= 1e-3 * abs(L_ref)
    assert np.linalg.norm(f64(db) - dR_ref) <= 1e-2 * np.linalg.norm(dR_ref)
    Ra, Rb = R.clone(), R.clone()
    ra = keep.fit(X, Ra, 3, 1e-2, history=True)
    rb = reco.fit(X, Rb, 3, 1e-2, history=True)
    assert torch.equal(Ra, Rb) and ra["loss_history"] == rb["loss_history"]
    keep.close()
    reco.close()


@pytest.mark.parametrize("N,d,init,scale", [(2048, 256, "identity", 1.0), (900, 1024, "orth", 1.0),
                                            (128 * 40 + 9, 384, "orth", 2.0 ** -12), (333, 4096, "hadamard", 2.0 ** 8),
                                            (700, 640, "orth", 1.0)])
def test_backward_from_float16_y(N, d, init, scale):
    # The default keeps Y between the two passes as float16 with one power-of-two factor per row and half column
    # tile: the loss (computed from the float32 accumulators) is the recomputing mode's, the gradient differs from
    # it by the rounding of Y to 11 significant bits only, whatever the scale of X (the factor follows the data; the
    # scales here keep the fourth powers of the float32 moment sums inside float32's range),
    # and it is held to the oracle at the same tolerance.  Rows of zeros and a row with one huge entry are mixed in.
    X = (make_x(N, d, seed=47).float() * scale)
    X[5] = 0.0
    X[7] = 0.0
    X[7, 3] = 3.0e4 * scale
    X = X.to(torch.bfloat16)
    half = kurtail.Context(DEV)
    full = kurtail.Context(DEV, backward_mode=2)
    R = rand_orth(d, seed=8) if init == "orth" else half.init_rotation(d, init)
    la, da = half.loss_grad(X, R)
    lb, db = full.loss_grad(X, R)
    assert la == lb
    assert torch.isfinite(da).all()
    assert rel_fro(f64(da), f64(db)) <= 4e-3
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(la - L_ref) <= 1e-3 * abs(L_ref)
    assert rel_fro(f64(da), dR_ref) <= 1e-2
    # reruns give the same bits
    lc, dc = half.loss_grad(X, R)
    assert lc == la and torch.equal(dc, da)
    half.close()
    full.close()


@pytest.mark.parametrize("N,d", [(1000, 256), (129, 512), (128 * 40 + 9, 1024), (300, 4096)])
def test_cta_pairs_give_the_same_bits_as_single_ctas(N, d):
    # 256-wide tiles run on pairs of CTAs by default (one MMA over both SMs); the accumulation order over k is the
    # same as with one CTA per tile, so every result must be bit-identical
    X = make_x(N, d, seed=46)
    pair = kurtail.Context(DEV)
    solo = kurtail.Context(DEV, cta_pairs=0)
    R = rand_orth(d, seed=4)
    assert torch.equal(pair.rotate(X, R), solo.rotate(X, R))
    la, da = pair.loss_grad(X, R)
    lb, db = solo.loss_grad(X, R)
    assert la == lb and torch.equal(da, db)
    assert pair.quant4_error(X, R) == solo.quant4_error(X, R)
    Ra, Rb = R.clone(), R.clone()
    pair.fit(X, Ra, 3, 1e-2)
    solo.fit(X, Rb, 3, 1e-2)
    assert torch.equal(Ra, Rb)
    pair.close()
    solo.close()


def test_loss_grad_tiny_config_float32(ctx):
    cfg = synth.config("tiny", device=DEV)
    X = cfg["X"]
    R = ctx.init_rotation(256, "identity")
    loss, dR = ctx.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), np.eye(256))
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    assert np.linalg.norm(f64(dR) - dR_ref) / np.linalg.norm(dR_ref) <= 1e-2


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_float16_forward_operands_on_wide_rows(ctx, dtype):
    # d > 512: the forward GEMMs read a float16 copy of X with one power-of-two factor per row and R rounded to
    # float16.  Rows of very different scale, a row of zeros, a strided X and a float32 X all take that path; the
    # results are held to the oracle (which sees X's own values), rerun bit for bit, and are the bf16-operand path's
    # for an R that bf16 holds exactly.
    N, d = 700, 1024
    big = synth.activations(N, 2 * d, "student_t", 3.0, 8, 50.0, seed=48, dtype=torch.float32, device=DEV)
    big *= torch.logspace(-8, 8, N, base=2.0, device=DEV)[:, None]
    big[11] = 0.0
    X = big.to(dtype)[:, :d]                     # leading dimension 2 d
    R = rand_orth(d, seed=9)
    loss, dR = ctx.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    assert rel_fro(f64(dR), dR_ref) <= 1e-2
    l2, d2 = ctx.loss_grad(X.contiguous(), R)
    assert l2 == loss and torch.equal(d2, dR)
    Y = ctx.rotate(X, R)
    ref = f64(X.to(torch.bfloat16)) @ f64(R)
    assert np.abs(f64(Y) - ref).max() <= 2e-3 * np.abs(ref).max()
    Rb = R.to(torch.bfloat16).float()            # exact in bf16, and in float16 but for entries below 2^-17
    b = kurtail.Context(DEV, forward_bf16=1)
    Ya, Yb = ctx.rotate(X, Rb), b.rotate(X, Rb)
    assert np.abs(f64(Ya) - f64(Yb)).max() <= 1e-5 * np.abs(f64(Yb)).max()
    b.close()


def test_loss_grad_is_deterministic(ctx):
    X = make_x(3000, 256, seed=41)
    R = rand_orth(256, seed=6)
    l1, d1 = ctx.loss_grad(X, R)
    l2, d2 = ctx.loss_grad(X, R)
    assert l1 == l2 and torch.equal(d1, d2)


def test_low_kurtosis_rows_flip_the_sign(ctx):
    # uniform rows have kappa < 1.8 after few-channel mixing: gradient sign must follow
    g = torch.Generator(device="cpu").manual_seed(9)
    X = (torch.rand((512, 256), generator=g) * 2 - 1).to(torch.bfloat16).to(DEV)
    R = ctx.init_rotation(256, "identity")
    loss, dR = ctx.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), np.eye(256))
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    assert np.linalg.norm(f64(dR) - dR_ref) / np.linalg.norm(dR_ref) <= 1e-2


# ------------------------------------------- d = 128: the single-pass kernel
@pytest.mark.parametrize("N", [128, 333, 5000, 128 * 300 + 17])
def test_single_pass_kernel_d128(ctx, N):
    X = synth.kv_heads(1, N, 128, 30.0, seed=N, device=DEV)
    X[N // 2] = 0                                        # a degenerate row in the middle
    R = rand_orth(128, seed=12)
    loss, dR = ctx.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    assert np.linalg.norm(f64(dR) - dR_ref) / np.linalg.norm(dR_ref) <= 1e-2
    # the general three-GEMM path computes the same thing
    gen = kurtail.Context(DEV, small_d_fused=0)
    loss_g, dR_g = gen.loss_grad(X, R)
    # (the general path uses R as two bf16 terms; the single-pass kernel uses one and corrects the loss to first
    # order with its own gradient: what is left is second order in the rounding of R)
    assert abs(loss - loss_g) <= 1e-4 * abs(loss_g)
    assert np.linalg.norm(f64(dR) - f64(dR_g)) / np.linalg.norm(f64(dR_g)) <= 8e-3
    gen.close()
    # two bf16 terms of R in the single-pass kernel itself (no correction): the general path's loss to float32 noise
    two = kurtail.Context(DEV, forward_terms=2)
    loss_2, dR_2 = two.loss_grad(X, R)
    assert abs(loss_2 - loss_g) <= 1e-5 * abs(loss_g)
    assert np.linalg.norm(f64(dR_2) - dR_ref) / np.linalg.norm(dR_ref) <= 1e-2
    two.close()
    # fixed-order reductions: a second evaluation is bit-identical
    loss2, dR2 = ctx.loss_grad(X, R)
    assert loss2 == loss and torch.equal(dR2, dR)


def test_single_head_rows_meet_the_loss_tolerance(ctx):
    # every token puts its energy into the same two channels: the rounding of R is then systematic over tokens,
    # which is why R is used as a two-term bf16 split at small d (one term gives 2e-3 here)
    X = synth.kv_heads(1, 200000, 128, 30.0, seed=200000, device=DEV)
    R = rand_orth(128, seed=12)
    loss, dR = ctx.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(loss - L_ref) <= 1e-3 * abs(L_ref)
    assert np.linalg.norm(f64(dR) - dR_ref) / np.linalg.norm(dR_ref) <= 1e-2
    gen = kurtail.Context(DEV, small_d_fused=0)
    assert abs(gen.kurtosis_loss(X, R) - L_ref) <= 1e-3 * abs(L_ref)
    gen.close()


def test_single_pass_kernel_fit_kv_heads(ctx):
    cfg = synth.config("kv_heads", device=DEV, rows=32 * 1024)
    X = cfg["X"]
    R = ctx.init_rotation(128, "identity")
    L0 = ctx.kurtosis_loss(X, R)
    rep = ctx.fit(X, R, 20, cfg["lr"], history=True)
    assert rep["loss_history"][0] == pytest.approx(L0, rel=1e-6)
    assert rep["loss_history"][-1] < rep["loss_history"][0]
    assert ctx.orth_error(R) <= 1e-4
    L_ref = ko.kurtosis_loss(f64(X), f64(R))
    assert abs(ctx.kurtosis_loss(X, R) - L_ref) <= 1e-3 * abs(L_ref)


# ------------------------------------------------------------ the Cayley step
@pytest.mark.parametrize("d,lr", [(128, 1e-2), (256, 1e-2), (512, 0.5), (1024, 5.0)])
def test_orth_step_matches_stepwise_oracle(ctx, d, lr):
    X = make_x(1024, d, seed=51)
    R = rand_orth(d, seed=7)
    _, dR = ctx.loss_grad(X, R)
    R0, dR0 = f64(R), f64(dR)
    ref, alpha, wn = ko.orth_step(R0, dR0, lr, iters=2, q=0.5, eps=1e-8, polish_thresh=1e-5)
    Rn = ctx.orth_step(R.clone(), dR, lr)
    upd = np.abs(ref - R0).max()
    err = np.abs(f64(Rn) - ref).max()
    # W is used as bf16 (2^-9 relative) and the iterate as a two-term bf16 split:
    # the update is matched to ~1% of its own size, plus float32 round-off of R
    assert err <= 2e-2 * upd + 3e-7, (err, upd)
    assert ctx.orth_error(Rn) <= 1e-5


def test_orth_step_zero_gradient_keeps_r(ctx):
    d = 256
    R = rand_orth(d, seed=8)
    Rn = ctx.orth_step(R.clone(), torch.zeros_like(R), 1e-2)
    assert np.abs(f64(Rn) - f64(R)).max() <= 2e-7


def test_orth_error_measures_deviation(ctx):
    d = 256
    R = rand_orth(d, seed=9)
    assert ctx.orth_error(R) <= 3e-6          # noise floor of the two-term bf16 split at d = 256
    R2 = R.clone()
    R2[3, 7] += 1e-2
    assert ctx.orth_error(R2) == pytest.approx(ko.orthogonality_error(f64(R2)), rel=1e-3)


def test_polish_restores_orthogonality(ctx):
    d = 256
    g = torch.Generator(device="cpu").manual_seed(4)
    R = rand_orth(d, seed=10) + (1e-3 * torch.randn((d, d), generator=g)).to(DEV)
    e0 = ctx.orth_error(R)
    Rn = ctx.orth_step(R.clone(), torch.zeros_like(R), 1e-2)
    e1 = ctx.orth_error(Rn)
    # one Newton-Schulz step squares the (spectral) error; the oracle's polish is the yardstick
    want = ko.orthogonality_error(ko.polish(f64(R)))
    assert e0 > 1e-3 and e1 < 0.2 * e0
    assert e1 == pytest.approx(want, rel=0.05, abs=2e-6)
    assert np.abs(f64(Rn) - ko.polish(f64(R))).max() <= 1e-2 * np.abs(ko.polish(f64(R)) - f64(R)).max() + 3e-7


# -------------------------------------------------------------------- the fit
def test_fit_tiny_config(ctx):
    cfg = synth.config("tiny", device=DEV)
    X = cfg["X"]
    R = ctx.init_rotation(256, "identity")
    rep = ctx.fit(X, R, cfg["steps"], cfg["lr"], history=True)
    assert rep["steps_done"] == 20
    assert rep["loss_history"][-1] < rep["loss_history"][0]
    assert rep["loss_first"] == rep["loss_history"][0] and rep["loss_last"] == rep["loss_history"][-1]
    assert ctx.orth_error(R) <= 1e-4
    # teacher forcing: the loss the library reports at its own R matches the oracle at that R
    L_gpu = ctx.kurtosis_loss(X, R)
    L_ref = ko.kurtosis_loss(f64(X), f64(R))
    assert abs(L_gpu - L_ref) <= 1e-3 * abs(L_ref)


def test_fit_100_steps_stays_orthogonal_and_descends(ctx):
    X = make_x(4096, 512, seed=61, n_out=8, scale=100.0)
    R = ctx.init_rotation(512, "hadamard")
    L0 = ctx.kurtosis_loss(X, R)
    rep = ctx.fit(X, R, 100, 1e-2)
    assert ctx.orth_error(R) <= 1e-4
    assert ko.orthogonality_error(f64(R)) <= 1e-4
    assert ctx.kurtosis_loss(X, R) < L0
    assert rep["loss_first"] == pytest.approx(L0, rel=1e-12)


@pytest.mark.parametrize("d,extra", [(256, {}), (1024, {}),
                                     # one float16 term of R with the one-launch step, which leaves no float16 form
                                     (256, {"forward_terms": 1}),
                                     # a threshold every step exceeds: the polish rewrites R and all its 16-bit forms
                                     (1024, {"polish_thresh": 1e-9})])
def test_fit_equals_composed_calls(d, extra):
    # the identity holds when every step measures orthogonality (guard_every = 1), as kt_orth_step always does.
    # Inside the fit the forward pass reads the 16-bit forms of R that the previous step left behind; the composed
    # calls make them afresh from R every time.
    ctx = kurtail.Context(DEV, guard_every=1, **extra)
    X = make_x(1500, d, seed=71)
    Ra = ctx.init_rotation(d, "hadamard")
    Rb = Ra.clone()
    rep = ctx.fit(X, Ra, 4, 1e-2, history=True)
    losses = []
    for _ in range(4):
        l, dR = ctx.loss_grad(X, Rb)
        losses.append(l)
        ctx.orth_step(Rb, dR, 1e-2)
    assert torch.equal(Ra, Rb)
    assert losses == rep["loss_history"]
    ctx.close()


def test_adaptive_step_matches_forced_precision():
    # default: the device picks the number of series terms and of bf16 terms of R, and measures orthogonality only
    # when its drift bound asks; forcing everything must give the same trajectory to well within the step's tolerance
    d = 1024
    X = make_x(2048, d, seed=72, n_out=8, scale=100.0)
    auto = kurtail.Context(DEV)
    full = kurtail.Context(DEV, retract_terms=2, guard_every=1)
    Ra = auto.init_rotation(d, "hadamard")
    Rf = Ra.clone()
    R0 = Ra.clone()
    ra = auto.fit(X, Ra, 30, 1e-2, history=True)
    rf = full.fit(X, Rf, 30, 1e-2, history=True)
    moved = float((Rf - R0).norm())
    assert float((Ra - Rf).norm()) <= 2e-2 * moved
    assert ra["loss_history"][-1] == pytest.approx(rf["loss_history"][-1], rel=1e-4)
    assert auto.orth_error(Ra) <= 1e-4 and ko.orthogonality_error(f64(Ra)) <= 1e-4
    auto.close()
    full.close()


def test_fit_teacher_forced_steps(ctx):
    # each GPU step, started from the GPU's own R_k, lands where the oracle's step from R_k lands
    X = make_x(1024, 256, seed=81)
    R = ctx.init_rotation(256, "hadamard")
    for _ in range(3):
        Rk = f64(R)
        l, dR = ctx.loss_grad(X, R)
        L_ref, dR_ref = ko.loss_grad(f64(X), Rk)
        assert abs(l - L_ref) <= 1e-3 * abs(L_ref)
        ref, _, _ = ko.orth_step(Rk, dR_ref, 1e-2, polish_thresh=1e-5)
        ctx.orth_step(R, dR, 1e-2)
        # the step inherits the gradient's 1e-2 (Frobenius) tolerance, plus bf16 W
        assert np.linalg.norm(f64(R) - ref) <= 2e-2 * np.linalg.norm(ref - Rk) + 1e-7 * 256


def test_fit_layers_matches_fit(ctx):
    Xs = [make_x(640, 256, seed=90 + l) for l in range(3)]
    Ra = [ctx.init_rotation(256, "hadamard") for _ in range(3)]
    Rb = [r.clone() for r in Ra]
    reps = ctx.fit_layers(Xs, Ra, 3, 1e-2)
    for l in range(3):
        ctx.fit(Xs[l], Rb[l], 3, 1e-2)
        assert torch.equal(Ra[l], Rb[l])
        assert reps[l]["steps_done"] == 3
    # resume: skipping finished layers leaves them untouched
    Rc = [r.clone() for r in Ra]
    ctx.fit_layers(Xs, Rc, 3, 1e-2, first_layer=3)
    assert all(torch.equal(a, c) for a, c in zip(Ra, Rc))


def test_fit_host_matches_fit(ctx):
    X = make_x(512, 256, seed=95)
    Xh = X.cpu().pin_memory()
    Rh = ko.hadamard(256).astype(np.float32)
    Rh_t = torch.from_numpy(Rh.copy()).pin_memory()
    stage = torch.empty_like(X)
    Rdev = torch.empty((256, 256), dtype=torch.float32, device=DEV)
    ctx.fit_host(Xh, stage, Rh_t, Rdev, 3, 1e-2)
    Rb = torch.from_numpy(Rh.copy()).to(DEV)
    ctx.fit(X, Rb, 3, 1e-2)
    assert torch.equal(Rh_t.to(DEV), Rb)


# -------------------------------------------------------------- the quantizer
@pytest.mark.parametrize("N,d", [(64, 128), (300, 256), (50, 14336)])
def test_quant4_codes_bit_exact(ctx, N, d):
    g = torch.Generator(device="cpu").manual_seed(N)
    Y = torch.randn((N, d), generator=g) * torch.rand((N, 1), generator=g) * 10
    Y[1] = 0
    Y[2, :] = torch.arange(d) % 15 - 7.0           # exact multiples incl. ties
    Y[3, :8] = torch.tensor([7, 0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5])
    Y[3, 8:] = 0
    codes, scales = ctx.quant4_codes(Y.to(DEV))
    c_ref, s_ref = ko.quant4_codes(Y.numpy())
    assert np.array_equal(scales.cpu().numpy(), s_ref)
    assert np.array_equal(codes.cpu().numpy(), c_ref)


@pytest.mark.parametrize("N,d,init", [(1000, 256, "identity"), (1000, 256, "hadamard"), (700, 1024, "orth")])
def test_quant4_error(ctx, N, d, init):
    X = make_x(N, d, seed=101)
    R = ctx.init_rotation(d, init) if init != "orth" else rand_orth(d, seed=11)
    mse = ctx.quant4_error(X, R)
    ref = ko.quant4_error_rotated(f64(X), f64(R))
    assert abs(mse - ref) <= 2e-2 * ref
    # given the GPU's own float32 Y, the error is reproduced almost exactly
    Y = ctx.rotate(X, R)
    assert mse == pytest.approx(ko.quant4_error(Y.cpu().numpy()), rel=1e-5)


# ---------------------------------------------------------------- initialisers
def test_init_rotation(ctx):
    for d in (128, 256, 2048):
        H = ctx.init_rotation(d, "hadamard").cpu().numpy()
        assert np.array_equal(H, ko.hadamard(d).astype(np.float32))
        assert np.array_equal(ctx.init_rotation(d, "identity").cpu().numpy(), np.eye(d, dtype=np.float32))
    with pytest.raises(kurtail.KtError) as e:
        ctx.init_rotation(384, "hadamard")
    assert e.value.status == 2


# --------------------------------------------------------------- error returns
def test_argument_errors_do_no_work(ctx):
    X = make_x(256, 256, seed=111)
    R = ctx.init_rotation(256, "identity")
    with pytest.raises(kurtail.KtError) as e:
        ctx.kurtosis_loss(X[:, :200], R)              # d not a multiple of 128
    assert e.value.status == 2
    with pytest.raises(kurtail.KtError) as e:
        ctx.kurtosis_loss(X[:, 1:129], R[:128, :128].contiguous())   # base not 16-byte aligned
    assert e.value.status == 3
    small = kurtail.Context(DEV)
    with pytest.raises(kurtail.KtError) as e:
        m = kurtail.as_mat(X)
        import ctypes as C
        out = C.c_double()
        kurtail._check(kurtail.lib().kt_kurtosis_loss(small._h, m, R.data_ptr(), C.byref(out)), "kt_kurtosis_loss")
    assert e.value.status == 4                        # no workspace set
    small.close()
