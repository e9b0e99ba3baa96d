"""Pins for the float64 oracle: closed forms, invariants, finite differences,
library routines and brute force -- none of them a re-typing of the oracle's own
formula.  A dropped term, a wrong sign or a transposed operand fails at least
one test here."""
import math
import os

import numpy as np
import pytest
import scipy.linalg
import scipy.stats

from oracle import kurtail_oracle as ko

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden_values():
    out = {}
    with open(os.path.join(GOLD, "kurtosis_closed_forms.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, val = line.split()[:2]
            out[name] = float(val)
    return out


GV = _golden_values()


# ---------------- kurtosis (Eq. 3) ----------------
def test_gaussian_rows_give_three():
    rng = np.random.default_rng(0)
    n = 4096
    Y = rng.standard_normal((512, n))
    k = ko.kurtosis_rows(Y)
    # E[k] = 3 (n-1)/(n+1), sd ~ sqrt(24/n)
    assert abs(k.mean() - GV["normal"] * (n - 1) / (n + 1)) < 4 * math.sqrt(24 / n / 512)
    assert np.all(np.abs(k - 3) < 6 * math.sqrt(24 / n))


def test_uniform_and_laplace_samples():
    rng = np.random.default_rng(1)
    n = 200000
    ku = ko.kurtosis_rows(rng.uniform(-2, 5, (4, n)))
    kl = ko.kurtosis_rows(rng.laplace(0.3, 1.7, (4, n)))
    assert np.allclose(ku, GV["uniform"], atol=0.02)
    assert np.allclose(kl, GV["laplace"], atol=0.35)
    assert ko.KAPPA_UNIFORM == GV["uniform"]


def test_exact_closed_forms():
    a = 3.7
    two_point = np.array([[a, -a] * 64])
    assert ko.kurtosis_rows(two_point)[0] == pytest.approx(GV["two_point"], abs=1e-14)
    ints = np.arange(256, dtype=np.float64)[None, :]
    assert ko.kurtosis_rows(ints)[0] == pytest.approx(GV["integers_0_255"], rel=1e-13)
    assert GV["integers_0_255"] == pytest.approx(3 - 1.2 * (256 ** 2 + 1) / (256 ** 2 - 1), rel=1e-15)
    onehot = np.zeros((1, 256)); onehot[0, 17] = -5.0
    assert ko.kurtosis_rows(onehot)[0] == pytest.approx(GV["one_hot_256"], rel=1e-13)


def test_matches_scipy_library_routines():
    rng = np.random.default_rng(2)
    Y = rng.standard_t(3, (64, 300)) + rng.normal(0, 3, (64, 1))
    k = ko.kurtosis_rows(Y)
    assert np.allclose(k, scipy.stats.kurtosis(Y, axis=1, fisher=False, bias=True), rtol=1e-12)
    mu, m2, m3, m4 = ko.row_moments(Y)
    assert np.allclose(mu, Y.mean(axis=1))
    for order, m in ((2, m2), (3, m3), (4, m4)):
        assert np.allclose(m, scipy.stats.moment(Y, order, axis=1), rtol=1e-12, atol=1e-12)


def test_kurtosis_invariances_and_bound():
    rng = np.random.default_rng(3)
    Y = rng.standard_t(4, (32, 128))
    k = ko.kurtosis_rows(Y)
    assert np.all(k >= 1.0)
    assert np.allclose(ko.kurtosis_rows(7.5 * Y - 11.0), k, rtol=1e-10)
    assert np.allclose(ko.kurtosis_rows(Y[:, rng.permutation(128)]), k, rtol=1e-12)
    assert np.allclose(ko.kurtosis_rows(-Y), k, rtol=1e-12)


def test_degenerate_rows_are_skipped():
    Y = np.ones((3, 16)); Y[1] = 0.0; Y[2] = np.arange(16)
    deg = ko.degenerate_rows(Y)
    assert list(deg) == [True, True, False]
    k2 = ko.kurtosis_rows(Y)[2]
    assert ko.kurtosis_loss(Y, np.eye(16)) == pytest.approx(abs(k2 - 1.8) / 3)
    _, dR = ko.loss_grad(Y, np.eye(16))
    assert np.all(np.isfinite(dR))


# ---------------- loss ----------------
def test_loss_identity_rotation_is_raw_kurtosis():
    rng = np.random.default_rng(4)
    X = rng.standard_t(3, (40, 64))
    direct = np.mean(np.abs(scipy.stats.kurtosis(X, axis=1, fisher=False) - 9 / 5))
    assert ko.kurtosis_loss(X, np.eye(64)) == pytest.approx(direct, rel=1e-12)


def test_loss_brute_force_tiny():
    rng = np.random.default_rng(5)
    X = rng.normal(size=(5, 4)); R = scipy.stats.ortho_group.rvs(4, random_state=1)
    total = 0.0
    for t in range(5):
        y = [sum(X[t, i] * R[i, j] for i in range(4)) for j in range(4)]
        mu = sum(y) / 4
        m2 = sum((v - mu) ** 2 for v in y) / 4
        m4 = sum((v - mu) ** 4 for v in y) / 4
        total += abs(m4 / m2 ** 2 - 1.8)
    assert ko.kurtosis_loss(X, R) == pytest.approx(total / 5, rel=1e-12)


def test_orthogonal_rotation_preserves_row_norms_and_mean_identity():
    rng = np.random.default_rng(6)
    X = rng.standard_t(3, (16, 32))
    R = scipy.stats.ortho_group.rvs(32, random_state=2)
    Y = ko.rotate(X, R)
    assert np.allclose((Y ** 2).sum(1), (X ** 2).sum(1), rtol=1e-12)
    mu, m2, _, _ = ko.row_moments(Y)
    assert np.allclose(m2 + mu ** 2, (X ** 2).sum(1) / 32, rtol=1e-12)
    assert np.allclose(mu, X @ R.sum(axis=1) / 32, rtol=1e-10, atol=1e-12)


def test_hadamard_flattens_one_hot_outlier():
    d = 64
    H = ko.hadamard(d)
    assert np.allclose(H.T @ H, np.eye(d), atol=1e-14)
    assert np.allclose(np.abs(H), 1 / math.sqrt(d))
    assert np.array_equal(np.sign(H), scipy.linalg.hadamard(d))
    X = np.zeros((2, d)); X[0, 5] = 9.0; X[1, 0] = 9.0
    Y = ko.rotate(X, H)
    assert np.allclose(np.abs(Y[0]), 9.0 / math.sqrt(d))        # max shrinks by sqrt(d)
    assert ko.kurtosis_rows(Y)[0] == pytest.approx(1.0, abs=1e-12)  # +-a row
    assert ko.degenerate_rows(Y)[1]                                 # channel 0 -> constant row
    # the raw one-hot row has the largest kurtosis an n-vector can have
    assert ko.kurtosis_rows(X)[0] == pytest.approx((d * d - 3 * d + 3) / (d - 1))


# ---------------- gradient ----------------
def _rows_away_from_kink(X, R, margin=1e-3):
    k = ko.kurtosis_rows(ko.rotate(X, R))
    return np.all(np.abs(k - 1.8) > margin)


@pytest.mark.parametrize("N,d,seed", [(8, 4, 0), (16, 8, 1), (32, 16, 2)])
def test_gradient_matches_central_differences(N, d, seed):
    rng = np.random.default_rng(seed)
    X = rng.standard_t(3, (N, d)) + 0.3       # non-zero mean and skew: exercises the m3 term
    R = scipy.stats.ortho_group.rvs(d, random_state=seed) + 0.01 * rng.normal(size=(d, d))
    assert _rows_away_from_kink(X, R)
    _, dR = ko.loss_grad(X, R)
    h = 1e-6
    fd = np.zeros_like(dR)
    for i in range(d):
        for j in range(d):
            Rp = R.copy(); Rp[i, j] += h
            Rm = R.copy(); Rm[i, j] -= h
            fd[i, j] = (ko.kurtosis_loss(X, Rp) - ko.kurtosis_loss(X, Rm)) / (2 * h)
    assert np.linalg.norm(dR - fd) / np.linalg.norm(fd) < 1e-6


def test_gradient_with_low_kurtosis_rows_has_negative_sign():
    # balanced rows of +-1 plus small noise have kappa < 1.8: sign flips
    rng = np.random.default_rng(7)
    base = np.array([1.0, -1.0] * 4)
    X = np.stack([rng.permutation(base) for _ in range(6)]) + 0.05 * rng.normal(size=(6, 8))
    R = np.eye(8)
    assert np.all(ko.kurtosis_rows(X) < 1.8)
    _, dR = ko.loss_grad(X, R)
    h = 1e-6
    Rp = R.copy(); Rp[2, 3] += h
    Rm = R.copy(); Rm[2, 3] -= h
    fd = (ko.kurtosis_loss(X, Rp) - ko.kurtosis_loss(X, Rm)) / (2 * h)
    assert dR[2, 3] == pytest.approx(fd, rel=1e-5)


def test_dY_is_orthogonal_to_ones_and_to_Y():
    rng = np.random.default_rng(8)
    Y = rng.standard_t(3, (20, 48)) + 0.7
    G = ko.loss_dY(Y)
    assert np.allclose(G.sum(axis=1), 0, atol=1e-14)       # kappa is shift invariant
    assert np.allclose((G * Y).sum(axis=1), 0, atol=1e-13)  # kappa is scale invariant
    # hence <R, dR> = tr(Y^T G) = 0 for any R
    X = rng.normal(size=(20, 48)); R = scipy.stats.ortho_group.rvs(48, random_state=3)
    _, dR = ko.loss_grad(X, R)
    assert abs((R * dR).sum()) < 1e-12 * np.abs(R * dR).sum() + 1e-15


# ---------------- Cayley step ----------------
def test_skew_direction_is_skew_and_tangent():
    rng = np.random.default_rng(9)
    R = scipy.stats.ortho_group.rvs(12, random_state=4)
    dR = rng.normal(size=(12, 12))
    W = ko.skew_direction(R, dR)
    assert np.array_equal(W, -W.T)
    # W R equals the projection of dR onto the tangent space {R S : S skew}
    S = 0.5 * (R.T @ dR - dR.T @ R)
    assert np.allclose(W @ R, R @ S, atol=1e-12)


def test_cayley_exact_is_orthogonal_and_matches_scipy():
    rng = np.random.default_rng(10)
    d = 16
    R = scipy.stats.ortho_group.rvs(d, random_state=5)
    W = ko.skew_direction(R, rng.normal(size=(d, d)))
    a = 0.3
    Rn = ko.cayley_exact(R, W, a)
    assert ko.orthogonality_error(Rn) < 1e-13
    assert np.sign(np.linalg.det(Rn)) == np.sign(np.linalg.det(R))
    ref = scipy.linalg.inv(np.eye(d) + a / 2 * W) @ (np.eye(d) - a / 2 * W) @ R
    assert np.allclose(Rn, ref, atol=1e-12)
    assert np.allclose(ko.cayley_exact(R, np.zeros((d, d)), a), R)
    # first order: R+ = R - a W R + O(a^2)
    small = 1e-5
    assert np.allclose(ko.cayley_exact(R, W, small), R - small * W @ R, atol=10 * small ** 2 * np.linalg.norm(W) ** 2)


def test_cayley_closed_form_rotation_angle_d2():
    th, w, a = 0.4, 1.3, 0.25
    R = np.array([[math.cos(th), -math.sin(th)], [math.sin(th), math.cos(th)]])
    W = w * np.array([[0.0, -1.0], [1.0, 0.0]])
    Rn = ko.cayley_exact(R, W, a)
    th_new = math.atan2(Rn[1, 0], Rn[0, 0])
    assert th_new - th == pytest.approx(-2 * math.atan(a * w / 2), abs=1e-13)


@pytest.mark.parametrize("iters", [0, 1, 2, 3, 4])
def test_stepwise_converges_to_exact_geometrically(iters):
    rng = np.random.default_rng(11)
    d = 10
    R = scipy.stats.ortho_group.rvs(d, random_state=6)
    W = ko.skew_direction(R, rng.normal(size=(d, d)))
    a = 0.6 / np.linalg.norm(W, 2)             # ||a W / 2||_2 = 0.3
    err = np.linalg.norm(ko.cayley_stepwise(R, W, a, iters) - ko.cayley_exact(R, W, a), 2)
    rho = 0.3
    assert err <= 2.5 * rho ** (iters + 1) * 1.0 + 1e-14
    if iters:
        prev = np.linalg.norm(ko.cayley_stepwise(R, W, a, iters - 1) - ko.cayley_exact(R, W, a), 2)
        assert err <= rho * prev * 1.0001


def test_step_size_rule_and_descent():
    rng = np.random.default_rng(12)
    W = rng.normal(size=(6, 6)); W = W - W.T
    nrm = np.linalg.norm(W)
    assert ko.step_size(W, 1e-3) == 1e-3
    assert ko.step_size(W, 1e3) == pytest.approx(1.0 / (nrm + 1e-8))
    X = rng.standard_t(3, (64, 8)); X[:, 2] *= 30
    R = scipy.stats.ortho_group.rvs(8, random_state=7)
    L0, dR = ko.loss_grad(X, R)
    Rn, alpha, _ = ko.orth_step(R, dR, 1e-3)
    assert ko.kurtosis_loss(X, Rn) < L0


def test_polish_is_quadratic_and_fit_stays_orthogonal():
    rng = np.random.default_rng(13)
    R = scipy.stats.ortho_group.rvs(12, random_state=8) + 1e-3 * rng.normal(size=(12, 12))
    e0 = ko.orthogonality_error(R)
    e1 = ko.orthogonality_error(ko.polish(R))
    assert e1 < 3 * 12 * e0 ** 2
    X = rng.standard_t(3, (128, 12)); X[:, 5] *= 40
    R0 = np.eye(12)
    Rf, losses = ko.fit(X, R0, 100, 5e-3)
    assert ko.orthogonality_error(Rf) < 1e-9
    assert losses[-1] < losses[0]


def test_cayley_adam_invariants():
    rng = np.random.default_rng(14)
    d = 8
    R = scipy.stats.ortho_group.rvs(d, random_state=9)
    st = dict(M=np.zeros((d, d)), v=0.0, k=0)
    for _ in range(5):
        Rprev = R
        R = ko.cayley_adam_step(R, rng.normal(size=(d, d)), st, 1e-2)
        assert ko.orthogonality_error(R) < 1e-6
        assert abs((st["M"] * Rprev).sum()) < 1e-12  # momentum is tangent at the old point: <W R, R> = 0


def test_cayley_adam_first_step_is_scale_free_normalised_sgd():
    # From a zero state the bias corrections cancel the decays: M = (1 - b1) G, r = (1 - b1) ||G||_F, so
    # W = skew(G R^T) / ||G||_F whatever b1, b2 and the scale of G are: the first step equals the (pinned) SGD step
    # along G / ||G||_F.  A missing bias correction, a wrong power or a misplaced square root breaks this.
    rng = np.random.default_rng(15)
    d = 10
    R = scipy.stats.ortho_group.rvs(d, random_state=10)
    G = rng.normal(size=(d, d))
    want, _, _ = ko.orth_step(R, G / np.linalg.norm(G), 3e-2, polish_thresh=0.0)
    for b1, b2, scale in [(0.9, 0.99, 1.0), (0.5, 0.999, 1e3), (0.0, 0.0, 1e-3)]:
        st = dict(M=np.zeros((d, d)), v=0.0, k=0)
        got = ko.cayley_adam_step(R, scale * G, st, 3e-2, beta1=b1, beta2=b2, adam_eps=1e-30)
        assert np.abs(got - want).max() < 1e-12
        assert st["k"] == 1 and st["v"] == pytest.approx((1 - b2) * scale ** 2 * (G * G).sum(), rel=1e-12)
        # the stored momentum is the tangent projection of (1 - b1) G: r W R = (1 - b1) skew(G R^T) R
        assert np.abs(st["M"] - (1 - b1) * scale * ko.skew_direction(R, G) @ R).max() < 1e-12 * scale


def test_cayley_adam_without_decay_is_normalised_sgd_every_step():
    # b1 = b2 = 0: no memory; each step is SGD along G / sqrt(||G||^2 + eps)
    rng = np.random.default_rng(16)
    d = 6
    R = scipy.stats.ortho_group.rvs(d, random_state=11)
    st = dict(M=rng.normal(size=(d, d)), v=123.0, k=7)  # stale state must not matter
    for _ in range(3):
        G = rng.normal(size=(d, d))
        want, _, _ = ko.orth_step(R, G / np.sqrt((G * G).sum() + 1e-8), 1e-2, polish_thresh=0.0)
        R = ko.cayley_adam_step(R, G, st, 1e-2, beta1=0.0, beta2=0.0, adam_eps=1e-8)
        assert np.abs(R - want).max() < 1e-12


def test_cayley_adam_second_moment_and_momentum_recurrences_d2():
    # d = 2: every skew matrix is w J, so the whole recursion is scalar and can be followed by hand.
    # With R_k = rotation(theta_k) and G = g_k J R_k: skew(G R_k^T) = g_k J.  The stored momentum m_{k-1} J R_{k-1} sits
    # at the previous point; seen from R_k its skew part is m_{k-1} cos(theta_k - theta_{k-1}) J (the algorithm does
    # no parallel transport), so m_k = b1 m_{k-1} cos(dtheta_{k-1}) + (1-b1) g_k; v_k = b2 v_{k-1} + (1-b2) 2 g_k^2;
    # w_k = m_k / r_k; theta moves by the angle of the s-step iterate.
    J = np.array([[0.0, -1.0], [1.0, 0.0]])
    th = 0.3
    R = np.array([[np.cos(th), -np.sin(th)], [np.sin(th), np.cos(th)]])
    b1, b2, eps_a, lr = 0.8, 0.95, 1e-12, 1e-3
    st = dict(M=np.zeros((2, 2)), v=0.0, k=0)
    m = v = dth = 0.0
    for k, g in enumerate([2.0, -1.0, 0.5], start=1):
        G = g * J @ R
        Rn = ko.cayley_adam_step(R, G, st, lr, beta1=b1, beta2=b2, adam_eps=eps_a, polish_thresh=np.inf)
        m = b1 * m * np.cos(dth) + (1 - b1) * g
        v = b2 * v + (1 - b2) * 2 * g * g
        r = (1 - b1 ** k) * np.sqrt(v / (1 - b2 ** k) + eps_a)
        w = m / r
        alpha = min(lr, 2 * 0.5 / (abs(w) * np.sqrt(2) + 1e-8))
        assert st["v"] == pytest.approx(v, rel=1e-13)
        assert np.abs(st["M"] - m * J @ R).max() < 1e-13      # r * (w J) R = m J R
        # exact Cayley rotates by -2 atan(alpha w / 2); the two-iteration form differs at order (alpha w / 2)^3
        dth = np.arctan2(Rn[1, 0], Rn[0, 0]) - np.arctan2(R[1, 0], R[0, 0])
        assert dth == pytest.approx(-2 * np.arctan(alpha * w / 2), abs=2 * abs(alpha * w / 2) ** 3 + 1e-15)
        R = Rn


def test_cayley_adam_start_of_the_fixed_point_iteration_does_not_move_its_limit():
    # The publication cited for Cayley Adam starts the fixed-point iteration from R - alpha M (M = r W R after the
    # re-projection), cayley_adam_step starts it from R - alpha W R.  The map Y -> R - alpha/2 W (R + Y) contracts with
    # factor ||alpha W / 2||_2 towards the exact Cayley transform whatever the start, so the two differ from it by
    #   (alpha ||W||_2 / 2)^s ||Y0 - Y*||:  O((alpha ||W|| / 2)^(s+1)) for R - alpha W R, and the same times |1 - r|
    # more for R - alpha M.  Checked for several s against cayley_exact.
    rng = np.random.default_rng(17)
    d = 9
    R = scipy.stats.ortho_group.rvs(d, random_state=12)
    A = rng.normal(size=(d, d))
    W = 0.5 * (A - A.T)
    W /= np.linalg.norm(W, 2)                      # ||W||_2 = 1
    alpha = 0.2
    c = alpha / 2.0                                # contraction factor
    exact = ko.cayley_exact(R, W, alpha)
    assert ko.orthogonality_error(exact) < 1e-13
    for r in (0.05, 1.0, 3.0):                     # r = (1 - beta1^k) sqrt(v_hat + eps) takes any positive value
        M = r * (W @ R)
        e_prev = None
        for s in range(0, 6):
            own = ko.cayley_stepwise(R, W, alpha, s)
            cited = ko.cayley_stepwise(R, W, alpha, s, start=R - alpha * M)
            e_own = np.linalg.norm(own - exact, 2)
            e_cit = np.linalg.norm(cited - exact, 2)
            d0_own = np.linalg.norm((R - alpha * (W @ R)) - exact, 2)
            d0_cit = np.linalg.norm((R - alpha * M) - exact, 2)
            assert e_own <= c ** s * d0_own * (1 + 1e-9) + 1e-15
            assert e_cit <= c ** s * d0_cit * (1 + 1e-9) + 1e-15
            assert d0_own <= 2.5 * c ** 1 * alpha + 1e-15          # Y0 - Y* = O(alpha^2 ||W||^2 / 2)
            if e_prev is not None:
                assert e_cit <= c * e_prev * (1 + 1e-9) + 1e-15   # geometric, whatever the start
            e_prev = e_cit
        # with the two iterations the library runs, both starts sit within (alpha/2)^2 (1 + |1 - r|) alpha of the limit
        two_own = np.linalg.norm(ko.cayley_stepwise(R, W, alpha, 2) - exact, 2)
        two_cit = np.linalg.norm(ko.cayley_stepwise(R, W, alpha, 2, start=R - alpha * M) - exact, 2)
        assert two_own <= c ** 3 * 2.5 * alpha
        assert two_cit <= c ** 2 * alpha * (abs(1 - r) + 2.5 * c)


# ---------------- flattened (whole-layer) kurtosis and the RMSNorm ----------------
def test_flat_kurtosis_library_and_closed_forms():
    rng = np.random.default_rng(21)
    Y = rng.standard_t(5, size=(37, 12)) + 0.3
    assert ko.kurtosis_flat(Y) == pytest.approx(scipy.stats.kurtosis(Y.ravel(), fisher=False, bias=True), rel=1e-12)
    # the integers 0..n-1 laid out as a matrix: 3 - 1.2 (n^2 + 1)/(n^2 - 1)
    n = 24 * 16
    assert ko.kurtosis_flat(np.arange(n, dtype=float).reshape(24, 16)) == pytest.approx(
        3 - 1.2 * (n * n + 1) / (n * n - 1), rel=1e-12)
    # one token: the layer is the row
    X = rng.normal(size=(1, 16)); R = scipy.stats.ortho_group.rvs(16, random_state=3)
    assert ko.kurtosis_loss_flat(X, R) == pytest.approx(ko.kurtosis_loss(X, R), rel=1e-13)
    # rows with different means and scales: not the mean of the rows' kurtoses
    Y2 = np.vstack([rng.normal(size=(1, 4000)), 10 + 5 * rng.normal(size=(1, 4000))])
    assert abs(ko.kurtosis_flat(Y2) - np.nanmean(ko.kurtosis_rows(Y2))) > 0.3
    assert np.isnan(ko.kurtosis_flat(np.full((3, 4), 2.5)))
    assert ko.kurtosis_loss_flat(np.zeros((4, 4)), np.eye(4)) == 0.0


def test_flat_gradient_finite_differences_and_orthogonality_to_r():
    rng = np.random.default_rng(22)
    N, d = 12, 6
    X = rng.standard_t(4, size=(N, d)); X[:, 2] *= 7
    R = scipy.stats.ortho_group.rvs(d, random_state=4) + 0.01 * rng.normal(size=(d, d))
    L, dR = ko.loss_grad_flat(X, R)
    assert L == pytest.approx(ko.kurtosis_loss_flat(X, R), rel=1e-14)
    h = 1e-6
    num = np.zeros_like(dR)
    for i in range(d):
        for j in range(d):
            E = np.zeros((d, d)); E[i, j] = h
            num[i, j] = (ko.kurtosis_loss_flat(X, R + E) - ko.kurtosis_loss_flat(X, R - E)) / (2 * h)
    assert np.abs(num - dR).max() <= 1e-6 * np.abs(dR).max()
    # kurtosis is scale and shift invariant: <Y, dL/dY> = 0 and sum dL/dY = 0, hence <R, dR> = 0
    assert abs((R * dR).sum()) <= 1e-12 * np.abs(dR).sum()
    # below the target the sign flips (uniform-ish data, kappa < 1.8 needs a two-point law)
    Xl = rng.choice([-1.0, 1.0], size=(N, d)) + 0.01 * rng.normal(size=(N, d))
    Ll, dRl = ko.loss_grad_flat(Xl, np.eye(d))
    assert ko.kurtosis_flat(Xl) < 1.8
    E = 1e-6 * rng.normal(size=(d, d))
    num = (ko.kurtosis_loss_flat(Xl, np.eye(d) + E) - ko.kurtosis_loss_flat(Xl, np.eye(d) - E)) / 2
    assert num == pytest.approx((dRl * E).sum(), rel=1e-4)


def test_rmsnorm_commutes_with_a_rotation_and_drops_out_of_the_tangent_gradient():
    rng = np.random.default_rng(23)
    N, d = 10, 8
    X = rng.standard_t(3, size=(N, d)); X[:, 1] *= 20
    R = scipy.stats.ortho_group.rvs(d, random_state=5)
    Z = ko.rmsnorm_rows(X, rms_eps=0.0)
    assert np.allclose((Z * Z).mean(axis=1), 1.0, rtol=1e-13)
    assert np.allclose(ko.rmsnorm_rows(3.7 * X, rms_eps=0.0), Z, rtol=1e-13)
    eps = 1e-6
    # orthogonal R keeps row norms: RMSNorm(X R) = RMSNorm(X) R
    assert np.abs(ko.small_network(X, R, eps) - ko.rmsnorm_rows(X, eps) @ R).max() <= 1e-13
    # Along any direction that stays on the group, R(t) = (I - t W) R with W skew, the row norms do not change to
    # first order, so the derivative of the loss of the true network (linear layer, then RMSNorm) equals the one
    # computed from the pre-normalised X with the RMSNorm left out:  d/dt = -<dR_pre, W R>.
    _, dR_pre = ko.loss_grad_flat(ko.rmsnorm_rows(X, eps), R)
    _, dR_row = ko.loss_grad(ko.rmsnorm_rows(X, eps), R)
    for seed in range(3):
        A = np.random.default_rng(seed).normal(size=(d, d))
        W = A - A.T
        t = 1e-6

        def net_loss(tt, flat):
            Y = ko.small_network(X, (np.eye(d) - tt * W) @ R, eps)
            if flat:
                return abs(ko.kurtosis_flat(Y) - ko.KAPPA_UNIFORM)
            return float(np.abs(ko.kurtosis_rows(Y) - ko.KAPPA_UNIFORM).mean())

        for flat, g in ((True, dR_pre), (False, dR_row)):
            num = (net_loss(t, flat) - net_loss(-t, flat)) / (2 * t)
            assert num == pytest.approx(-(g * (W @ R)).sum(), rel=1e-5, abs=1e-9)


# ---------------- shared rotation on shuffled minibatches ----------------
def test_fit_shared_reduces_to_fit_and_gathers_the_named_rows():
    rng = np.random.default_rng(31)
    d, rps, spb, nb = 8, 4, 3, 2
    bufs = [rng.standard_t(3, size=(rps * spb, d)) for _ in range(nb)]
    # the gather: buffer and row range of every id, in the order given
    G = ko.gather_samples(bufs, rps, [4, 0, 5])
    assert np.array_equal(G[:rps], bufs[1][rps:2 * rps])
    assert np.array_equal(G[rps:2 * rps], bufs[0][:rps])
    assert np.array_equal(G[2 * rps:], bufs[1][2 * rps:])
    R0 = scipy.stats.ortho_group.rvs(d, random_state=6)
    # one buffer, every step the whole buffer in order: the plain full-batch fit
    one = [np.concatenate(bufs, axis=0)]
    order = list(range(nb * spb)) * 5
    Ra, la = ko.fit_shared(one, rps, order, nb * spb, R0, 5, 1e-2)
    Rb, lb = ko.fit(one[0], R0, 5, 1e-2)
    assert np.array_equal(Ra, Rb) and la == lb
    # the per-token loss does not care about the order of the rows: a permuted batch gives the same step
    perm = rng.permutation(nb * spb).tolist()
    Rc, lc = ko.fit_shared(one, rps, perm, nb * spb, R0, 1, 1e-2)
    Rd, ld = ko.fit_shared(one, rps, sorted(perm), nb * spb, R0, 1, 1e-2)
    assert np.abs(Rc - Rd).max() < 1e-13 and lc[0] == pytest.approx(ld[0], rel=1e-13)
    # step k sees only its own minibatch: losses equal the loss of that batch at the R of that step
    order2 = rng.integers(0, nb * spb, size=3 * 2).tolist()
    R = R0.copy()
    Rf, lf = ko.fit_shared(bufs, rps, order2, 2, R0, 3, 1e-2, flat=True, adam=True)
    st = dict(M=np.zeros((d, d)), v=0.0, k=0)
    for k in range(3):
        Xk = ko.gather_samples(bufs, rps, order2[2 * k:2 * k + 2])
        L, dR = ko.loss_grad_flat(Xk, R)
        assert L == lf[k]
        R = ko.cayley_adam_step(R, dR, st, 1e-2)
    assert np.array_equal(R, Rf)


# ---------------- quantizer ----------------
def _golden_quant_cases():
    rows, codes = [], []
    with open(os.path.join(GOLD, "quant4_cases.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            a, b = line.split(";")
            rows.append([float(v) for v in a.split()])
            codes.append([int(float(v)) for v in b.split()])
    return np.array(rows, dtype=np.float32), np.array(codes, dtype=np.int8)


def test_quant4_golden_codes_and_ties():
    Y, want = _golden_quant_cases()
    codes, s = ko.quant4_codes(Y)
    assert np.array_equal(s, np.ones(len(Y), dtype=np.float32))
    assert np.array_equal(codes, want)


def test_quant4_exact_multiples_have_zero_error():
    rng = np.random.default_rng(15)
    q = rng.integers(-7, 8, size=(32, 64)); q[:, 0] = 7
    s = rng.uniform(0.01, 3.0, size=(32, 1)).astype(np.float32)
    Y = (q.astype(np.float32) * np.float32(0.125) * 8).astype(np.float32) * np.float32(1.0)
    Y = (q * 0.25).astype(np.float32)     # s = 7*0.25/7 = 0.25 exactly
    codes, sc = ko.quant4_codes(Y)
    assert np.array_equal(codes, q)
    assert np.all(sc == np.float32(0.25))
    assert ko.quant4_error(Y) == 0.0


def test_quant4_range_max_and_zero_row():
    rng = np.random.default_rng(16)
    Y = rng.standard_t(3, (64, 128)).astype(np.float32)
    Y[5] = 0
    codes, s = ko.quant4_codes(Y)
    assert codes.min() >= -7 and codes.max() <= 7
    am = np.abs(Y).argmax(axis=1)
    assert np.all(np.abs(codes[np.arange(64), am])[np.arange(64) != 5] == 7)
    assert s[5] == 0 and np.all(codes[5] == 0)
    # reconstruction error is at most half a step everywhere
    err = np.abs(Y - codes.astype(np.float32) * s[:, None])
    assert np.all(err <= 0.5 * s[:, None] * (1 + 1e-5))


def test_quant4_uniform_rows_give_step_squared_over_twelve():
    rng = np.random.default_rng(17)
    Y = rng.uniform(-1, 1, (256, 4096)).astype(np.float32)
    s = 1.0 / 7
    # rounding error is uniform on (-s/2, s/2) except in the clipped half-bins at the ends
    assert ko.quant4_error(Y) == pytest.approx(s * s / 12, rel=0.02)


def test_quant4_error_rotated_uses_the_product():
    rng = np.random.default_rng(18)
    X = rng.standard_t(3, (32, 16)); X[:, 3] *= 50
    H = ko.hadamard(16)
    assert ko.quant4_error_rotated(X, np.eye(16)) == pytest.approx(ko.quant4_error(X.astype(np.float32)))
    # a one-hot row becomes +-a/sqrt(d) everywhere: every entry sits on the +-7 level
    E1 = np.zeros((4, 16)); E1[np.arange(4), [1, 5, 9, 14]] = [3.0, -2.0, 8.0, 0.5]
    assert ko.quant4_error_rotated(E1, H) < 1e-12
    # a transposed operand would change this: column scaling vs row scaling
    A = rng.normal(size=(16, 16))
    assert ko.quant4_error_rotated(X, A) == pytest.approx(ko.quant4_error((X @ A).astype(np.float32)))
    assert ko.quant4_error_rotated(X, A) != pytest.approx(ko.quant4_error((X @ A.T).astype(np.float32)))


# ---------------- general k-bit quantizer and the success rate ----------------
def test_quant_general_reduces_to_the_4bit_case_and_hits_the_grid():
    rng = np.random.default_rng(41)
    Y = rng.normal(size=(20, 64)).astype(np.float32)
    c4, s4 = ko.quant4_codes(Y)
    c, s, b = ko.quant_codes(Y, 4, False, 1.0)
    assert np.array_equal(c, c4) and np.array_equal(s, s4) and not b.any()
    assert ko.quant_error(Y, 4, False, 1.0) == ko.quant4_error(Y)
    for bits in (2, 3, 8):
        # asymmetric: a row that already sits on the grid b + i*s is reproduced exactly, with codes i
        lv = 2 ** bits
        i = rng.integers(0, lv, size=(6, 40)); i[:, 0] = 0; i[:, 1] = lv - 1
        step, shift = np.float32(0.25), np.float32(-3.0)
        G = (shift + i.astype(np.float32) * step).astype(np.float32)
        c, s, b = ko.quant_codes(G, bits, True, 1.0)
        assert np.array_equal(c, i) and np.all(s == step) and np.all(b == shift)
        assert ko.quant_error(G, bits, True, 1.0) == 0.0
        # symmetric: integer multiples of max/L
        L = 2 ** (bits - 1) - 1
        k = rng.integers(-L, L + 1, size=(6, 40)); k[:, 0] = L
        S = (k * np.float32(0.5)).astype(np.float32)
        c, s, b = ko.quant_codes(S, bits, False, 1.0)
        assert np.array_equal(c, k) and ko.quant_error(S, bits, False, 1.0) == 0.0


def test_quant_uniform_rows_give_step_squared_over_twelve_and_clip_saturates():
    rng = np.random.default_rng(42)
    Y = rng.uniform(-1, 1, size=(64, 4096)).astype(np.float32)
    for bits, asym in ((4, False), (4, True), (6, True), (8, False)):
        _, s, _ = ko.quant_codes(Y, bits, asym, 1.0)
        assert ko.quant_error(Y, bits, asym, 1.0) == pytest.approx(float((s.astype(np.float64) ** 2).mean()) / 12,
                                                                   rel=0.03)
    # the asymmetric grid has 2^k - 1 steps over the range, the symmetric one 2^k - 2: the asymmetric step is smaller
    assert ko.quant_error(Y, 4, True) < ko.quant_error(Y, 4, False)
    # shifted rows: the asymmetric quantizer does not care, the symmetric one wastes its range
    assert ko.quant_error(Y + 5, 4, True) == pytest.approx(ko.quant_error(Y, 4, True), rel=0.05)
    assert ko.quant_error(Y + 5, 4, False) > 5 * ko.quant_error(Y, 4, False)
    # clip: values beyond clip*max saturate at the last level
    row = np.array([[1.0, -1.0, 0.5, 0.25, 0.0, -0.125, 0.8, 0.6]], dtype=np.float32)
    c, s, b = ko.quant_codes(row, 4, False, 0.5)
    assert s[0] == np.float32(0.5 / 7) and c[0, 0] == 7 and c[0, 1] == -7 and c[0, 6] == 7 and c[0, 2] == 7
    assert c[0, 3] == np.rint(np.float32(0.25) / s[0])
    c, s, b = ko.quant_codes(row, 4, True, 0.5)
    assert b[0] == np.float32(-0.5) and s[0] == np.float32(1.0) / np.float32(15.0) and c[0, 0] == 15 and c[0, 1] == 0
    # a heavy tail: clipping at 0.9 of the maximum lowers the error of a Gaussian row with one large outlier
    Z = rng.normal(size=(32, 1024)).astype(np.float32); Z[:, 3] = 12.0
    assert ko.quant_error(Z, 4, False, 0.5) < ko.quant_error(Z, 4, False, 1.0)
    # constant rows: step 0, codes 0, exact when unclipped
    cst = np.full((2, 8), 3.0, dtype=np.float32)
    assert ko.quant_error(cst, 4, True, 1.0) == 0.0 and not ko.quant_codes(cst, 4, True, 1.0)[0].any()


def test_rowmax_success_rate():
    d = 64
    H = ko.hadamard(d)
    # one-hot tokens (channel != 0): the Hadamard rotation spreads them, max drops from a to a/sqrt(d): success 1
    X = np.zeros((10, d)); X[np.arange(10), 1 + np.arange(10)] = 3.0
    assert ko.rowmax_success(X, H) == 1.0
    assert ko.rowmax_success(X, np.eye(d)) == 0.0           # strict inequality: equal maxima are no success
    assert ko.rowmax_success(X, np.eye(d), H) == 0.0 and ko.rowmax_success(X, H, np.eye(d)) == 1.0
    # constant tokens are concentrated by the Hadamard rotation (all mass to channel 0): success 0
    assert ko.rowmax_success(np.ones((4, d)), H) == 0.0
    # a mix: exactly the one-hot half succeeds
    assert ko.rowmax_success(np.vstack([X, np.ones((10, d))]), H) == 0.5


# ---------------- quantile clipping of the symmetric quantizer ----------------
def _golden_quantile_cases():
    cases = []
    with open(os.path.join(GOLD, "quant_quantile_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bits, level, vals, rng, codes = [p.strip() for p in line.split(";")]
            cases.append((int(bits), float(level), np.array(vals.split(), dtype=np.float32)[None, :], float(rng),
                          np.array(codes.split(), dtype=np.int16)))
    return cases


def test_quantile_clip_golden_rows():
    cases = _golden_quantile_cases()
    assert len(cases) == 5
    for bits, level, Y, rng, want in cases:
        assert float(ko.row_abs_quantile(Y, level)[0]) == pytest.approx(rng, rel=1e-6)
        codes, s, b = ko.quant_codes(Y, bits, False, level, clip_quantile=True)
        assert np.array_equal(codes[0], want), (level, codes[0], want)
        assert s[0] == pytest.approx(rng / (2 ** (bits - 1) - 1), rel=1e-6) and b[0] == 0.0


def test_row_abs_quantile_is_the_library_quantile_of_the_magnitudes():
    # the written-out rule against numpy's routine (method "linear"), on ragged sizes, with ties and with signs
    rng = np.random.default_rng(3)
    for n in (2, 5, 128, 1000, 4097):
        Y = rng.standard_t(3, size=(7, n)).astype(np.float32)
        Y[1, : n // 2] = Y[1, 0]                        # many equal magnitudes
        Y[2] = -np.abs(Y[2])
        for level in (0.0, 0.25, 0.5, 0.9, 0.98, 0.999, 1.0):
            got = ko.row_abs_quantile(Y, level)
            want = np.quantile(np.abs(Y).astype(np.float64), level, axis=1, method="linear")
            assert np.allclose(got, want, rtol=2e-6, atol=0.0), (n, level)
    # level 1 is the maximum exactly, level 0 the smallest magnitude exactly; monotone in the level
    Y = rng.standard_normal((4, 333)).astype(np.float32)
    assert np.array_equal(ko.row_abs_quantile(Y, 1.0), np.abs(Y).max(axis=1))
    assert np.array_equal(ko.row_abs_quantile(Y, 0.0), np.abs(Y).min(axis=1))
    qs = np.stack([ko.row_abs_quantile(Y, q) for q in np.linspace(0, 1, 21)])
    assert np.all(np.diff(qs, axis=0) >= 0)


def test_quantile_clip_saturates_the_expected_share_and_reduces_to_no_clipping():
    rng = np.random.default_rng(4)
    Y = rng.standard_t(3, size=(64, 4096)).astype(np.float32)
    # level 1: the plain quantizer, bit for bit
    c1, s1, _ = ko.quant_codes(Y, 4, False, 1.0, clip_quantile=True)
    c0, s0, _ = ko.quant_codes(Y, 4, False, 1.0)
    assert np.array_equal(c1, c0) and np.array_equal(s1, s0)
    assert ko.quant_error(Y, 4, False, 1.0, clip_quantile=True) == ko.quant_error(Y, 4, False, 1.0)
    # level 0.98: about 2 % of every row lies beyond the range and saturates at the largest code
    c, s, _ = ko.quant_codes(Y, 4, False, 0.98, clip_quantile=True)
    beyond = (np.abs(Y) > (7.0 * s)[:, None]).mean()
    assert beyond == pytest.approx(0.02, abs=5e-4)
    assert np.all(np.abs(c[np.abs(Y) > (7.0 * s)[:, None]]) == 7)
    # on heavy-tailed rows clipping at the quantile lowers the 4-bit error (the reason "Setup" gives for it)
    assert ko.quant_error(Y, 4, False, 0.98, clip_quantile=True) < ko.quant_error(Y, 4, False, 1.0)
    # not defined for the asymmetric quantizer
    with pytest.raises(ValueError):
        ko.quant_codes(Y, 4, True, 0.98, clip_quantile=True)
