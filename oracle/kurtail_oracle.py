"""Float64 CPU oracle for KurTail rotation learning (arXiv 2503.01483).

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, definitional
implementation of what the CUDA library computes, written from the paper's
equations.  It shares no code with the CUDA path and imports nothing from it.
Only the test-suite, the smoke check and the CPU-baseline leg of the benchmark
may call it.

What follows the paper, and where:

* ``row_moments`` / ``kurtosis_rows``  -- Section 2 "Kurtosis", Eq. 3:
  kappa = E[(x-mu)^4] / (E[(x-mu)^2])^2 with population (1/n) expectations,
  raw (non-excess) kurtosis, so a normal sample gives 3.
* ``kurtosis_loss``  -- Section 2, the (unnumbered) loss equation after Eq. 3:
  mean over the units of |kappa - kappa_u|, kappa_u the kurtosis of the
  uniform distribution (= 9/5).  The unit is one token (row); see the
  readings list in the design notes for why.
* ``loss_grad``  -- the derivative of that loss through Y = X R (Section 3,
  "Learning the Rotations": the rotation is the weight of a linear layer).
* ``kurtosis_loss_flat`` / ``loss_grad_flat``  -- the same loss equation read
  literally: kappa of the concatenation of all tokens' activations of the layer.
  ``rmsnorm_rows`` / ``small_network``  -- Section 3, "Learning the Rotations":
  the trained network is the linear layer followed by an RMSNorm.
  ``gather_samples`` / ``fit_shared``  -- same paragraph: one rotation trained on
  shuffled minibatches of the stored inputs of all layers and both blocks.
* ``skew_direction``, ``cayley_exact``, ``cayley_stepwise``, ``orth_step`` --
  Section 3, "Optimization in the Orthogonal Space": Cayley SGD on the
  Stiefel manifold.  The paper gives the method by citation only (Li et al.
  2020); the iteration written here is that published algorithm with zero
  momentum, specialised to a square orthogonal R.
* ``orthogonality_error`` / ``polish``  -- Section 3, "Placement of the
  Rotations": R^T = R^-1 for an orthogonal matrix.  The Newton--Schulz
  correction is a build-side guard, not in the paper.
* ``quant4_codes`` / ``quant4_error``  -- Section 2, "Uniform Quantization
  for k-bit Precision" (symmetric case, k = 4) and Eq. 1 (MSE); one scale
  per token as in Section 4 "Setup".
  ``quant_codes`` / ``quant_error``: the same paragraph for k bits, symmetric
  or asymmetric, with the clip ratio of Section 4 "Setup"; ``rowmax_success``:
  the success rate of Section 3 (per-token maxima).
* ``hadamard``  -- Section 3 (Hadamard rotations), Sylvester construction.

Parity status: every function above is pinned by tests/test_oracle_pins.py
against closed forms, invariants, finite differences, library routines or
brute force.  Cayley *Adam* (``cayley_adam_step``) is "parity unpinned" as far
as the paper goes: its constants and exact form are nowhere in the paper.  As a
restatement of the cited publication's algorithm it is pinned by its reduction
to the SGD step (first step; zero decays), by the scalar recursion followed by
hand at d = 2, and by invariants (orthogonality, tangency of the momentum).

All floating point is float64 except the quantizer, which works in float32
because the integer codes are decided in float32 on both sides.
"""
from __future__ import annotations

import numpy as np

KAPPA_UNIFORM = 9.0 / 5.0  # ((b-a)^4/80) / ((b-a)^2/12)^2
DEGENERATE_REL = 1e-6      # a row with m2 <= DEGENERATE_REL * mean(Y^2) is skipped


# --------------------------------------------------------------------------
# Eq. 3: moments and kurtosis of each row
# --------------------------------------------------------------------------
def row_moments(Y):
    """Per row of Y (N x n): mean, and the 2nd, 3rd, 4th central moments with
    population (1/n) normalisation.  Two-pass, exactly as Eq. 3 defines them."""
    Y = np.asarray(Y, dtype=np.float64)
    mu = Y.mean(axis=1)
    c = Y - mu[:, None]
    m2 = (c ** 2).mean(axis=1)
    m3 = (c ** 3).mean(axis=1)
    m4 = (c ** 4).mean(axis=1)
    return mu, m2, m3, m4


def degenerate_rows(Y):
    """Rows with no spread to speak of (constant or all-zero rows): their
    kurtosis is 0/0.  They contribute nothing to loss or gradient."""
    Y = np.asarray(Y, dtype=np.float64)
    _, m2, _, _ = row_moments(Y)
    ms = (Y ** 2).mean(axis=1)
    return (ms == 0.0) | (m2 <= DEGENERATE_REL * ms)


def kurtosis_rows(Y):
    """kappa_t = m4 / m2^2 for each row (Eq. 3).  Degenerate rows give NaN."""
    _, m2, _, m4 = row_moments(Y)
    deg = degenerate_rows(Y)
    with np.errstate(divide="ignore", invalid="ignore"):
        k = m4 / (m2 * m2)
    return np.where(deg, np.nan, k)


# --------------------------------------------------------------------------
# The kurtosis loss and its gradient
# --------------------------------------------------------------------------
def rotate(X, R):
    """Y = X R: the 'linear layer' of Section 3."""
    return np.asarray(X, dtype=np.float64) @ np.asarray(R, dtype=np.float64)


def kurtosis_loss(X, R, kappa_target=KAPPA_UNIFORM):
    """L = (1/N) sum_t |kappa(Y_t) - kappa_u|,  Y = X R.
    Degenerate rows add 0 but still count in N."""
    Y = rotate(X, R)
    k = kurtosis_rows(Y)
    terms = np.where(np.isnan(k), 0.0, np.abs(k - kappa_target))
    return float(terms.sum() / Y.shape[0])


def loss_grad(X, R, kappa_target=KAPPA_UNIFORM):
    """Returns (L, dR) with dR = dL/dR (Euclidean gradient, d x d).

    d kappa / d Y_j = 4/(n m2^2) * (c_j^3 - m3 - kappa m2 c_j),  c = Y - mu.
    (The -m3 term is the dependence of m4 on the mean; the corresponding term
    of m2 vanishes because sum c = 0.)  dL/dY_t = sgn(kappa_t - kappa_u)/N times
    that, with sgn(0) = 0; dR = X^T (dL/dY)."""
    X = np.asarray(X, dtype=np.float64)
    Y = rotate(X, R)
    N, n = Y.shape
    mu, m2, m3, m4 = row_moments(Y)
    deg = degenerate_rows(Y)
    m2s = np.where(deg, 1.0, m2)
    kappa = m4 / (m2s * m2s)
    sgn = np.where(deg, 0.0, np.sign(kappa - kappa_target))
    c = Y - mu[:, None]
    dk = (4.0 / (n * m2s * m2s))[:, None] * (c ** 3 - m3[:, None] - (kappa * m2s)[:, None] * c)
    G = (sgn / N)[:, None] * dk
    L = float((np.where(deg, 0.0, np.abs(kappa - kappa_target))).sum() / N)
    return L, X.T @ G


# --------------------------------------------------------------------------
# The loss equation of Section 2 taken literally: one kurtosis per layer over
# the concatenation of all tokens' activations; and the RMSNorm of the small
# network of Section 3, "Learning the Rotations"
# --------------------------------------------------------------------------
def rmsnorm_rows(X, rms_eps=1e-6):
    """Unit-gain RMSNorm of each row: x / sqrt(mean(x^2) + rms_eps)."""
    X = np.asarray(X, dtype=np.float64)
    return X / np.sqrt((X * X).mean(axis=1, keepdims=True) + rms_eps)


def small_network(X, R, rms_eps=1e-6):
    """The network the paper trains for R1: a linear layer (the rotation)
    followed by an RMSNorm (unit gain)."""
    return rmsnorm_rows(rotate(X, R), rms_eps)


def kurtosis_flat(Y):
    """Eq. 3 over all N*n entries of Y as one sample.  NaN when Y has no spread."""
    v = np.asarray(Y, dtype=np.float64).reshape(1, -1)
    return float(kurtosis_rows(v)[0])


def kurtosis_loss_flat(X, R, kappa_target=KAPPA_UNIFORM):
    """|kappa(concatenation over tokens of Y_t) - kappa_u|, Y = X R (one layer, L = 1)."""
    k = kurtosis_flat(rotate(X, R))
    return 0.0 if np.isnan(k) else abs(k - kappa_target)


def loss_grad_flat(X, R, kappa_target=KAPPA_UNIFORM):
    """(L, dR) of kurtosis_loss_flat: the per-row derivative of loss_grad with
    the row replaced by the whole layer (n = N*d entries, one mean, one set of
    moments): dL/dY = sgn(kappa - kappa_u) 4/(n m2^2) (c^3 - m3 - kappa m2 c)."""
    X = np.asarray(X, dtype=np.float64)
    Y = rotate(X, R)
    g = loss_dY(Y.reshape(1, -1), kappa_target).reshape(Y.shape)
    return kurtosis_loss_flat(X, R, kappa_target), X.T @ g


def loss_dY(Y, kappa_target=KAPPA_UNIFORM):
    """dL/dY alone for a given Y (used to check the elementwise backward)."""
    Y = np.asarray(Y, dtype=np.float64)
    N, n = Y.shape
    mu, m2, m3, m4 = row_moments(Y)
    deg = degenerate_rows(Y)
    m2s = np.where(deg, 1.0, m2)
    kappa = m4 / (m2s * m2s)
    sgn = np.where(deg, 0.0, np.sign(kappa - kappa_target))
    c = Y - mu[:, None]
    return (sgn / N * 4.0 / (n * m2s * m2s))[:, None] * (c ** 3 - m3[:, None] - (kappa * m2s)[:, None] * c)


# --------------------------------------------------------------------------
# Cayley SGD on the orthogonal group
# --------------------------------------------------------------------------
def skew_direction(R, dR):
    """W = (A - A^T)/2 with A = dR R^T.  For a square orthogonal R, W R is the
    projection of dR onto the tangent space at R."""
    R = np.asarray(R, dtype=np.float64)
    dR = np.asarray(dR, dtype=np.float64)
    A = dR @ R.T
    return 0.5 * (A - A.T)


def step_size(W, lr, q=0.5, eps=1e-8):
    """alpha = min(lr, 2q / (||W||_F + eps)): keeps the fixed-point iteration
    a contraction (||alpha W / 2|| <= q)."""
    return min(float(lr), 2.0 * q / (float(np.linalg.norm(W)) + eps))


def cayley_exact(R, W, alpha):
    """R+ = (I + a/2 W)^-1 (I - a/2 W) R, solved exactly (LU)."""
    d = R.shape[0]
    I = np.eye(d)
    return np.linalg.solve(I + 0.5 * alpha * W, (I - 0.5 * alpha * W) @ np.asarray(R, dtype=np.float64))


def cayley_stepwise(R, W, alpha, iters=2, start=None):
    """The same map by the fixed-point iteration the Cayley-SGD algorithm uses:
    Y0 = R - a W R;  Yi = R - a/2 W (R + Y(i-1)),  i = 1..iters.
    `start` replaces Y0 (the iteration contracts towards the Cayley transform
    from any start; the cited Cayley-Adam listing starts it from R - a M)."""
    R = np.asarray(R, dtype=np.float64)
    Y = R - alpha * (W @ R) if start is None else np.asarray(start, dtype=np.float64)
    for _ in range(iters):
        Y = R - 0.5 * alpha * (W @ (R + Y))
    return Y


def orthogonality_error(R):
    """max |R^T R - I|."""
    R = np.asarray(R, dtype=np.float64)
    return float(np.abs(R.T @ R - np.eye(R.shape[0])).max())


def polish(R):
    """One Newton--Schulz step towards the nearest orthogonal matrix:
    R <- R - R (R^T R - I)/2."""
    R = np.asarray(R, dtype=np.float64)
    E = R.T @ R - np.eye(R.shape[0])
    return R - 0.5 * (R @ E)


def orth_step(R, dR, lr, iters=2, q=0.5, eps=1e-8, polish_thresh=0.0):
    """One Cayley-SGD step followed by the orthogonality guard: the polish runs
    when max|R^T R - I| exceeds polish_thresh (a negative threshold means
    always, +inf never).  Returns (R_next, alpha, ||W||_F)."""
    W = skew_direction(R, dR)
    alpha = step_size(W, lr, q, eps)
    Rn = cayley_stepwise(R, W, alpha, iters)
    if orthogonality_error(Rn) > polish_thresh:
        Rn = polish(Rn)
    return Rn, alpha, float(np.linalg.norm(W))


def fit(X, R, steps, lr, kappa_target=KAPPA_UNIFORM, iters=2, q=0.5, eps=1e-8, polish_thresh=0.0):
    """steps x (loss_grad; orth_step).  Returns (R_final, [loss per step])."""
    R = np.asarray(R, dtype=np.float64).copy()
    losses = []
    for _ in range(steps):
        L, dR = loss_grad(X, R, kappa_target)
        losses.append(L)
        R, _, _ = orth_step(R, dR, lr, iters, q, eps, polish_thresh)
    return R, losses


def cayley_adam_step(R, dR, state, lr, beta1=0.9, beta2=0.99, adam_eps=1e-8,
                     iters=2, q=0.5, eps=1e-8, polish_thresh=0.0):
    """Cayley Adam (Section 3, "Optimization in the Orthogonal Space", names the
    optimiser only; the update is the algorithm of the publication it cites, Li
    et al. 2020, for a square orthogonal R, with the fixed-point iteration
    started from Y0 = R - alpha W R as in cayley_stepwise).
    state = dict(M=d x d, v=scalar, k=step count), updated in place.
    Pins (tests): reduction to the SGD step along G/||G|| on the first step and
    with zero decays, the scalar recursion followed by hand at d = 2, tangency
    of M and orthogonality.  What no test can pin is the paper's own choice of
    beta1, beta2, learning rate and iteration count: it prints none."""
    R = np.asarray(R, dtype=np.float64)
    dR = np.asarray(dR, dtype=np.float64)
    state["k"] += 1
    k = state["k"]
    state["M"] = beta1 * state["M"] + (1.0 - beta1) * dR
    state["v"] = beta2 * state["v"] + (1.0 - beta2) * float((dR * dR).sum())
    vhat = state["v"] / (1.0 - beta2 ** k)
    r = (1.0 - beta1 ** k) * np.sqrt(vhat + adam_eps)
    W = skew_direction(R, state["M"]) / r
    state["M"] = r * (W @ R)
    alpha = step_size(W, lr, q, eps)
    Rn = cayley_stepwise(R, W, alpha, iters)
    if orthogonality_error(Rn) > polish_thresh:
        Rn = polish(Rn)
    return Rn


# --------------------------------------------------------------------------
# Section 3, "Learning the Rotations": one rotation for the stored inputs of
# all layers and both blocks, trained on shuffled minibatches
# --------------------------------------------------------------------------
def gather_samples(X_bufs, rows_per_sample, ids):
    """The minibatch named by `ids`: sample id = buffer * samples_per_buffer +
    index within the buffer; a sample is rows_per_sample consecutive rows.  The
    samples' rows are stacked in the order of `ids`."""
    spb = X_bufs[0].shape[0] // rows_per_sample
    parts = []
    for i in ids:
        b, s = divmod(int(i), spb)
        parts.append(np.asarray(X_bufs[b], dtype=np.float64)[s * rows_per_sample:(s + 1) * rows_per_sample])
    return np.concatenate(parts, axis=0)


def fit_shared(X_bufs, rows_per_sample, order, batch, R, steps, lr, flat=False, rmsnorm=False, adam=False,
               rms_eps=1e-6, kappa_target=KAPPA_UNIFORM, polish_thresh=0.0):
    """steps x (gather the step's minibatch; [RMSNorm its rows]; loss and
    gradient, per token or over the whole minibatch; Cayley SGD or Cayley Adam
    step).  `order` holds steps*batch sample ids: the shuffle is an input.
    Returns (R_final, [loss per step])."""
    R = np.asarray(R, dtype=np.float64).copy()
    d = R.shape[0]
    state = dict(M=np.zeros((d, d)), v=0.0, k=0)
    lg = loss_grad_flat if flat else loss_grad
    losses = []
    for k in range(steps):
        Xk = gather_samples(X_bufs, rows_per_sample, order[k * batch:(k + 1) * batch])
        if rmsnorm:
            Xk = rmsnorm_rows(Xk, rms_eps)
        L, dR = lg(Xk, R, kappa_target)
        losses.append(L)
        if adam:
            R = cayley_adam_step(R, dR, state, lr, polish_thresh=polish_thresh)
        else:
            R, _, _ = orth_step(R, dR, lr, polish_thresh=polish_thresh)
    return R, losses


# --------------------------------------------------------------------------
# Symmetric 4-bit per-token quantizer (float32 decisions)
# --------------------------------------------------------------------------
def quant4_codes(Y32):
    """Per row: s = max|Y| / 7 (float32 divide); code = clamp(rint(Y / s), -7, 7)
    with a true float32 divide and ties to even.  s == 0 gives zero codes.
    Returns (codes int8 N x n, scales float32 N)."""
    Y = np.asarray(Y32, dtype=np.float32)
    amax = np.abs(Y).max(axis=1).astype(np.float32)
    s = (amax / np.float32(7.0)).astype(np.float32)
    safe = np.where(s == 0, np.float32(1.0), s).astype(np.float32)
    q = np.rint((Y / safe[:, None]).astype(np.float32))
    q = np.clip(q, -7.0, 7.0)
    q = np.where((s == 0)[:, None], 0.0, q)
    return q.astype(np.int8), s


def quant4_error(Y32):
    """Eq. 1 over all N*n entries: mean (Y - Q(Y))^2, Q(Y) = code * s formed in
    float32, the difference and the sum in float64."""
    Y = np.asarray(Y32, dtype=np.float32)
    codes, s = quant4_codes(Y)
    deq = (codes.astype(np.float32) * s[:, None]).astype(np.float32)
    diff = Y.astype(np.float64) - deq.astype(np.float64)
    return float((diff * diff).sum() / Y.size)


def row_abs_quantile(Y32, level):
    """Per row, the `level`-quantile of |y| with linear interpolation between
    order statistics: sort the n magnitudes, h = level*(n-1), lo = floor(h),
    value = a[lo] + (h - lo)*(a[lo+1] - a[lo]).  The position is taken in
    float64, the interpolation in float32.  (Section 4, "Setup": activations are
    "clipped using a quantile of 0.98", read as a per-token quantile of the
    magnitudes.)"""
    A = np.sort(np.abs(np.asarray(Y32, dtype=np.float32)), axis=1)
    n = A.shape[1]
    h = float(level) * (n - 1)
    lo = int(np.floor(h))
    hi = min(lo + 1, n - 1)
    t = np.float32(h - lo)
    a0, a1 = A[:, lo], A[:, hi]
    return (a0 + (t * (a1 - a0).astype(np.float32)).astype(np.float32)).astype(np.float32)


def quant_codes(Y32, bits=4, asymmetric=False, clip=1.0, clip_quantile=False):
    """The k-bit quantizer of Section 2, "Uniform Quantization for k-bit
    Precision", per row, in float32 throughout:
      symmetric:  b = 0, s = clip*max|y| / (2^(k-1) - 1), codes in [-(2^(k-1)-1), 2^(k-1)-1];
      asymmetric: b = clip*min(y), s = (clip*max(y) - b) / (2^k - 1), codes in [0, 2^k - 1];
      code = clamp(rint((y - b) / s), lo, hi), ties to even; s == 0 gives code 0.
    `clip` in (0, 1] shrinks the range towards zero (Section 4, "Setup" clips
    activations).  clip_quantile (symmetric only): the range is not clip*max|y|
    but the clip-quantile of the row's |y| (row_abs_quantile); larger entries
    saturate.  Returns (codes int16 N x n, s float32 N, b float32 N)."""
    Y = np.asarray(Y32, dtype=np.float32)
    c = np.float32(clip)
    if clip_quantile and asymmetric:
        raise ValueError("quantile clipping is defined for the symmetric quantizer only")
    if asymmetric:
        den = np.float32(2 ** bits - 1)
        lo, hi = np.float32(0.0), den
        b = (c * Y.min(axis=1)).astype(np.float32)
        rng = ((c * Y.max(axis=1)).astype(np.float32) - b).astype(np.float32)
    else:
        den = np.float32(2 ** (bits - 1) - 1)
        lo, hi = -den, den
        b = np.zeros(Y.shape[0], dtype=np.float32)
        rng = row_abs_quantile(Y, clip) if clip_quantile else (c * np.abs(Y).max(axis=1)).astype(np.float32)
    s = (rng / den).astype(np.float32)
    safe = np.where(s == 0, np.float32(1.0), s).astype(np.float32)
    q = np.rint(((Y - b[:, None]).astype(np.float32) / safe[:, None]).astype(np.float32))
    q = np.clip(q, lo, hi)
    q = np.where((s == 0)[:, None], 0.0, q)
    return q.astype(np.int16), s, b


def quant_error(Y32, bits=4, asymmetric=False, clip=1.0, clip_quantile=False):
    """Eq. 1 for quant_codes: mean (Y - Q(Y))^2 with Q(Y) = code*s + b formed in
    float32, the difference and the sum in float64."""
    Y = np.asarray(Y32, dtype=np.float32)
    codes, s, b = quant_codes(Y, bits, asymmetric, clip, clip_quantile)
    deq = ((codes.astype(np.float32) * s[:, None]).astype(np.float32) + b[:, None]).astype(np.float32)
    diff = Y.astype(np.float64) - deq.astype(np.float64)
    return float((diff * diff).sum() / Y.size)


def rowmax_success(X, R_a, R_b=None):
    """Section 3's success rate: the fraction of tokens whose largest magnitude
    after rotation R_a is smaller than after R_b (R_b None: the un-rotated token)."""
    X = np.asarray(X, dtype=np.float64)
    a = np.abs(rotate(X, R_a)).max(axis=1)
    b = np.abs(X if R_b is None else rotate(X, R_b)).max(axis=1)
    return float((a < b).mean())


def quant4_error_rotated(X, R):
    """quant4_error of Y = X R, the product formed in float64 then rounded to
    float32 (what an exact GEMM would hand the quantizer)."""
    return quant4_error(rotate(X, R).astype(np.float32))


# --------------------------------------------------------------------------
# Rotation initialisers
# --------------------------------------------------------------------------
def hadamard(d):
    """Normalised Sylvester Hadamard matrix H_d / sqrt(d), d a power of two,
    by the doubling H_2n = [[H, H], [H, -H]]."""
    if d < 1 or d & (d - 1):
        raise ValueError("d must be a power of two")
    H = np.ones((1, 1))
    while H.shape[0] < d:
        H = np.block([[H, H], [H, -H]])
    return H / np.sqrt(float(d))
