"""Seeded synthetic calibration activations and rotation initialisers.

Inputs only: nothing here computes a moment, a loss, a gradient, a retraction or
a quantizer.  The same tensors are handed to the CUDA library and (copied to the
host) to the CPU checker, so neither side depends on the other's random numbers.

The shapes and value distributions stand in for the block inputs the paper
captures from Llama models on WikiText (Section 4, "Setup"): heavy-tailed
entries plus a few fixed channels that are much larger than the rest
(Section 1 and Fig. 2 describe that outlier structure).
"""
from __future__ import annotations

import math

import torch


def outlier_channels(d: int, n_out: int):
    """Evenly spread fixed channel indices j_k = k*(d/n_out) + d/(2 n_out)."""
    if n_out <= 0:
        return []
    step = d / n_out
    return [int(k * step + step / 2) for k in range(n_out)]


def _student_t(shape, nu, device):
    z = torch.randn(shape, device=device, dtype=torch.float32)
    # chi2(nu) = 2 * Gamma(nu/2, 1)
    g = torch._standard_gamma(torch.full(shape, nu / 2.0, device=device, dtype=torch.float32))
    return z / torch.sqrt((2.0 * g / nu).clamp_(min=1e-20))


def _laplace(shape, device):
    u = torch.rand(shape, device=device, dtype=torch.float32) - 0.5
    # rand() can return exactly 0, i.e. |u| = 0.5 and log(0): keep the argument of the log positive
    return -torch.sign(u) * torch.log1p(-(2.0 * u.abs()).clamp_(max=1.0 - 2.0 ** -24))


def activations(N, d, dist="student_t", nu=3.0, n_outliers=0, outlier_scale=1.0,
                seed=0, dtype=torch.bfloat16, device="cpu", chunk_rows=8192):
    """X (N x d): i.i.d. entries from `dist` ('student_t' with `nu` degrees of
    freedom, 'laplace' (0,1) or 'gauss'), then the fixed outlier channels
    multiplied by `outlier_scale`, rounded to `dtype`.  Deterministic for a
    given (seed, device type)."""
    dev = torch.device(device)
    X = torch.empty((N, d), dtype=dtype, device=dev)
    cols = outlier_channels(d, n_outliers)
    devices = [dev] if dev.type == "cuda" else []
    with torch.random.fork_rng(devices=devices):
        torch.manual_seed(seed)
        for r0 in range(0, N, chunk_rows):
            r1 = min(N, r0 + chunk_rows)
            shape = (r1 - r0, d)
            if dist == "student_t":
                blk = _student_t(shape, nu, dev)
            elif dist == "laplace":
                blk = _laplace(shape, dev)
            elif dist == "gauss":
                blk = torch.randn(shape, device=dev, dtype=torch.float32)
            else:
                raise ValueError(dist)
            if cols:
                blk[:, cols] *= outlier_scale
            X[r0:r1] = blk.to(dtype)
    return X


def kv_heads(heads, tokens, head_dim=128, outlier_scale=30.0, seed=0,
             dtype=torch.bfloat16, device="cpu"):
    """(heads*tokens) x head_dim Gaussian values; head h has two outlier dims
    (3+5h) mod head_dim and (64+11h) mod head_dim scaled by `outlier_scale`."""
    dev = torch.device(device)
    X = torch.empty((heads * tokens, head_dim), dtype=dtype, device=dev)
    devices = [dev] if dev.type == "cuda" else []
    with torch.random.fork_rng(devices=devices):
        torch.manual_seed(seed)
        for h in range(heads):
            blk = torch.randn((tokens, head_dim), device=dev, dtype=torch.float32)
            blk[:, (3 + 5 * h) % head_dim] *= outlier_scale
            blk[:, (64 + 11 * h) % head_dim] *= outlier_scale
            X[h * tokens:(h + 1) * tokens] = blk.to(dtype)
    return X


def random_orthogonal(d, seed=0, device="cpu"):
    """Q factor of a seeded Gaussian matrix (float64 QR, signs fixed so that
    diag(R) > 0), returned as float32."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    A = torch.randn((d, d), generator=g, dtype=torch.float64)
    Q, Rr = torch.linalg.qr(A)
    Q = Q * torch.sign(torch.diagonal(Rr))[None, :]
    return Q.to(torch.float32).to(device)


def config(name, device="cpu", rows=None, layers=None):
    """The benchmark workloads.  `rows` overrides N (reduced-N parity cases use
    the same d and distribution); returns a dict with X (or a list of X for the
    layer sweep), d, R-init kind, steps and lr."""
    if name == "tiny":
        N = rows or 2048
        X = activations(N, 256, "student_t", 3.0, 4, 50.0, seed=0, dtype=torch.float32, device=device)
        return dict(X=X, d=256, init="identity", steps=20, lr=1e-2)
    if name == "llama2_7b_attn":
        N = rows or 65536
        X = activations(N, 4096, "student_t", 3.0, 16, 100.0, seed=1, device=device)
        return dict(X=X, d=4096, init="hadamard", steps=100, lr=1e-2)
    if name == "kv_heads":
        tokens = (rows // 32) if rows else 65536
        X = kv_heads(32, tokens, 128, 30.0, seed=2, device=device)
        return dict(X=X, d=128, init="identity", steps=200, lr=1e-2)
    if name == "llama3_8b_down":
        N = rows or 32768
        X = activations(N, 14336, "laplace", 0.0, 64, 80.0, seed=3, device=device)
        return dict(X=X, d=14336, init="random_orthogonal", steps=50, lr=1e-2)
    if name == "llama3_70b_sweep":
        N = rows or 32768
        L = layers or 80
        Xs = [activations(N, 8192, "student_t", 2.5, 32, 200.0, seed=1000 + l, device=device) for l in range(L)]
        return dict(X=Xs, d=8192, init="hadamard", steps=50, lr=1e-2)
    if name == "llama2_7b_r1_shared":
        # stored inputs of 32 layers x 2 blocks: same outlier channels everywhere, scale growing with depth
        N = rows or 8192
        L = layers or 64
        Xs = [(activations(N, 4096, "student_t", 3.0, 16, 100.0, seed=2000 + l, device=device).float()
               * (1.0 + l / 16.0)).to(torch.bfloat16) for l in range(L)]
        return dict(X=Xs, d=4096, init="hadamard", steps=100, lr=1e-2)
    raise ValueError(name)


def is_pow2(d):
    return d > 0 and (d & (d - 1)) == 0


def sqrt_inv(d):
    return 1.0 / math.sqrt(float(d))
