"""General k-bit quantizer (kt_quant_error, kt_quant_codes) and the per-token success rate on the GPU."""
import numpy as np
import pytest
import torch

from oracle import kurtail_oracle as ko
from paper_2503_01483_b200 import kurtail, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def f64(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


@pytest.fixture(scope="module")
def ctx():
    c = kurtail.Context(DEV)
    yield c
    c.close()


SPECS = [(4, False, 1.0), (4, True, 1.0), (8, False, 1.0), (8, True, 0.9), (2, True, 1.0), (3, False, 0.98),
         (6, True, 0.5)]


@pytest.mark.parametrize("bits,asym,clip", SPECS)
@pytest.mark.parametrize("N,d", [(300, 256), (50, 14336)])
def test_quant_codes_bit_exact(ctx, N, d, bits, asym, clip):
    g = torch.Generator(device="cpu").manual_seed(N + d + bits)
    Y = (torch.randn((N, d), generator=g) * 3 + 0.7).to(DEV)
    Y[0] = 0.0                       # an all-zero row
    Y[1] = 2.5                       # a constant row
    Y[2, :] = torch.arange(d, device=DEV) % 7 - 3.0   # ties
    codes, s, b = ctx.quant_codes(Y, bits, asym, clip)
    rc, rs, rb = ko.quant_codes(Y.cpu().numpy(), bits, asym, clip)
    assert np.array_equal(s.cpu().numpy(), rs)
    assert np.array_equal(b.cpu().numpy(), rb)
    assert np.array_equal(codes.cpu().numpy(), rc)


@pytest.mark.parametrize("bits,asym,clip", SPECS)
def test_quant_error_matches_oracle(ctx, bits, asym, clip):
    N, d = 1000, 512
    X = synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=4, outlier_scale=50.0, seed=301,
                          dtype=torch.bfloat16, device=DEV)
    X = (X.float() + 0.5).to(torch.bfloat16)          # off-centre rows: the asymmetric case differs
    R = synth.random_orthogonal(d, seed=31, device=DEV).contiguous()
    got = ctx.quant_error(X, R, bits, asym, clip)
    want = ko.quant_error(ko.rotate(f64(X), f64(R)).astype(np.float32), bits, asym, clip)
    assert got == pytest.approx(want, rel=2e-2)
    if (bits, asym, clip) == (4, False, 1.0):
        assert got == ctx.quant4_error(X, R)


def test_quant_error_several_column_tiles_and_spec_errors(ctx):
    N, d = 700, 1024                                   # 4 column tiles: row range merged across tiles by atomics
    X = synth.activations(N, d, dist="laplace", nu=0.0, n_outliers=8, outlier_scale=30.0, seed=302,
                          dtype=torch.bfloat16, device=DEV)
    R = ctx.init_rotation(d, "hadamard")
    Y32 = ko.rotate(f64(X), f64(R)).astype(np.float32)
    for bits, asym, clip in ((4, True, 1.0), (4, True, 0.9), (8, True, 1.0)):
        assert ctx.quant_error(X, R, bits, asym, clip) == pytest.approx(ko.quant_error(Y32, bits, asym, clip), rel=2e-2)
    for bad in ((1, False, 1.0), (9, False, 1.0), (4, False, 0.0), (4, False, 1.5)):
        with pytest.raises(kurtail.KtError) as e:
            ctx.quant_error(X, R, *bad)
        assert e.value.status == 1


def test_quant_error_with_rmsnorm_context():
    c = kurtail.Context(DEV, rmsnorm=1)
    N, d = 900, 256
    X = synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=4, outlier_scale=50.0, seed=303,
                          dtype=torch.bfloat16, device=DEV)
    R = c.init_rotation(d, "hadamard")
    Xn = ko.rmsnorm_rows(f64(X), 1e-6)
    want = ko.quant_error(ko.rotate(Xn, f64(R)).astype(np.float32), 4, False, 1.0)
    assert c.quant4_error(X, R) == pytest.approx(want, rel=2e-2)
    c.close()


def test_rowmax_success(ctx):
    N, d = 2000, 256
    X = synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=4, outlier_scale=50.0, seed=304,
                          dtype=torch.bfloat16, device=DEV)
    H = ctx.init_rotation(d, "hadamard")
    Rr = synth.random_orthogonal(d, seed=32, device=DEV).contiguous()
    for Ra, Rb in ((H, None), (Rr, H), (H, Rr)):
        got = ctx.rowmax_success(X, Ra, Rb)
        Ya = np.abs(ko.rotate(f64(X), f64(Ra))).max(axis=1)
        Yb = np.abs(f64(X) if Rb is None else ko.rotate(f64(X), f64(Rb))).max(axis=1)
        # tokens whose two maxima are closer than the GEMM's rounding can fall either way
        close = np.abs(Ya - Yb) <= 1e-2 * np.maximum(Ya, Yb)
        lo = float(((Ya < Yb) & ~close).mean())
        hi = float(((Ya < Yb) | close).mean())
        assert lo <= got <= hi
        assert abs(got - ko.rowmax_success(f64(X), f64(Ra), None if Rb is None else f64(Rb))) <= close.mean() + 1e-12
    # outlier channels: the Hadamard rotation lowers nearly every token's maximum
    assert ctx.rowmax_success(X, H) > 0.95
    # identity against the un-rotated token: equal maxima, strict inequality, no success
    assert ctx.rowmax_success(X, ctx.init_rotation(d, "identity")) == 0.0


# ------------------------------------------------- the range as a per-row quantile of the magnitudes
def _f32(level):
    """The level as the library sees it (kt_quant_spec.clip is a float32)."""
    return float(np.float32(level))


@pytest.mark.parametrize("bits,level", [(4, 0.98), (4, 0.5), (8, 0.999), (3, 0.25), (4, 1.0)])
@pytest.mark.parametrize("N,d", [(300, 256), (64, 4096), (20, 14336), (9, 1000)])
def test_quantile_clip_codes_bit_exact(ctx, N, d, bits, level):
    # the order statistic is an exact selection on the float32 bit patterns and the interpolation is float32 on both
    # sides: scales and codes must agree bit for bit, ties, repeated magnitudes and constant rows included
    g = torch.Generator(device="cpu").manual_seed(N + d + bits)
    Y = torch.distributions.StudentT(3.0).sample((N, d)).float()
    Y = (Y * torch.rand((N, 1), generator=g) * 10).to(DEV)
    Y[0] = 0.0                                               # an all-zero row
    Y[1] = -2.5                                              # a constant row
    Y[2, :] = (torch.arange(d, device=DEV) % 7 - 3.0)        # seven magnitudes, each many times
    Y[3, : d // 2] = Y[3, 0]                                 # half of the row equal
    Y[4, 0] = 1.0e30                                         # one huge entry
    codes, s, b = ctx.quant_codes(Y, bits, False, level, clip_mode=1)
    rc, rs, rb = ko.quant_codes(Y.cpu().numpy(), bits, False, _f32(level), clip_quantile=True)
    assert np.array_equal(s.cpu().numpy(), rs)
    assert float(b.abs().max()) == 0.0
    assert np.array_equal(codes.cpu().numpy(), rc)
    if level == 1.0:                                         # the plain quantizer
        c0, s0, _ = ctx.quant_codes(Y, bits, False, 1.0)
        assert torch.equal(c0, codes) and torch.equal(s0, s)


@pytest.mark.parametrize("bits,asym,clip,mode", [(4, False, 0.98, 1), (4, False, 0.9, 1), (4, False, 1.0, 0),
                                                 (8, True, 0.9, 0)])
def test_quant_error_of_a_given_y(ctx, bits, asym, clip, mode):
    # Eq. 1 on a given Y (here the library's own X R), for both readings of "Setup"'s clipping
    N, d = 1000, 1024
    X = synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=4, outlier_scale=50.0, seed=303,
                          dtype=torch.bfloat16, device=DEV)
    R = synth.random_orthogonal(d, seed=32, device=DEV).contiguous()
    Y = ctx.rotate(X, R)
    got = ctx.quant_error_given(Y, bits, asym, clip, clip_mode=mode)
    want = ko.quant_error(Y.cpu().numpy(), bits, asym, _f32(clip), clip_quantile=bool(mode))
    assert got == pytest.approx(want, rel=1e-9)
    assert ctx.quant_error_given(Y, bits, asym, clip, clip_mode=mode) == got      # fixed-order sums
    if mode == 0:
        # the same quantity from the two GEMM passes that never store Y
        assert ctx.quant_error(X, R, bits, asym, clip) == pytest.approx(got, rel=1e-6)


def test_quantile_clip_lowers_the_4bit_error_of_heavy_tailed_tokens(ctx):
    # why "Setup" clips: on heavy-tailed rows the 0.98-quantile as range beats the maximum
    N, d = 2048, 4096
    X = synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=16, outlier_scale=100.0, seed=304,
                          dtype=torch.bfloat16, device=DEV)
    R = ctx.init_rotation(d, "hadamard")
    Y = ctx.rotate(X, R)
    plain = ctx.quant_error_given(Y, 4, False, 1.0)
    clipped = ctx.quant_error_given(Y, 4, False, 0.98, clip_mode=1)
    assert clipped < plain
    assert clipped == pytest.approx(ko.quant_error(Y.cpu().numpy(), 4, False, _f32(0.98), clip_quantile=True), rel=1e-9)


def test_quantile_clip_argument_errors(ctx):
    Y = torch.randn((8, 256), device=DEV)
    X = Y.to(torch.bfloat16)
    R = ctx.init_rotation(256, "identity")
    with pytest.raises(kurtail.KtError) as e:       # a quantile is defined for the symmetric quantizer only
        ctx.quant_codes(Y, 4, True, 0.98, clip_mode=1)
    assert e.value.status == 1
    with pytest.raises(kurtail.KtError) as e:       # the GEMM passes never hold a whole row
        ctx.quant_error(X, R, 4, False, 0.98, clip_mode=1)
    assert e.value.status == 1
    with pytest.raises(kurtail.KtError) as e:
        ctx.quant_codes(Y, 4, False, 0.98, clip_mode=2)
    assert e.value.status == 1
