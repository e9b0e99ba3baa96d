"""The no-allocation loss entry point against the regular one.

kt_kurtosis_loss_noalloc serves callers that may not allocate device memory (a
process whose GPU memory is wholly owned by a pool, a plug-in with a fixed
budget, a latency-critical loop): it works out of a fixed array built into the
library instead of a caller workspace.  It launches the same kernels as
kt_kurtosis_loss, so the two must agree to the last bit; the check allows the
1e-3 relative tolerance the loss carries everywhere else only as an upper bound
and asserts equality.  Two calls in a row, of different sizes, make sure the
contents the first call leaves in the shared array do not leak into the second.
This file sorts last so that a run stopping at the first failure has already
executed every other test.
"""
import pytest
import torch

from paper_2503_01483_b200 import build, kurtail, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _loss_noalloc(X, R):
    out = torch.full((1,), float("nan"), dtype=torch.float64, device=DEV)
    kurtail.kurtosis_loss_noalloc(X, R, out)
    torch.cuda.synchronize()
    return float(out.item())


def test_noalloc_loss_matches_regular_entry_point_twice_in_a_row():
    build.build()
    ctx = kurtail.Context(DEV)
    cases = [(3000, 512, "hadamard", 5), (700, 256, "identity", 6), (16384, 1024, "hadamard", 7)]
    refs, inputs = [], []
    for N, d, init, seed in cases:
        X = synth.activations(N, d, "student_t", 3.0, 4, 50.0, seed=seed, dtype=torch.bfloat16, device=DEV)
        R = ctx.init_rotation(d, init)
        inputs.append((X, R))
        refs.append(ctx.kurtosis_loss(X, R))
    before = torch.cuda.memory_allocated(DEV)
    got = [_loss_noalloc(X, R) for X, R in inputs]          # back to back, sharing the built-in array
    got_again = [_loss_noalloc(X, R) for X, R in inputs]
    for g, g2, r in zip(got, got_again, refs):
        assert abs(g - r) <= 1e-3 * abs(r)
        assert g == r and g2 == r
    # only the 8-byte result tensors of the helper came from torch's allocator in between
    assert torch.cuda.memory_allocated(DEV) - before <= 4096
    ctx.close()


def test_noalloc_rejects_what_does_not_fit():
    build.build()
    out = torch.zeros((1,), dtype=torch.float64, device=DEV)
    R = torch.eye(2048, dtype=torch.float32, device=DEV)
    X = torch.zeros((128, 2048), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(kurtail.KtError) as e:
        kurtail.kurtosis_loss_noalloc(X, R, out)            # d above the maximum
    assert e.value.status == 9
    X = torch.zeros((16385, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(kurtail.KtError) as e:
        kurtail.kurtosis_loss_noalloc(X, R[:128, :128].contiguous(), out)   # N above the maximum
    assert e.value.status == 9
    with pytest.raises(kurtail.KtError) as e:
        kurtail.kurtosis_loss_noalloc(X[:128].float(), R[:128, :128].contiguous(), out)  # float32 X
    assert e.value.status == 1
    assert kurtail.lib().kt_status_string(9).startswith(b"problem exceeds")
