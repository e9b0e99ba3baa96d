"""The no-allocation loss entry point against the regular one.

kt_kurtosis_loss_noalloc serves callers that may not allocate device memory (a
process whose GPU memory is wholly owned by a pool, a plug-in with a fixed
budget, a latency-critical loop): it works out of a fixed array built into the
library instead of a caller workspace.  It launches the same kernels as
kt_kurtosis_loss does with bf16 operands (forward_bf16 = 1: the float16 copy of
X that the regular call makes for wide rows has no room in the built-in array),
so the two must agree to the last bit; the check allows the
1e-3 relative tolerance the loss carries everywhere else only as an upper bound
and asserts equality.  Two calls in a row, of different sizes, make sure the
contents the first call leaves in the shared array do not leak into the second.
This file sorts last so that a run stopping at the first failure has already
executed every other test.
"""
import math

import numpy as np
import pytest
import torch

from oracle import kurtail_oracle as ko
from paper_2503_01483_b200 import build, kurtail, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _loss_noalloc(X, R, stream=None):
    out = torch.full((1,), float("nan"), dtype=torch.float64, device=DEV)
    if stream is not None:
        stream.wait_stream(torch.cuda.current_stream())      # `out` was filled on the current stream
    kurtail.kurtosis_loss_noalloc(X, R, out, stream)
    torch.cuda.synchronize()
    return float(out.item())


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def test_noalloc_loss_matches_regular_entry_point_twice_in_a_row():
    build.build()
    ctx = kurtail.Context(DEV, forward_bf16=1)
    # (d = 128 and d = 640 carve the array for 64-column moment records, the others for 128-column ones)
    cases = [(3000, 512, "hadamard", 5), (700, 256, "identity", 6), (16384, 1024, "hadamard", 7),
             (5000, 128, "hadamard", 8), (1111, 640, "identity", 9)]
    refs, inputs = [], []
    for N, d, init, seed in cases:
        X = synth.activations(N, d, "student_t", 3.0, 4, 50.0, seed=seed, dtype=torch.bfloat16, device=DEV)
        R = ctx.init_rotation(d, init)
        inputs.append((X, R))
        refs.append(ctx.kurtosis_loss(X, R))
    before = torch.cuda.memory_allocated(DEV)
    got = [_loss_noalloc(X, R) for X, R in inputs]          # back to back, sharing the built-in array
    got_again = [_loss_noalloc(X, R) for X, R in inputs]
    for g, g2, r, (X, R) in zip(got, got_again, refs, inputs):
        assert abs(g - r) <= 1e-3 * abs(r)
        assert g == r and g2 == r
        # and against the float64 definition itself, not only against the library's other entry point
        want = ko.kurtosis_loss(_f64(X), _f64(R))
        assert abs(g - want) <= 1e-3 * abs(want)
    # only the 8-byte result tensors of the helper came from torch's allocator in between
    assert torch.cuda.memory_allocated(DEV) - before <= 4096
    ctx.close()


def test_noalloc_on_a_stream_of_the_callers():
    # the call is ordered on the stream it is given, which need not be the default one; two calls on that stream run
    # one after the other and may share the array
    build.build()
    ctx = kurtail.Context(DEV, forward_bf16=1)
    side = torch.cuda.Stream(device=DEV)
    X = synth.activations(2500, 384, "student_t", 3.0, 4, 50.0, seed=10, dtype=torch.bfloat16, device=DEV)
    R = synth.random_orthogonal(384, seed=3, device=DEV).contiguous()
    ref = ctx.kurtosis_loss(X, R)
    torch.cuda.synchronize()
    a = _loss_noalloc(X, R, side)
    b = _loss_noalloc(X, R, side)
    assert a == ref and b == ref
    want = ko.kurtosis_loss(_f64(X), _f64(R))
    assert abs(a - want) <= 1e-3 * abs(want)
    # a non-finite X is not an error of this call (it never reads the result back): the NaN is simply stored
    Xbad = X.clone()
    Xbad[17, 3] = float("nan")
    assert math.isnan(_loss_noalloc(Xbad, R, side))
    assert _loss_noalloc(X, R, side) == ref
    ctx.close()


def test_noalloc_rejects_pointers_that_are_not_device_memory():
    build.build()
    out = torch.zeros((1,), dtype=torch.float64, device=DEV)
    X = torch.zeros((128, 128), dtype=torch.bfloat16, device=DEV)
    R = torch.eye(128, dtype=torch.float32, device=DEV)
    host_out = torch.zeros((1,), dtype=torch.float64).pin_memory()
    with pytest.raises(kurtail.KtError) as e:
        kurtail.kurtosis_loss_noalloc(X, R, host_out)        # pinned host memory is not the current device's
    assert e.value.status == 1
    with pytest.raises(kurtail.KtError) as e:
        kurtail.kurtosis_loss_noalloc(X, torch.eye(128).pin_memory(), out)
    assert e.value.status == 1
    kurtail.kurtosis_loss_noalloc(X, R, out)                  # all-zero rows: every row degenerate, loss 0
    torch.cuda.synchronize()
    assert float(out.item()) == 0.0


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
