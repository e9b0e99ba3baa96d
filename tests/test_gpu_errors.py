"""Error returns of the library on a GPU, and the sharded fit's hook, without ever faulting the device.

  * NaN or Inf in X gives KT_ERR_NONFINITE from every call that returns a loss, with the outputs written;
  * a bounded device-side wait that runs out (a test kernel waits on a barrier that nothing signals, for a few
    milliseconds, through the same wait every kernel uses) makes the next synchronising call return
    KT_ERR_TIMEOUT, after which the context works as before;
  * kt_fit_sharded with no hook, or with a hook that adds nothing, is kt_fit bit for bit, and with a hook that adds
    a second shard's contributions it takes the step of the whole batch.
"""
import numpy as np
import pytest
import torch

from oracle import kurtail_oracle as ko
from paper_2503_01483_b200 import build, dist_util, kurtail, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def make_x(N, d, seed, dtype=torch.bfloat16):
    return synth.activations(N, d, dist="student_t", nu=3.0, n_outliers=4, outlier_scale=50.0, seed=seed, dtype=dtype,
                             device=DEV)


@pytest.fixture(scope="module")
def ctx():
    build.build()
    c = kurtail.Context(DEV)
    yield c
    c.close()


# --------------------------------------------------------------- non-finite X
@pytest.mark.parametrize("d", [128, 256, 1024])
@pytest.mark.parametrize("bad", [float("nan"), float("inf"), float("-inf")])
def test_nonfinite_x_is_reported_by_every_call_that_returns_a_loss(ctx, d, bad):
    X = make_x(700, d, seed=401)
    X[333, 5] = bad
    R = ctx.init_rotation(d, "hadamard")
    for call in (lambda: ctx.kurtosis_loss(X, R), lambda: ctx.loss_grad(X, R), lambda: ctx.quant4_error(X, R),
                 lambda: ctx.fit(X, R.clone(), 2, 1e-2)):
        with pytest.raises(kurtail.KtError) as e:
            call()
        assert e.value.status == 7
    # outputs are written all the same: dR comes back (not the fill value), poisoned by the bad row
    dR = torch.full((d, d), 7.0, dtype=torch.float32, device=DEV)
    with pytest.raises(kurtail.KtError):
        ctx.loss_grad(X, R, dR=dR)
    assert not bool((dR == 7.0).all()) and not bool(torch.isfinite(dR).all())
    # the stream-ordered form (no loss asked for) enqueues and returns ok
    ctx.loss_grad(X, R, want_loss=False)
    torch.cuda.synchronize()
    # and the context is as good as new for finite data
    X[333, 5] = 1.0
    L = ctx.kurtosis_loss(X, R)
    assert L == pytest.approx(ko.kurtosis_loss(f64(X), f64(R)), rel=1e-3)


def test_nonfinite_float32_x(ctx):
    X = make_x(300, 256, seed=402, dtype=torch.float32)
    X[7, 100] = float("nan")
    R = ctx.init_rotation(256, "identity")
    with pytest.raises(kurtail.KtError) as e:
        ctx.kurtosis_loss(X, R)
    assert e.value.status == 7


# ------------------------------------------------------- a wait that runs out
def test_bounded_wait_runs_out_and_the_context_recovers(ctx):
    X = make_x(512, 256, seed=403)
    R = ctx.init_rotation(256, "hadamard")
    L0 = ctx.kurtosis_loss(X, R)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    ctx.test_wait_timeout(5)                    # a 5 ms wait on a barrier nobody arrives on
    t1.record()
    with pytest.raises(kurtail.KtError) as e:   # the next synchronising call reports it ...
        ctx.kurtosis_loss(X, R)
    assert e.value.status == 8
    assert 4.0 <= t0.elapsed_time(t1) <= 500.0  # the kernel gave up after its limit and returned
    assert ctx.kurtosis_loss(X, R) == L0        # ... and the one after that works, same bits as before
    # the same through a fit: the record is reported once, the fit's work itself is intact
    ctx.test_wait_timeout(2)
    Ra = R.clone()
    with pytest.raises(kurtail.KtError) as e:
        ctx.fit(X, Ra, 2, 1e-2)
    assert e.value.status == 8
    Rb = R.clone()
    ctx.fit(X, Rb, 2, 1e-2)
    assert torch.equal(Ra, Rb)
    with pytest.raises(kurtail.KtError) as e:
        ctx.test_wait_timeout(0)
    assert e.value.status == 1


def test_short_wait_limit_still_lets_real_kernels_finish():
    # wait_limit_ms is a bound, not a pace: with 50 ms every legitimate wait of these launches still ends in time
    c = kurtail.Context(DEV, wait_limit_ms=50)
    X = make_x(4096, 1024, seed=404)
    R = c.init_rotation(1024, "hadamard")
    l, dR = c.loss_grad(X, R)
    L_ref, dR_ref = ko.loss_grad(f64(X), f64(R))
    assert abs(l - L_ref) <= 1e-3 * abs(L_ref)
    assert np.linalg.norm(f64(dR) - dR_ref) <= 1e-2 * np.linalg.norm(dR_ref)
    c.close()


# ------------------------------------------------------------- the sharded fit
@pytest.mark.parametrize("d,kw", [(256, {}), (1024, {}), (128, {}), (1024, dict(optimizer=1)),
                                  (512, dict(loss_mode=1, rmsnorm=1))])
def test_sharded_fit_with_one_shard_is_the_plain_fit(d, kw):
    c = kurtail.Context(DEV, **kw)
    X = make_x(1500, d, seed=405)
    Ra = c.init_rotation(d, "hadamard")
    Rb, Rc = Ra.clone(), Ra.clone()
    ra = c.fit(X, Ra, 4, 1e-2, history=True)
    rb = c.fit_sharded(X, Rb, X.shape[0], None, 4, 1e-2, history=True)
    calls = []

    def nothing_to_add(ptr, count, dtype, stream):
        calls.append((count, dtype))
        return 0

    rc = c.fit_sharded(X, Rc, X.shape[0], nothing_to_add, 4, 1e-2, history=True)
    assert torch.equal(Ra, Rb) and ra["loss_history"] == rb["loss_history"]
    assert torch.equal(Ra, Rc) and ra["loss_history"] == rc["loss_history"]
    per_step = [(1, 2), (3, 2), (d * d, 1)] if kw.get("loss_mode") else [(1, 2), (d * d, 1)]
    if d == 128:
        per_step = [(1, 2), (d * d, 1)]
    assert calls == per_step * 4
    c.close()


@pytest.mark.parametrize("d,kw", [(256, {}), (1024, {}), (128, {}), (512, dict(loss_mode=1)),
                                  (512, dict(loss_mode=1, rmsnorm=1)), (1024, dict(optimizer=1))])
def test_sharded_fit_takes_the_step_of_the_whole_batch(d, kw):
    # two shards of unequal size on one GPU, one after the other: shard B's fit records what it hands to the hook,
    # shard A's hook adds those records -- what an all-reduce would have delivered -- and A's R must land where the
    # oracle's full-batch step lands.  (Nothing here waits on another kernel.)
    c = kurtail.Context(DEV, **kw)
    X = make_x(1200, d, seed=406)
    X[::3] *= 3.0
    XA, XB = X[:500].contiguous(), X[500:].contiguous()
    N = X.shape[0]
    R0 = synth.random_orthogonal(d, seed=19, device=DEV).contiguous()
    flat, rms, adam = bool(kw.get("loss_mode")), bool(kw.get("rmsnorm")), bool(kw.get("optimizer"))

    # what the other shard contributes to each reduction of the first step: its own partial sums.  For the
    # whole-layer loss the later partial sums depend on the earlier reduced ones, so B needs A's too: run the pair
    # twice, each pass feeding the other's records of the pass before (the first reduction, the mean, needs none).
    def run(Xl, theirs, record):
        i = [0]

        def hook(ptr, count, dtype, stream):
            t = torch.as_tensor(dist_util._DeviceBuffer(ptr, count, "<f4" if dtype == 1 else "<f8"), device=DEV)
            record.append(t.clone())
            if i[0] < len(theirs):
                t += theirs[i[0]]
            i[0] += 1
            return 0

        R = R0.clone()
        rep = c.fit_sharded(Xl, R, N, hook, 1, 1e-2, history=True)
        return R, rep

    recA, recB = [], []
    passes = 3 if flat else 1
    for _ in range(passes):
        newA, newB = [], []
        run(XA, recB, newA)
        run(XB, recA, newB)
        recA, recB = newA, newB
    RA, repA = run(XA, recB, [])
    RB, repB = run(XB, recA, [])
    assert torch.equal(RA, RB) or np.abs(f64(RA) - f64(RB)).max() <= 1e-6       # a + b vs b + a in float32
    Xin = f64(X)
    if rms:
        Xin = ko.rmsnorm_rows(Xin, 1e-6)
    L_ref, dR_ref = (ko.loss_grad_flat if flat else ko.loss_grad)(Xin, f64(R0))
    assert repA["loss_history"][0] == pytest.approx(L_ref, rel=1e-3)
    assert repB["loss_history"][0] == pytest.approx(L_ref, rel=1e-3)
    if adam:
        st = dict(M=np.zeros((d, d)), v=0.0, k=0)
        ref = ko.cayley_adam_step(f64(R0), dR_ref, st, 1e-2, polish_thresh=1e-5)
    else:
        ref, _, _ = ko.orth_step(f64(R0), dR_ref, 1e-2, polish_thresh=1e-5)
    moved = np.linalg.norm(ref - f64(R0))
    assert np.linalg.norm(f64(RA) - ref) <= 3e-2 * moved + 2.0 ** -23 * np.linalg.norm(ref)
    c.close()


def test_failing_hook_ends_the_fit_with_its_own_status(ctx):
    X = make_x(512, 256, seed=407)
    R = ctx.init_rotation(256, "hadamard")
    with pytest.raises(kurtail.KtError) as e:
        ctx.fit_sharded(X, R, 512, lambda *a: 1, 2, 1e-2)
    assert e.value.status == 11
    torch.cuda.synchronize()
    with pytest.raises(kurtail.KtError) as e:
        ctx.fit_sharded(X, R, 100, None, 2, 1e-2)          # fewer rows in total than this shard holds
    assert e.value.status == 1
