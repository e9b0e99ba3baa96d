"""kt_fit_shared: one rotation trained on shuffled minibatches of several activation buffers."""
import numpy as np
import pytest
import torch

from oracle import kurtail_oracle as ko
from paper_2503_01483_b200 import kurtail, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def f64(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def buffers(n_bufs, rows, d, dtype=torch.bfloat16, seed=200):
    return [synth.activations(rows, d, dist="student_t", nu=3.0, n_outliers=4, outlier_scale=50.0, seed=seed + b,
                              dtype=dtype, device=DEV) for b in range(n_bufs)]


def shuffle(n_samples, batch, steps, seed):
    # epochs of a seeded permutation, cut into minibatches
    rng = np.random.default_rng(seed)
    ids = []
    while len(ids) < steps * batch:
        ids.extend(rng.permutation(n_samples).tolist())
    return ids[:steps * batch]


@pytest.mark.parametrize("d,dtype", [(256, torch.bfloat16), (128, torch.bfloat16), (1024, torch.float32)])
def test_shared_fit_equals_fit_on_gathered_batches(d, dtype):
    # bit-identical to calling kt_loss_grad / kt_orth_step on minibatches gathered by the caller
    rps, spb, nb, batch, steps = 64, 5, 3, 4, 5
    c = kurtail.Context(DEV, guard_every=1)
    Xs = buffers(nb, rps * spb, d, dtype)
    order = shuffle(nb * spb, batch, steps, seed=1)
    Ra = c.init_rotation(d, "hadamard")
    Rb = Ra.clone()
    rep = c.fit_shared(Xs, rps, order, batch, Ra, steps, 1e-2, history=True)
    losses = []
    for k in range(steps):
        rows = []
        for i in order[k * batch:(k + 1) * batch]:
            b, s = divmod(i, spb)
            rows.append(Xs[b][s * rps:(s + 1) * rps])
        Xk = torch.cat(rows, 0).to(torch.bfloat16).contiguous()
        l, dR = c.loss_grad(Xk, Rb)
        losses.append(l)
        c.orth_step(Rb, dR, 1e-2)
    assert torch.equal(Ra, Rb)
    assert losses == rep["loss_history"]
    c.close()


@pytest.mark.parametrize("flat,rms,adam,dtype", [(False, False, False, torch.bfloat16),
                                                 (True, True, True, torch.bfloat16),
                                                 (True, False, False, torch.bfloat16),
                                                 (False, True, True, torch.bfloat16),
                                                 (True, True, False, torch.float32)])
def test_shared_fit_follows_the_oracle(flat, rms, adam, dtype):
    d, rps, spb, nb, batch, steps = 256, 128, 4, 3, 3, 3
    c = kurtail.Context(DEV, loss_mode=int(flat), rmsnorm=int(rms), optimizer=int(adam))
    Xs = buffers(nb, rps * spb, d, dtype)
    Xs[1] *= 4.0                                     # buffers of different scale, as layers are
    order = shuffle(nb * spb, batch, steps, seed=2)
    R0 = synth.random_orthogonal(d, seed=21, device=DEV).contiguous()
    R = R0.clone()
    rep = c.fit_shared(Xs, rps, order, batch, R, steps, 1e-2, history=True)
    # (float32 buffers are rounded to bf16 when they are gathered, as every float32 X is on entry)
    Rf, lf = ko.fit_shared([f64(x.to(torch.bfloat16)) for x in Xs], rps, order, batch, f64(R0), steps, 1e-2, flat=flat,
                           rmsnorm=rms, adam=adam, polish_thresh=1e-5)
    # free-running for three steps: the first loss is a pure parity check, the later ones inherit the steps' tolerance
    assert rep["loss_history"][0] == pytest.approx(lf[0], rel=1e-3)
    assert rep["loss_history"][-1] == pytest.approx(lf[-1], rel=5e-3)
    moved = np.linalg.norm(Rf - f64(R0))
    assert np.linalg.norm(f64(R) - Rf) <= 3e-2 * moved
    assert ko.orthogonality_error(f64(R)) <= 1e-4
    c.close()


def test_shared_fit_rejects_bad_ids_and_shapes():
    c = kurtail.Context(DEV)
    Xs = buffers(2, 256, 256)
    R = c.init_rotation(256, "identity")
    R0 = R.clone()
    with pytest.raises(kurtail.KtError) as e:
        c.fit_shared(Xs, 64, [0, 1, 8, 2], 2, R, 2, 1e-2)          # 8 samples exist: ids 0..7
    assert e.value.status == 1
    with pytest.raises(kurtail.KtError) as e:
        c.fit_shared(Xs, 100, [0, 1], 2, R, 1, 1e-2)               # 256 rows are not a multiple of 100
    assert e.value.status == 2
    with pytest.raises(kurtail.KtError) as e:
        c.fit_shared([Xs[0], Xs[1][:128]], 64, [0, 1], 2, R, 1, 1e-2)
    assert e.value.status == 2
    assert torch.equal(R, R0)
    c.close()


def test_shared_fit_many_steps_refills_the_id_chunk():
    # more steps than one chunk of ids held on the device (256): the result must not depend on the chunking
    d, rps, spb, nb, batch, steps = 128, 32, 8, 2, 2, 300
    Xs = buffers(nb, rps * spb, d)
    order = shuffle(nb * spb, batch, steps, seed=3)
    c = kurtail.Context(DEV)
    Ra = c.init_rotation(d, "identity")
    ra = c.fit_shared(Xs, rps, order, batch, Ra, steps, 1e-3, history=True)
    Rb = c.init_rotation(d, "identity")
    rb1 = c.fit_shared(Xs, rps, order[:250 * batch], batch, Rb, 250, 1e-3, history=True)
    # (a second call continues from Rb; SGD has no state, but the first and last steps of a call always measure
    # orthogonality, so compare the losses of the first 250 steps only)
    assert ra["loss_history"][:250] == rb1["loss_history"]
    assert ko.orthogonality_error(f64(Ra)) <= 1e-4
    c.close()
