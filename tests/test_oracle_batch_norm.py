"""Pins of the checker's batch normalisation inside f_theta (Section 2.2 names batch and layer normalisation
among the parts of f_theta; reading: Linear -> BatchNorm -> ReLU, batch statistics with biased variance while
training, running statistics moved by a momentum with the unbiased variance, running statistics at
evaluation).  None of them retypes the checker's formulas: autograd and the buffers of a library batch norm,
central finite differences of the loss, and properties of what the normalisation emits."""
import numpy as np
import pytest
import torch

import oracle


def _case(seed, d=9, h=16, c=5, n=48):
    rng = np.random.default_rng(seed)
    w = dict(w1=rng.normal(size=(d, h)) * 0.4, b1=rng.normal(size=h) * 0.1, w2=rng.normal(size=(h, c)) * 0.4,
             b2=rng.normal(size=c) * 0.1, g=1.0 + 0.3 * rng.normal(size=h), be=0.2 * rng.normal(size=h),
             rm=0.1 * rng.normal(size=h), rv=1.0 + 0.2 * rng.random(h))
    x = rng.normal(size=(n, d)).astype(np.float32)
    y = rng.integers(0, c, n).astype(np.int32)
    return d, h, c, w, x, y


def _model(d, h, c, w, **kw):
    return oracle.Mlp(d, h, c, w["w1"], w["b1"], w["w2"], w["b2"], batch_norm=True, ln_gamma=w["g"], ln_beta=w["be"],
                      bn_mean=w["rm"], bn_var=w["rv"], **kw)


def _torch_run(w, x, y, training, momentum=0.1, eps=1e-5):
    t = {k: torch.tensor(np.asarray(v, dtype=np.float64), requires_grad=k not in ("rm", "rv")) for k, v in w.items()}
    X = torch.tensor(x.astype(np.float64), requires_grad=True)
    z = X @ t["w1"] + t["b1"]
    rm, rv = t["rm"].clone(), t["rv"].clone()
    hd = torch.relu(torch.nn.functional.batch_norm(z, rm, rv, t["g"], t["be"], training, momentum, eps))
    logits = hd @ t["w2"] + t["b2"]
    loss = torch.nn.functional.cross_entropy(logits, torch.tensor(y.astype(np.int64)))
    return loss, t, X, hd, logits, rm, rv


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_training_step_matches_autograd_and_the_buffers_of_the_library_batch_norm(seed):
    d, h, c, w, x, y = _case(seed)
    m = _model(d, h, c, w, optimizer=oracle.SGD, lr=0.0, round_bf16=False, bn_momentum=0.1)
    loss, grad, dx = m.train_step_dx(x, y)
    ref, t, X, _, _, rm, rv = _torch_run(w, x, y, True)
    ref.backward()
    want = np.concatenate([t[k].grad.numpy().ravel() for k in ("w1", "b1", "w2", "b2", "g", "be")] + [np.zeros(2 * h)])
    assert abs(loss - ref.item()) < 1e-12
    np.testing.assert_allclose(grad, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(dx, X.grad.numpy(), rtol=0, atol=1e-12)
    u = m.unpack()
    # the running statistics moved as the library moves them (unbiased variance, momentum 0.1); lr = 0 left the rest
    np.testing.assert_allclose(u["bn_mean"], rm.numpy(), rtol=0, atol=1e-13)
    np.testing.assert_allclose(u["bn_var"], rv.numpy(), rtol=0, atol=1e-13)
    assert np.abs(u["bn_mean"] - w["rm"]).max() > 1e-3
    np.testing.assert_array_equal(u["w1"], w["w1"])


def test_evaluation_uses_the_running_statistics():
    d, h, c, w, x, y = _case(4)
    m = _model(d, h, c, w, round_bf16=False)
    got = m.embed(x, y=y, want_hidden=True)
    _, _, _, hd, logits, _, _ = _torch_run(w, x, y, False)
    np.testing.assert_allclose(got["hidden"], hd.detach().numpy().astype(np.float32), atol=1e-6)
    np.testing.assert_allclose(got["logits"], logits.detach().numpy().astype(np.float32), atol=1e-5)
    # ... and not the batch's own: a batch shifted by a constant row gives shifted outputs at evaluation
    w2 = dict(w, rm=w["rm"] + 1.0)
    assert np.abs(_model(d, h, c, w2, round_bf16=False).embed(x, want_hidden=True)["hidden"] - got["hidden"]).max() > 1e-2


def test_gradient_matches_central_differences_of_the_loss():
    d, h, c, w, x, y = _case(7, d=5, h=8, c=4, n=20)
    m0 = _model(d, h, c, w, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    _, grad, _ = m0.copy().train_step_dx(x, y)
    n_trained = grad.shape[0] - 2 * h
    rng = np.random.default_rng(3)
    step = 1e-6
    for p in rng.choice(n_trained, size=40, replace=False).tolist() + [n_trained - 1, n_trained - h - 1]:
        lo, hi = m0.copy(), m0.copy()
        lo.theta[p] -= step
        hi.theta[p] += step
        fd = (hi.train_step(x, y) - lo.train_step(x, y)) / (2 * step)
        assert abs(fd - grad[p]) < 1e-7, (p, fd, grad[p])
    # the training loss does not depend on the running statistics, and their gradient entries are 0
    assert np.all(grad[n_trained:] == 0.0)


def test_training_output_has_zero_mean_and_unit_variance_per_unit_and_training_lowers_the_loss():
    d, h, c, w, x, y = _case(11, n=200)
    w = dict(w, g=np.ones(h), be=np.zeros(h))
    z = x.astype(np.float64) @ w["w1"] + w["b1"]
    zhat = (z - z.mean(axis=0)) / np.sqrt(z.var(axis=0) + 1e-5)
    # shifting b1 leaves the normalised values, hence the training loss, unchanged
    a = _model(d, h, c, w, round_bf16=False).train_step(x, y)
    b = _model(d, h, c, dict(w, b1=w["b1"] + 3.0), round_bf16=False).train_step(x, y)
    assert abs(a - b) < 1e-10
    assert abs(zhat.mean()) < 1e-12
    rnd = _model(d, h, c, w, round_bf16=True, lr=0.01)
    first = rnd.copy().train_step(x, y)
    for _ in range(60):
        last = rnd.train_step(x, y)
    assert last < 0.8 * first
    u = rnd.unpack()
    # after 60 steps of momentum 0.1 the running mean has reached the batch mean of the current weights' z
    z_now = x.astype(np.float64) @ u["w1"] + u["b1"]
    assert np.abs(u["bn_mean"] - z_now.mean(axis=0)).max() < 0.05 * max(1.0, np.abs(z_now.mean(axis=0)).max())


def test_k_round_run_with_batch_norm():
    from paper_2302_13053_b200 import workloads as wl
    w = wl.make_config(1, scale=0.05)
    ws = wl.initial_weights(w)
    r = oracle.lmp_train(w.aggr, w.K, 6, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                         w.train_idx, w.val_idx, w.test_idx, ws, batch_norm=True)
    plain = oracle.lmp_train(w.aggr, w.K, 6, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                             w.train_idx, w.val_idx, w.test_idx, ws)
    assert abs(r["rounds"][0]["losses"][0] - plain["rounds"][0]["losses"][0]) > 1e-4
    assert r["rounds"][0]["model"].theta.shape[0] == plain["rounds"][0]["model"].theta.shape[0] + 4 * w.hidden
