"""Pins of the checker's layer normalisation inside f_theta (Section 2.2 lists normalisation layers among
the parts of f_theta; reading: Linear -> LayerNorm -> ReLU, statistics over the hidden units of a row, biased
variance, trainable gamma / beta at the end of theta).  None of them retypes the checker's formulas:
autograd of a library layer norm, central finite differences of the loss, and properties the normalisation
must have (zero mean / unit variance of what it emits, invariance under a rescaling of what it is fed)."""
import numpy as np
import pytest
import torch

import oracle


def _case(seed, d=9, h=16, c=5, n=48):
    rng = np.random.default_rng(seed)
    w = dict(w1=rng.normal(size=(d, h)) * 0.4, b1=rng.normal(size=h) * 0.1, w2=rng.normal(size=(h, c)) * 0.4,
             b2=rng.normal(size=c) * 0.1, g=1.0 + 0.3 * rng.normal(size=h), be=0.2 * rng.normal(size=h))
    x = rng.normal(size=(n, d)).astype(np.float32)
    y = rng.integers(0, c, n).astype(np.int32)
    return d, h, c, w, x, y


def _model(d, h, c, w, **kw):
    return oracle.Mlp(d, h, c, w["w1"], w["b1"], w["w2"], w["b2"], layer_norm=True, ln_gamma=w["g"], ln_beta=w["be"], **kw)


def _torch_loss(w, x, y, h, eps=1e-5):
    t = {k: torch.tensor(np.asarray(v, dtype=np.float64), requires_grad=True) for k, v in w.items()}
    X = torch.tensor(x.astype(np.float64), requires_grad=True)
    z = X @ t["w1"] + t["b1"]
    hd = torch.relu(torch.nn.functional.layer_norm(z, (h,), t["g"], t["be"], eps))
    loss = torch.nn.functional.cross_entropy(hd @ t["w2"] + t["b2"], torch.tensor(y.astype(np.int64)))
    return loss, t, X, hd


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_loss_and_every_gradient_match_autograd_of_the_library_layer_norm(seed):
    d, h, c, w, x, y = _case(seed)
    m = _model(d, h, c, w, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    loss, grad, dx = m.train_step_dx(x, y)
    ref, t, X, _ = _torch_loss(w, x, y, h)
    ref.backward()
    want = np.concatenate([t[k].grad.numpy().ravel() for k in ("w1", "b1", "w2", "b2", "g", "be")])
    assert abs(loss - ref.item()) < 1e-12
    np.testing.assert_allclose(grad, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(dx, X.grad.numpy(), rtol=0, atol=1e-12)
    # a plausible slip (gamma left out of the gradient that leaves the normalisation, or the two mean terms
    # dropped) moves d W1 by far more than this tolerance
    assert np.abs(want[:d * h]).max() > 1e-4


def test_gradient_matches_central_differences_of_the_loss():
    d, h, c, w, x, y = _case(7, d=5, h=8, c=4, n=20)
    m0 = _model(d, h, c, w, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    _, grad, _ = m0.copy().train_step_dx(x, y)
    rng = np.random.default_rng(3)
    step = 1e-6
    for p in rng.choice(grad.shape[0], size=40, replace=False).tolist() + [grad.shape[0] - 1, grad.shape[0] - h - 1]:
        lo, hi = m0.copy(), m0.copy()
        lo.theta[p] -= step
        hi.theta[p] += step
        fd = (hi.train_step(x, y) - lo.train_step(x, y)) / (2 * step)
        assert abs(fd - grad[p]) < 1e-7, (p, fd, grad[p])


def test_emitted_rows_are_normalised_and_blind_to_the_scale_of_what_feeds_the_normalisation():
    d, h, c, w, x, y = _case(11)
    w = dict(w, g=np.ones(h), be=np.zeros(h))
    # with gamma = 1, beta = 0 the hidden output is ReLU(zhat): compare against numpy statistics of X W1 + b1
    m = _model(d, h, c, w, round_bf16=False)
    hid = m.embed(x, want_hidden=True)["hidden"]
    z = x.astype(np.float64) @ w["w1"] + w["b1"]
    zhat = (z - z.mean(axis=1, keepdims=True)) / np.sqrt(z.var(axis=1, keepdims=True) + 1e-5)
    np.testing.assert_allclose(hid, np.maximum(zhat, 0.0).astype(np.float32), atol=1e-6)
    # scaling W1 and b1 by a positive factor changes z's scale only: what the normalisation emits, and so the
    # loss, stays (up to eps next to the variance, made negligible here)
    big = dict(w, w1=w["w1"] * 64.0, b1=w["b1"] * 64.0)
    a = _model(d, h, c, dict(w, w1=w["w1"] * 8.0, b1=w["b1"] * 8.0), round_bf16=False, ln_eps=1e-12).train_step(x, y)
    b = _model(d, h, c, big, round_bf16=False, ln_eps=1e-12).train_step(x, y)
    assert abs(a - b) < 1e-9


def test_rounded_mode_stays_close_to_the_wide_one_and_trains():
    d, h, c, w, x, y = _case(5, n=200)
    wide = _model(d, h, c, w, round_bf16=False, lr=0.01)
    rnd = _model(d, h, c, w, round_bf16=True, lr=0.01)
    l0 = wide.copy().train_step(x, y)
    _, gw, _ = wide.copy().train_step_dx(x, y)
    _, gr, _ = rnd.copy().train_step_dx(x, y)
    assert np.abs(gw - gr).max() < 2e-2 * np.abs(gw).max()
    for _ in range(60):
        last = rnd.train_step(x, y)
    assert last < 0.8 * l0
    # gamma and beta have moved: they are trained
    u = rnd.unpack()
    assert np.abs(u["ln_gamma"] - w["g"]).max() > 1e-3 and np.abs(u["ln_beta"] - w["be"]).max() > 1e-3


def test_k_round_run_with_layer_norm_hands_on_normalised_representations():
    from paper_2302_13053_b200 import workloads as wl
    w = wl.make_config(1, scale=0.05)
    ws = wl.initial_weights(w)
    r = oracle.lmp_train(w.aggr, w.K, 6, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                         w.train_idx, w.val_idx, w.test_idx, ws, layer_norm=True)
    plain = oracle.lmp_train(w.aggr, w.K, 6, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                             w.train_idx, w.val_idx, w.test_idx, ws)
    assert len(r["rounds"]) == w.K
    # same initial weights, gamma = 1, beta = 0: the first loss differs from the plain model's (the
    # normalisation is really applied), and the kept parameter vectors carry 2 * hidden more entries
    assert abs(r["rounds"][0]["losses"][0] - plain["rounds"][0]["losses"][0]) > 1e-4
    assert r["rounds"][0]["model"].theta.shape[0] == plain["rounds"][0]["model"].theta.shape[0] + 2 * w.hidden
