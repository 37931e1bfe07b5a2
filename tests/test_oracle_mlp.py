"""Pins for the CPU checker's per-node model: training step (Section 2.3 /
3.1), embedding emission and prediction.  References are closed forms, finite
differences, and torch's CPU autograd + optimisers as a library special case.
"""
import math

import numpy as np
import pytest
import torch

import oracle


def make(d_in, hidden, n_classes, seed, **kw):
    rng = np.random.default_rng(seed)
    out1 = hidden if hidden > 0 else n_classes
    w1 = rng.standard_normal((d_in, out1)) * 0.3
    b1 = rng.standard_normal(out1) * 0.1
    w2 = rng.standard_normal((hidden, n_classes)) * 0.3 if hidden else None
    b2 = rng.standard_normal(n_classes) * 0.1 if hidden else None
    return oracle.Mlp(d_in, hidden, n_classes, w1, b1, w2, b2, **kw)


def torch_model(m: oracle.Mlp):
    u = m.unpack()
    ps = {k: torch.tensor(np.array(v), dtype=torch.float64, requires_grad=True) for k, v in u.items()}

    def fwd(x):
        if m.hidden > 0:
            return torch.relu(x @ ps["w1"] + ps["b1"]) @ ps["w2"] + ps["b2"]
        return x @ ps["w1"] + ps["b1"]
    return ps, fwd


def test_bf16_rounding_matches_torch_including_ties_and_specials():
    rng = np.random.default_rng(0)
    vals = np.concatenate([
        rng.standard_normal(2000).astype(np.float32),
        (rng.standard_normal(500) * 1e-30).astype(np.float32),
        (rng.standard_normal(500) * 1e30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8,
                  np.inf, -np.inf, 3.3895314e38, 1e-40], dtype=np.float32)])
    ref = torch.from_numpy(vals).to(torch.bfloat16).to(torch.float32).numpy()
    got = oracle.bf16_round(vals)
    np.testing.assert_array_equal(got.view(np.uint32), ref.view(np.uint32))
    assert math.isnan(float(oracle.bf16_round(np.array([np.nan], dtype=np.float32))[0]))


@pytest.mark.parametrize("hidden", [0, 6])
def test_zero_weights_give_log_of_class_count_and_hand_gradient(hidden):
    n, d, o = 11, 5, 4
    rng = np.random.default_rng(1)
    x = rng.standard_normal((n, d)).astype(np.float32)
    y = rng.integers(0, o, n).astype(np.int32)
    out1 = hidden if hidden else o
    m = oracle.Mlp(d, hidden, o, np.zeros((d, out1)), np.zeros(out1),
                   np.zeros((hidden, o)) if hidden else None, np.zeros(o) if hidden else None,
                   optimizer=oracle.SGD, lr=0.1, round_bf16=False)
    loss, grad = m.train_step(x, y, return_grad=True)
    assert abs(loss - math.log(o)) < 1e-14
    g = m.unpack(grad)
    dl = (np.full((n, o), 1.0 / o) - np.eye(o)[y]) / n
    if hidden == 0:
        np.testing.assert_allclose(g["w1"], x.astype(np.float64).T @ dl, atol=1e-15)
        np.testing.assert_allclose(g["b1"], dl.sum(0), atol=1e-15)
    else:   # hidden units are all 0 -> ReLU gate closed: only b2 moves
        assert np.all(g["w1"] == 0) and np.all(g["b1"] == 0) and np.all(g["w2"] == 0)
        np.testing.assert_allclose(g["b2"], dl.sum(0), atol=1e-15)


@pytest.mark.parametrize("hidden", [0, 5])
def test_gradient_matches_central_finite_differences(hidden):
    n, d, o = 9, 4, 3
    rng = np.random.default_rng(2)
    x = rng.standard_normal((n, d)).astype(np.float32)
    y = rng.integers(0, o, n).astype(np.int32)
    base = make(d, hidden, o, 3, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    _, grad = base.copy().train_step(x, y, return_grad=True)

    def loss_at(theta):
        m = base.copy()
        m.theta = theta.copy()
        return m.train_step(x, y)      # lr = 0: evaluates only

    h = 1e-6
    for p in rng.choice(base.theta.shape[0], size=min(25, base.theta.shape[0]), replace=False):
        tp, tm = base.theta.copy(), base.theta.copy()
        tp[p] += h
        tm[p] -= h
        fd = (loss_at(tp) - loss_at(tm)) / (2 * h)
        assert abs(fd - grad[p]) < 1e-7, (p, fd, grad[p])


@pytest.mark.parametrize("hidden", [0, 7])
@pytest.mark.parametrize("opt", [oracle.SGD, oracle.ADAM])
def test_steps_match_torch_autograd_and_optimisers(hidden, opt):
    n_all, d, o = 40, 6, 5
    rng = np.random.default_rng(4)
    x = rng.standard_normal((n_all, d)).astype(np.float32)
    idx = np.sort(rng.choice(n_all, 23, replace=False)).astype(np.int32)
    y = rng.integers(0, o, idx.shape[0]).astype(np.int32)
    m = make(d, hidden, o, 5, optimizer=opt, lr=0.05, round_bf16=False)
    ps, fwd = torch_model(m)
    order = ["w1", "b1", "w2", "b2"] if hidden else ["w1", "b1"]
    topt = (torch.optim.SGD if opt == oracle.SGD else torch.optim.Adam)([ps[k] for k in order], lr=0.05)
    xt = torch.tensor(x[idx], dtype=torch.float64)
    yt = torch.tensor(y, dtype=torch.long)
    for it in range(6):
        topt.zero_grad()
        tl = torch.nn.functional.cross_entropy(fwd(xt), yt)
        tl.backward()
        loss, grad = m.train_step(x, y, row_idx=idx, return_grad=True)
        assert abs(loss - tl.item()) < 1e-12
        tg = np.concatenate([ps[k].grad.numpy().ravel() for k in order])
        np.testing.assert_allclose(grad, tg, atol=1e-13)
        topt.step()
        tt = np.concatenate([ps[k].detach().numpy().ravel() for k in order])
        np.testing.assert_allclose(m.theta, tt, atol=1e-10)


def test_two_class_linear_step_is_the_textbook_logistic_regression_step():
    n, d = 13, 3
    rng = np.random.default_rng(6)
    x = rng.standard_normal((n, d)).astype(np.float32)
    y = rng.integers(0, 2, n).astype(np.int32)
    w = rng.standard_normal((d, 2)) * 0.2
    b = rng.standard_normal(2) * 0.2
    m = oracle.Mlp(d, 0, 2, w, b, optimizer=oracle.SGD, lr=0.3, round_bf16=False)
    m.train_step(x, y)
    # softmax over 2 classes == sigmoid of the logit difference
    xd = x.astype(np.float64)
    z = xd @ (w[:, 1] - w[:, 0]) + (b[1] - b[0])
    p1 = 1 / (1 + np.exp(-z))
    g1 = xd.T @ (p1 - y) / n
    new = m.unpack()
    np.testing.assert_allclose(new["w1"][:, 1], w[:, 1] - 0.3 * g1, atol=1e-14)
    np.testing.assert_allclose(new["w1"][:, 0], w[:, 0] + 0.3 * g1, atol=1e-14)
    np.testing.assert_allclose(new["b1"][1], b[1] - 0.3 * np.mean(p1 - y), atol=1e-14)


def test_loss_decreases_on_a_separable_toy_with_small_learning_rate():
    rng = np.random.default_rng(7)
    y = rng.integers(0, 3, 90).astype(np.int32)
    x = (np.eye(3)[y] * 3 + rng.standard_normal((90, 3)) * 0.3).astype(np.float32)
    m = make(3, 8, 3, 8, optimizer=oracle.SGD, lr=0.05, round_bf16=False)
    losses = [m.train_step(x, y) for _ in range(40)]
    assert all(b < a for a, b in zip(losses, losses[1:]))
    assert m.embed(x, y=y)["correct"] >= 88


def test_operand_rounding_happens_exactly_at_the_matrix_products():
    """With the bf16 flag every product sees bf16-rounded operands while sums,
    biases and the softmax stay wide: reproduce one step in torch from
    explicitly rounded tensors."""
    n, d, h, o = 17, 5, 4, 3
    rng = np.random.default_rng(9)
    x = rng.standard_normal((n, d)).astype(np.float32)
    y = rng.integers(0, o, n).astype(np.int32)
    m = make(d, h, o, 10, optimizer=oracle.SGD, lr=0.1, round_bf16=True)
    u = {k: np.array(v) for k, v in m.unpack().items()}
    r = lambda a: torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).to(torch.float64)
    xt = r(x)
    a1 = xt @ r(u["w1"]) + torch.tensor(u["b1"])
    hd = torch.relu(a1)
    lg = r(hd.numpy()) @ r(u["w2"]) + torch.tensor(u["b2"])
    sm = torch.softmax(lg, 1)
    loss_ref = torch.nn.functional.cross_entropy(lg, torch.tensor(y, dtype=torch.long)).item()
    dl = (sm - torch.eye(o, dtype=torch.float64)[torch.tensor(y, dtype=torch.long)]) / n
    dw2 = r(hd.numpy()).T @ r(dl.numpy())
    dhd = (r(dl.numpy()) @ r(u["w2"]).T) * (a1 > 0)
    dw1 = xt.T @ r(dhd.numpy())
    loss, grad = m.train_step(x, y, return_grad=True)
    g = m.unpack(grad)
    assert abs(loss - loss_ref) < 1e-12
    np.testing.assert_allclose(g["w2"], dw2.numpy(), atol=1e-13)
    np.testing.assert_allclose(g["b2"], r(dl.numpy()).sum(0).numpy(), atol=1e-13)     # 1^T dL is a product too
    np.testing.assert_allclose(g["w1"], dw1.numpy(), atol=1e-13)
    np.testing.assert_allclose(g["b1"], r(dhd.numpy()).sum(0).numpy(), atol=1e-13)


def test_embed_hidden_logits_prediction_and_tie_rule():
    n, d, h, o = 12, 4, 5, 3
    rng = np.random.default_rng(11)
    x = rng.standard_normal((n, d)).astype(np.float32)
    m = make(d, h, o, 12, round_bf16=False)
    u = m.unpack()
    hid = np.maximum(x.astype(np.float64) @ u["w1"] + u["b1"], 0)
    lg = hid @ u["w2"] + u["b2"]
    y = lg.argmax(1).astype(np.int32)
    y[:3] = (y[:3] + 1) % o                       # three wrong labels
    out = m.embed(x, y=y, want_hidden=True)
    np.testing.assert_allclose(out["hidden"], hid, atol=1e-6)
    np.testing.assert_allclose(out["logits"], lg, atol=1e-6)
    np.testing.assert_array_equal(out["pred"], lg.argmax(1))
    assert out["correct"] == n - 3
    idx = np.array([7, 2, 2, 9], dtype=np.int32)
    sub = m.embed(x, row_idx=idx, want_hidden=True)
    np.testing.assert_array_equal(sub["hidden"], out["hidden"][idx])
    # exact ties -> lowest class index
    tie = oracle.Mlp(2, 0, 4, np.zeros((2, 4)), np.array([1.0, 3.0, 3.0, 3.0]), round_bf16=False)
    assert list(tie.embed(np.ones((3, 2), dtype=np.float32))["pred"]) == [1, 1, 1]


def test_apply_update_alone_equals_the_update_inside_a_step():
    rng = np.random.default_rng(13)
    x = rng.standard_normal((20, 6)).astype(np.float32)
    y = rng.integers(0, 3, 20).astype(np.int32)
    for opt in (oracle.SGD, oracle.ADAM):
        a = make(6, 4, 3, 14, optimizer=opt, lr=0.05, round_bf16=False)
        b = a.copy()
        for _ in range(3):
            probe = a.copy()
            _, g = probe.train_step(x, y, return_grad=True)
            a.train_step(x, y)
            b.apply_update(g)
            np.testing.assert_array_equal(a.theta, b.theta)
            assert a.step == b.step
