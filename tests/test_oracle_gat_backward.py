"""Pins for the CPU checker's GAT backward pass and for the per-node model's input gradient (what a round
needs when the aggregator itself is trained, Section 2.2 / 3.1).

Neither is compared with itself: the backward is checked against central finite differences of an
independent dense forward written in numpy (double), against torch's autograd on a dense masked softmax,
and against the closed form it reduces to with zero attention vectors; the input gradient against finite
differences and autograd."""
import numpy as np
import pytest
import torch

import oracle
from paper_2302_13053_b200 import workloads as wl
from test_oracle_aggregate import GRAPHS, dense_adj, gat_dense
from test_oracle_mlp import make, torch_model


def setup(n, heads, dh, seed):
    rng = np.random.default_rng(seed)
    p = rng.standard_normal((n, heads * dh)).astype(np.float32)
    a_src = (rng.standard_normal((heads, dh)) * 0.7).astype(np.float32)
    a_dst = (rng.standard_normal((heads, dh)) * 0.7).astype(np.float32)
    g = rng.standard_normal((n, heads * dh))
    return p, a_src, a_dst, g


@pytest.mark.parametrize("name,rowptr,colidx", GRAPHS[:5], ids=[g[0] for g in GRAPHS[:5]])
@pytest.mark.parametrize("self_loop", [1, 0])
def test_gat_backward_matches_finite_differences_of_a_dense_forward(name, rowptr, colidx, self_loop):
    n = rowptr.shape[0] - 1
    if not self_loop and (np.diff(rowptr) == 0).any():
        pytest.skip("a node without neighbours has an empty softmax set without the self loop")
    heads, dh, slope = 2, 3, 0.2
    p, a_src, a_dst, g = setup(n, heads, dh, 21)
    gat = dict(heads=heads, head_dim=dh, a_src=a_src, a_dst=a_dst, negative_slope=slope, add_self_loop=self_loop)
    dp, da_src, da_dst = oracle.gat_backward(rowptr, colidx, p, gat, g)

    def objective(pp, aa, bb):      # sum_v <g_v, Z_v> with Z from the dense double forward
        z, _ = gat_dense(rowptr, colidx, pp, heads, dh, aa, bb, slope, self_loop=bool(self_loop))
        return float((g * z).sum())

    h = 1e-6
    rng = np.random.default_rng(1)
    pd, ad, bd = p.astype(np.float64), a_src.astype(np.float64), a_dst.astype(np.float64)
    for _ in range(30):
        i, j = rng.integers(0, n), rng.integers(0, heads * dh)
        pp, pm = pd.copy(), pd.copy()
        pp[i, j] += h
        pm[i, j] -= h
        fd = (objective(pp, ad, bd) - objective(pm, ad, bd)) / (2 * h)
        assert abs(fd - dp[i, j]) < 2e-6 * (1 + abs(fd)), ("dp", i, j, fd, dp[i, j])
    for k in range(heads):
        for j in range(dh):
            for which, grad in (("src", da_src), ("dst", da_dst)):
                ap, am = (ad.copy(), ad.copy()) if which == "src" else (bd.copy(), bd.copy())
                ap[k, j] += h
                am[k, j] -= h
                if which == "src":
                    fd = (objective(pd, ap, bd) - objective(pd, am, bd)) / (2 * h)
                else:
                    fd = (objective(pd, ad, ap) - objective(pd, ad, am)) / (2 * h)
                assert abs(fd - grad[k, j]) < 2e-6 * (1 + abs(fd)), (which, k, j, fd, grad[k, j])


def test_gat_backward_matches_torch_autograd_on_a_dense_masked_softmax():
    rowptr, colidx = wl.random_small_graph(40, 150, seed=8)
    n, heads, dh, slope = 40, 3, 4, 0.2
    p, a_src, a_dst, g = setup(n, heads, dh, 5)
    adj = torch.tensor(dense_adj(rowptr, colidx) + np.eye(n))
    pt = torch.tensor(p, dtype=torch.float64, requires_grad=True)
    at = torch.tensor(a_src, dtype=torch.float64, requires_grad=True)
    bt = torch.tensor(a_dst, dtype=torch.float64, requires_grad=True)
    outs = []
    for k in range(heads):
        pk = pt[:, k * dh:(k + 1) * dh]
        z = (pk @ bt[k])[:, None] + (pk @ at[k])[None, :]
        e = torch.nn.functional.leaky_relu(z, slope).masked_fill(adj == 0, float("-inf"))
        outs.append(torch.softmax(e, dim=1) @ pk)
    (torch.cat(outs, dim=1) * torch.tensor(g)).sum().backward()
    gat = dict(heads=heads, head_dim=dh, a_src=a_src, a_dst=a_dst, negative_slope=slope, add_self_loop=1)
    dp, da_src, da_dst = oracle.gat_backward(rowptr, colidx, p, gat, g)
    np.testing.assert_allclose(dp, pt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(da_src, at.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(da_dst, bt.grad.numpy(), atol=1e-12)


def test_gat_backward_with_zero_attention_is_the_transposed_closed_neighbourhood_mean():
    """a_src = a_dst = 0: every weight is 1 / (deg v + 1), so dp = M^T dz with M the mean over N(v) and v
    (the terms through the scores vanish with the attention vectors); rows of dz outside a chosen subset
    are zero, as in training on a subset of the nodes."""
    rowptr, colidx = wl.random_small_graph(60, 200, seed=2)
    n, heads, dh = 60, 2, 5
    p, _, _, g = setup(n, heads, dh, 9)
    g[np.random.default_rng(0).random(n) < 0.5] = 0.0
    zero = np.zeros((heads, dh), dtype=np.float32)
    gat = dict(heads=heads, head_dim=dh, a_src=zero, a_dst=zero, negative_slope=0.2, add_self_loop=1)
    dp, da_src, da_dst = oracle.gat_backward(rowptr, colidx, p, gat, g)
    m = dense_adj(rowptr, colidx) + np.eye(n)
    m = m / m.sum(1, keepdims=True)
    np.testing.assert_allclose(dp, m.T @ g, atol=1e-13)
    # with equal weights the score gradients are slope * alpha * (dalpha - mean dalpha): they sum to zero per destination
    assert np.isfinite(da_src).all() and np.isfinite(da_dst).all()
    # permuting the heads permutes the gradients: heads are independent
    perm = [1, 0]
    cols = np.concatenate([np.arange(k * dh, (k + 1) * dh) for k in perm])
    a_src = np.random.default_rng(3).standard_normal((heads, dh)).astype(np.float32)
    gat2 = dict(gat, a_src=a_src, a_dst=a_src[::-1].copy())
    d1 = oracle.gat_backward(rowptr, colidx, p, gat2, g)
    gat3 = dict(gat, a_src=a_src[perm], a_dst=a_src[::-1][perm].copy())
    d2 = oracle.gat_backward(rowptr, colidx, p[:, cols], gat3, g[:, cols])
    np.testing.assert_allclose(d2[0], d1[0][:, cols], atol=1e-13)
    np.testing.assert_allclose(d2[1], d1[1][perm], atol=1e-13)


@pytest.mark.parametrize("hidden", [0, 6])
def test_input_gradient_matches_finite_differences_and_autograd(hidden):
    n, d, o = 11, 5, 4
    rng = np.random.default_rng(12)
    x = rng.standard_normal((n, d)).astype(np.float32)
    y = rng.integers(0, o, n).astype(np.int32)
    base = make(d, hidden, o, 8, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    loss, grad, dx = base.copy().train_step_dx(x, y)
    loss2, grad2 = base.copy().train_step(x, y, return_grad=True)
    assert loss == loss2 and np.array_equal(grad, grad2)             # the same step, one more output
    ps, fwd = torch_model(base)
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    torch.nn.functional.cross_entropy(fwd(xt), torch.tensor(y, dtype=torch.long)).backward()
    np.testing.assert_allclose(dx, xt.grad.numpy(), atol=1e-13)
    h = 1e-3                      # x is stored in fp32: a step that fp32 represents well
    for _ in range(12):
        i, k = rng.integers(0, n), rng.integers(0, d)
        xp, xm = x.copy(), x.copy()
        xp[i, k] += np.float32(h)
        xm[i, k] -= np.float32(h)
        fd = (base.copy().train_step(xp, y) - base.copy().train_step(xm, y)) / (float(xp[i, k]) - float(xm[i, k]))
        assert abs(fd - dx[i, k]) < 1e-6, (i, k, fd, dx[i, k])


def test_input_gradient_rounds_its_operands_like_every_other_product():
    n, d, h, o = 6, 4, 3, 2
    rng = np.random.default_rng(3)
    x = rng.standard_normal((n, d)).astype(np.float32)
    y = rng.integers(0, o, n).astype(np.int32)
    m = make(d, h, o, 2, optimizer=oracle.SGD, lr=0.0, round_bf16=True)
    _, grad, dx = m.copy().train_step_dx(x, y)
    # dX = bf16(dHd) bf16(W1)^T: rebuild dHd from the bias gradient's definition is not possible (it is a sum),
    # so recompute the row-local backward in numpy with the rounding points of the contract
    r = oracle.bf16_round
    w = m.unpack()
    xr, w1r, w2r = r(x).astype(np.float64), r(w["w1"]).astype(np.float64), r(w["w2"]).astype(np.float64)
    a1 = xr @ w1r + w["b1"]
    hd = r(np.maximum(a1, 0)).astype(np.float64)
    lg = hd @ w2r + w["b2"]
    sm = np.exp(lg - lg.max(1, keepdims=True))
    sm /= sm.sum(1, keepdims=True)
    dl = (sm - np.eye(o)[y]) / n
    dhd = (r(dl).astype(np.float64) @ w2r.T) * (a1 > 0)
    want = r(dhd).astype(np.float64) @ w1r.T
    np.testing.assert_allclose(dx, want, atol=1e-12)


def test_array_rounding_equals_the_scalar_routine():
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.standard_normal(4000).astype(np.float32) * 10.0 ** rng.integers(-20, 20, 4000),
                        np.array([0.0, -0.0, np.inf, -np.inf, np.nan, 1.00390625, 1.01171875, 3.3895314e38, 1e-45],
                                 dtype=np.float32)]).astype(np.float32)
    got, want = oracle.bf16_round_array(a), oracle.bf16_round(a)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def gat_layer(seed, n, d, heads, dh, hidden, o, lr=0.05, round_bf16=False, opt=oracle.SGD):
    rng = np.random.default_rng(seed)
    rowptr, colidx = wl.random_small_graph(n, 3 * n, seed=seed)
    mlp = make(heads * dh, hidden, o, seed + 1, optimizer=opt, lr=lr, round_bf16=round_bf16)
    gat = dict(heads=heads, head_dim=dh, negative_slope=0.2)
    layer = oracle.GatLayer(rowptr, colidx, gat, rng.standard_normal((d, heads * dh)) / np.sqrt(d),
                            rng.standard_normal((heads, dh)) * 0.5, rng.standard_normal((heads, dh)) * 0.5, mlp)
    q = rng.standard_normal((n, d)).astype(np.float32)
    return layer, q, rng


@pytest.mark.parametrize("hidden", [0, 6])
def test_whole_layer_gradient_matches_torch_autograd_through_projection_attention_and_model(hidden):
    """The composition the K-round loop trains (projection -> GAT -> per-node model -> loss), end to end
    against autograd on dense tensors, and the SGD step of every parameter."""
    n, d, heads, dh, o = 30, 7, 2, 3, 4
    layer, q, rng = gat_layer(4, n, d, heads, dh, hidden, o)
    train_idx = np.sort(rng.choice(n, 17, replace=False)).astype(np.int32)
    y = rng.integers(0, o, 17).astype(np.int32)
    before = layer.copy()
    loss, grad = layer.train_step(q, y, train_idx, return_grad=True)
    w_att, a_src, a_dst = before.parts()
    ps, fwd = torch_model(before.mlp)
    wt = torch.tensor(w_att, requires_grad=True)
    at = torch.tensor(a_src, requires_grad=True)
    bt = torch.tensor(a_dst, requires_grad=True)
    pt = torch.tensor(q, dtype=torch.float64) @ wt
    # the checker hands P on in fp32 (as the projection product leaves it): do the same, keeping the graph
    pt = pt + (pt.detach().to(torch.float32).to(torch.float64) - pt.detach())
    adj = torch.tensor(dense_adj(layer.rowptr, layer.colidx) + np.eye(n))
    outs = []
    for k in range(heads):
        pk = pt[:, k * dh:(k + 1) * dh]
        z = (pk @ bt[k])[:, None] + (pk @ at[k])[None, :]
        e = torch.nn.functional.leaky_relu(z, 0.2).masked_fill(adj == 0, float("-inf"))
        outs.append(torch.softmax(e, dim=1) @ pk)
    zt = torch.cat(outs, dim=1)[torch.tensor(train_idx, dtype=torch.long)]
    zt = zt + (zt.detach().to(torch.float32).to(torch.float64) - zt.detach())      # Z leaves the aggregation in fp32
    tl = torch.nn.functional.cross_entropy(fwd(zt), torch.tensor(y, dtype=torch.long))
    tl.backward()
    # (P and Z are handed on in fp32 on both sides; a sum taken in another order can land on the other side of
    #  an fp32 rounding boundary, which moves the loss by ~1e-9: hence 1e-8 and not 1e-12)
    assert abs(loss - tl.item()) < 1e-8
    order = ["w1", "b1", "w2", "b2"] if hidden else ["w1", "b1"]
    want = np.concatenate([wt.grad.numpy().ravel(), at.grad.numpy().ravel(), bt.grad.numpy().ravel()] +
                          [ps[k].grad.numpy().ravel() for k in order])
    np.testing.assert_allclose(grad, want, atol=1e-8)
    np.testing.assert_allclose(layer.att, before.att - 0.05 * grad[:before.att.shape[0]], atol=1e-14)
    np.testing.assert_allclose(layer.mlp.theta, before.mlp.theta - 0.05 * grad[before.att.shape[0]:], atol=1e-14)


def test_training_the_attention_lowers_the_loss_faster_than_leaving_it_frozen():
    n, d, heads, dh, o = 80, 6, 2, 4, 3
    layer, q, rng = gat_layer(7, n, d, heads, dh, 8, o, lr=0.02, opt=oracle.ADAM)
    labels = rng.integers(0, o, n).astype(np.int32)
    train_idx = np.arange(0, n, 2).astype(np.int32)
    frozen = layer.copy()
    x = frozen.aggregate(q, rows=train_idx.astype(np.int64))
    lt = [layer.train_step(q, labels[train_idx], train_idx) for _ in range(60)]
    lf = [frozen.mlp.train_step(x, labels[train_idx]) for _ in range(60)]
    assert abs(lt[0] - lf[0]) < 1e-12 and lt[-1] < lt[0]
    assert lt[-1] < lf[-1]                       # more parameters fitted to the same rows
    assert np.abs(layer.att - frozen.att).max() > 1e-3
