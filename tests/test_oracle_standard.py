"""Pins of the checker of standard (end-to-end) GNN training, the scheme Section 2.3 describes and lazy message
passing is compared with.  None of them retypes the checker's code path: autograd of a model written on a
dense adjacency matrix, the adjoint identity <A x, g> = <x, A^T g> taken against the (separately pinned)
aggregation checker, the one-layer case against the per-node model checker, and hand values on a path graph."""
import numpy as np
import pytest
import torch

import oracle
from oracle import standard


def _graph(n, seed, isolated=True):
    """Symmetric CSR without self loops or duplicates; node n - 1 isolated if asked."""
    rng = np.random.default_rng(seed)
    a = rng.random((n, n)) < 0.25
    a = np.triu(a, 1)
    a = a | a.T
    if isolated:
        a[n - 1, :] = a[:, n - 1] = False
    rowptr = np.concatenate([[0], np.cumsum(a.sum(1))]).astype(np.int64)
    colidx = np.concatenate([np.nonzero(r)[0] for r in a]).astype(np.int32)
    return a.astype(np.float64), rowptr, colidx


def _weights(dims, seed):
    rng = np.random.default_rng(seed)
    return [dict(w1=rng.normal(size=(dims[i], dims[i + 1])) * 0.5, b1=rng.normal(size=dims[i + 1]) * 0.1)
            for i in range(len(dims) - 1)]


def _dense_forward(aggr, a, f, ws):
    """The same model on a dense adjacency matrix, in torch (double)."""
    n = a.shape[0]
    A = torch.tensor(a)
    deg = A.sum(1)
    h = f
    for m, (w, b) in enumerate(ws):
        if aggr == oracle.GCN:
            nrm = 1.0 / torch.sqrt(deg + 1.0)
            x = nrm[:, None] * ((A + torch.eye(n, dtype=torch.float64)) @ (nrm[:, None] * h))
        else:
            mean = (A @ h) / torch.clamp(deg, min=1.0)[:, None]
            x = torch.cat([h, mean], dim=1)
        z = x @ w + b
        h = torch.relu(z) if m < len(ws) - 1 else z
    return h


@pytest.mark.parametrize("aggr", [oracle.GCN, oracle.SAGE_MEAN])
@pytest.mark.parametrize("K", [1, 2, 3])
def test_loss_and_every_gradient_match_autograd_of_a_dense_model(aggr, K):
    n, d0, hid, c = 23, 6, 8, 4
    a, rowptr, colidx = _graph(n, K)
    rng = np.random.default_rng(10 + K)
    f = rng.normal(size=(n, d0)).astype(np.float32)
    y = rng.integers(0, c, n).astype(np.int32)
    tr = rng.permutation(n)[:12]
    mult = 2 if aggr == oracle.SAGE_MEAN else 1
    dims_in = [d0 * mult] + [hid * mult] * (K - 1)
    outs = [hid] * (K - 1) + [c]
    rngw = np.random.default_rng(5)
    ws = [dict(w1=rngw.normal(size=(dims_in[m], outs[m])) * 0.5, b1=rngw.normal(size=outs[m]) * 0.1) for m in range(K)]
    model = standard.StandardGnn(aggr, rowptr, colidx, ws, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    loss, grads = model.train_step(f, y, tr, return_grad=True)
    tw = [(torch.tensor(w["w1"], requires_grad=True), torch.tensor(w["b1"], requires_grad=True)) for w in ws]
    logits = _dense_forward(aggr, a, torch.tensor(f.astype(np.float64)), tw)
    ref = torch.nn.functional.cross_entropy(logits[torch.tensor(tr)], torch.tensor(y[tr].astype(np.int64)))
    ref.backward()
    # (the last layer's input goes through the per-node checker's fp32 interface: 1e-6, not 1e-12)
    assert abs(loss - ref.item()) < 1e-6
    for m in range(K):
        want = np.concatenate([tw[m][0].grad.numpy().ravel(), tw[m][1].grad.numpy()])
        np.testing.assert_allclose(grads[m], want, rtol=0, atol=2e-7 * max(1.0, np.abs(want).max()))
        assert np.abs(want).max() > 1e-4
    np.testing.assert_allclose(model.forward(f)[2], logits.detach().numpy(), rtol=0, atol=1e-6)


@pytest.mark.parametrize("aggr", [oracle.GCN, oracle.SAGE_MEAN])
def test_forward_is_the_aggregation_checker_and_backward_is_its_adjoint(aggr):
    n, d = 40, 5
    _, rowptr, colidx = _graph(n, 3)
    # a directed (non-symmetric) pattern as well: the transpose must not rely on symmetry
    rng = np.random.default_rng(0)
    a = (rng.random((n, n)) < 0.2) & ~np.eye(n, dtype=bool)
    rp2 = np.concatenate([[0], np.cumsum(a.sum(1))]).astype(np.int64)
    ci2 = np.concatenate([np.nonzero(r)[0] for r in a]).astype(np.int32)
    for rp, ci in ((rowptr, colidx), (rp2, ci2)):
        model = standard.StandardGnn(aggr, rp, ci, [dict(w1=np.zeros((1, 1)), b1=np.zeros(1))], round_bf16=False)
        h = rng.normal(size=(n, d)).astype(np.float32)
        want = oracle.aggregate(aggr, rp, ci, h)
        got = model.aggregate(h.astype(np.float64))
        np.testing.assert_allclose(got, want, rtol=0, atol=2e-6)
        g = rng.normal(size=want.shape)
        lhs = float((want.astype(np.float64) * g).sum())
        rhs = float((h.astype(np.float64) * model.aggregate_transposed(g)).sum())
        assert abs(lhs - rhs) < 1e-5 * max(1.0, abs(lhs))


def test_one_layer_is_the_per_node_model_on_the_aggregated_rows():
    n, d0, c = 30, 7, 5
    _, rowptr, colidx = _graph(n, 8)
    rng = np.random.default_rng(2)
    f = rng.normal(size=(n, d0)).astype(np.float32)
    y = rng.integers(0, c, n).astype(np.int32)
    tr = np.arange(0, n, 2)
    ws = _weights([d0, c], 1)
    for rounded in (False, True):
        model = standard.StandardGnn(oracle.GCN, rowptr, colidx, ws, lr=0.01, round_bf16=rounded)
        ref = oracle.Mlp(d0, 0, c, ws[0]["w1"], ws[0]["b1"], lr=0.01, round_bf16=rounded)
        x = oracle.aggregate(oracle.GCN, rowptr, colidx, f)
        for _ in range(3):
            a, b = model.train_step(f, y, tr), ref.train_step(x, y[tr], row_idx=tr.astype(np.int32))
            assert abs(a - b) < 1e-6
        np.testing.assert_allclose(model.layers[0].theta, ref.theta, rtol=0, atol=1e-5)


def test_hand_values_on_a_path_of_three_nodes():
    # 0 - 1 - 2, scalar features (1, 2, 4), GCN, two layers with weights 1 and zero biases, node 1 trained:
    # degrees + 1 = (2, 3, 2); X^1 = Ahat f, H^1 = X^1 (all positive), X^2 = Ahat H^1
    rowptr = np.array([0, 1, 3, 4], dtype=np.int64)
    colidx = np.array([1, 0, 2, 1], dtype=np.int32)
    f = np.array([[1.0], [2.0], [4.0]], dtype=np.float32)
    s = 1.0 / np.sqrt(6.0)
    ahat = np.array([[0.5, s, 0.0], [s, 1.0 / 3.0, s], [0.0, s, 0.5]])
    ws = [dict(w1=np.ones((1, 1)), b1=np.zeros(1)), dict(w1=np.ones((1, 2)) * np.array([[1.0, -1.0]]), b1=np.zeros(2))]
    model = standard.StandardGnn(oracle.GCN, rowptr, colidx, ws, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    xs, zs, logits = model.forward(f)
    x1 = ahat @ f.astype(np.float64)
    x2 = ahat @ x1
    np.testing.assert_allclose(xs[0], x1, atol=1e-12)
    np.testing.assert_allclose(xs[1], x2, atol=1e-12)
    np.testing.assert_allclose(logits, x2 * np.array([[1.0, -1.0]]), atol=1e-12)
    loss, grads = model.train_step(f, np.array([0, 0, 0], dtype=np.int32), np.array([1]), return_grad=True)
    t = x2[1, 0]
    p1 = 1.0 / (1.0 + np.exp(2.0 * t))                 # soft-max weight of class 1 at logits (t, -t)
    assert abs(loss - np.log1p(np.exp(-2.0 * t))) < 1e-9
    # dLoss / dX^2[1] = -2 p1 (through both classes); layer-1 weight gradient = sum_v X^1[v] Ahat[1, v] dLoss/dX^2[1]
    want_w1 = -2.0 * p1 * float(ahat[1] @ x1[:, 0])
    want_b1 = -2.0 * p1 * float(ahat[1].sum())
    np.testing.assert_allclose(grads[0], [want_w1, want_b1], atol=1e-7)


def test_short_run_learns_and_counts_its_aggregations():
    from paper_2302_13053_b200 import workloads as wl
    w = wl.make_config(1, scale=0.15)
    ws = wl.initial_weights(w)
    out = standard.standard_train(w.aggr, 6, w.rowptr, w.colidx, w.features, w.labels, w.train_idx, w.val_idx,
                                  w.test_idx, ws, lr=0.01)
    assert out["losses"][-1] < out["losses"][0]
    assert out["n_aggregations_forward"] == 6 * (w.K - 1) + 1 and out["n_aggregations_backward"] == 6 * (w.K - 1)
    assert out["val_correct"][out["best_iter"] - 1] == out["best_val_correct"] == max(out["val_correct"])
