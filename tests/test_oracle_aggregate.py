"""Pins for the CPU checker's aggregation (Eq. 1, AGGR + COMBINE).

Each test compares the checker with something that is not the checker: a dense
matrix expression, a scipy.sparse product, a closed form or an invariant.
"""
import numpy as np
import pytest
import scipy.sparse as sp

import oracle
from paper_2302_13053_b200 import workloads as wl


def dense_adj(rowptr, colidx):
    n = rowptr.shape[0] - 1
    a = np.zeros((n, n))
    for v in range(n):
        a[v, colidx[rowptr[v]:rowptr[v + 1]]] = 1.0
    return a


def graphs():
    out = []
    out.append(("ring12", *wl.ring_graph(12)))
    out.append(("complete7", *wl.complete_graph(7)))
    out.append(("star9", *wl.star_graph(9)))
    rp, ci = wl.random_small_graph(48, 130, seed=3)
    out.append(("rand48", rp, ci))
    n, rp, ci, _ = wl.degree_ladder_graph([0, 1, 2, 5, 33], seed=1)
    out.append(("ladder", rp, ci))
    out.append(("empty5", np.zeros(6, dtype=np.int64), np.zeros(0, dtype=np.int32)))
    return out


GRAPHS = graphs()


@pytest.mark.parametrize("name,rowptr,colidx", GRAPHS, ids=[g[0] for g in GRAPHS])
@pytest.mark.parametrize("dim", [1, 3, 8])
def test_gcn_matches_dense_normalised_adjacency(name, rowptr, colidx, dim):
    n = rowptr.shape[0] - 1
    rng = np.random.default_rng(5)
    q = rng.standard_normal((n, dim)).astype(np.float32)
    a = dense_adj(rowptr, colidx) + np.eye(n)
    dinv = np.diag(a.sum(1) ** -0.5)
    ref = dinv @ a @ dinv @ q.astype(np.float64)
    got = oracle.aggregate(oracle.GCN, rowptr, colidx, q)
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-7 * (1 + np.abs(ref).max()))


def test_gcn_matches_scipy_sparse_product():
    rowptr, colidx = wl.random_small_graph(300, 2000, seed=11)
    n = 300
    q = np.random.default_rng(0).standard_normal((n, 17)).astype(np.float32)
    a = sp.csr_matrix((np.ones(colidx.shape[0]), colidx, rowptr), shape=(n, n)) + sp.identity(n)
    d = np.asarray(a.sum(1)).ravel() ** -0.5
    ref = sp.diags(d) @ a @ sp.diags(d) @ q.astype(np.float64)
    got = oracle.aggregate(oracle.GCN, rowptr, colidx, q)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-6)


@pytest.mark.parametrize("maker,deg", [(lambda: wl.ring_graph(10), 2), (lambda: wl.complete_graph(6), 5)])
def test_gcn_regular_graph_is_scaled_sum(maker, deg):
    rowptr, colidx = maker()
    n = rowptr.shape[0] - 1
    q = np.random.default_rng(1).standard_normal((n, 4)).astype(np.float32)
    a = dense_adj(rowptr, colidx)
    ref = (q.astype(np.float64) + a @ q.astype(np.float64)) / (deg + 1)
    got = oracle.aggregate(oracle.GCN, rowptr, colidx, q)
    np.testing.assert_allclose(got, ref, atol=1e-6)
    const = np.full((n, 3), 2.5, dtype=np.float32)
    np.testing.assert_allclose(oracle.aggregate(oracle.GCN, rowptr, colidx, const), const, atol=1e-6)


def test_gcn_isolated_node_is_identity_and_operator_is_symmetric_and_linear():
    n, rowptr, colidx, perm = wl.degree_ladder_graph([3, 0, 7], seed=2)
    rng = np.random.default_rng(2)
    x = rng.standard_normal((n, 5)).astype(np.float32)
    y = rng.standard_normal((n, 5)).astype(np.float32)
    ax = oracle.aggregate(oracle.GCN, rowptr, colidx, x).astype(np.float64)
    ay = oracle.aggregate(oracle.GCN, rowptr, colidx, y).astype(np.float64)
    iso = np.flatnonzero(np.diff(rowptr) == 0)
    assert iso.size >= 2
    np.testing.assert_array_equal(ax[iso], x[iso])
    # x^T (A y) == (A x)^T y for the symmetric operator
    assert abs(np.sum(x * ay) - np.sum(ax * y)) < 1e-4
    axy = oracle.aggregate(oracle.GCN, rowptr, colidx, (2 * x - 3 * y).astype(np.float32))
    np.testing.assert_allclose(axy, 2 * ax - 3 * ay, atol=1e-5)


@pytest.mark.parametrize("name,rowptr,colidx", GRAPHS, ids=[g[0] for g in GRAPHS])
def test_sage_matches_dense_row_normalised_adjacency(name, rowptr, colidx):
    n = rowptr.shape[0] - 1
    q = np.random.default_rng(7).standard_normal((n, 6)).astype(np.float32)
    a = dense_adj(rowptr, colidx)
    deg = a.sum(1)
    mean = np.divide(a @ q.astype(np.float64), deg[:, None], out=np.zeros((n, 6)), where=deg[:, None] > 0)
    got = oracle.aggregate(oracle.SAGE_MEAN, rowptr, colidx, q)
    assert got.shape == (n, 12)
    np.testing.assert_array_equal(got[:, :6], q)                 # self half: bit-for-bit
    np.testing.assert_allclose(got[:, 6:], mean, atol=1e-6)
    assert np.all(got[deg == 0, 6:] == 0.0)                      # no neighbours -> zeros


def test_sage_mean_of_constant_is_constant_and_star_closed_form():
    rowptr, colidx = wl.random_small_graph(40, 100, seed=4)
    deg = np.diff(rowptr)
    const = np.full((40, 3), -1.75, dtype=np.float32)
    got = oracle.aggregate(oracle.SAGE_MEAN, rowptr, colidx, const)
    np.testing.assert_array_equal(got[deg > 0, 3:], const[deg > 0])
    rowptr, colidx = wl.star_graph(8)
    q = np.arange(9 * 2, dtype=np.float32).reshape(9, 2)
    got = oracle.aggregate(oracle.SAGE_MEAN, rowptr, colidx, q)
    np.testing.assert_allclose(got[0, 2:], q[1:].mean(0), rtol=1e-7)   # centre = mean of leaves
    np.testing.assert_array_equal(got[1:, 2:], np.repeat(q[:1], 8, 0))  # leaf = centre


@pytest.mark.parametrize("name,rowptr,colidx", GRAPHS, ids=[g[0] for g in GRAPHS])
def test_sage_max_matches_dense_masked_maximum(name, rowptr, colidx):
    """Max-pooling aggregator (Section 2.2): brute force over the dense
    adjacency; all-negative features catch a maximum started at zero."""
    n = rowptr.shape[0] - 1
    rng = np.random.default_rng(8)
    q = (rng.standard_normal((n, 5)) - 3.0).astype(np.float32)
    a = dense_adj(rowptr, colidx) > 0
    got = oracle.aggregate(oracle.SAGE_MAX, rowptr, colidx, q)
    assert got.shape == (n, 10)
    np.testing.assert_array_equal(got[:, :5], q)
    for v in range(n):
        want = q[a[v]].max(0) if a[v].any() else np.zeros(5, dtype=np.float32)
        np.testing.assert_array_equal(got[v, 5:], want)


def test_sage_max_star_ring_and_monotone_map():
    rowptr, colidx = wl.star_graph(8)
    q = np.random.default_rng(3).standard_normal((9, 4)).astype(np.float32)
    got = oracle.aggregate(oracle.SAGE_MAX, rowptr, colidx, q)
    np.testing.assert_array_equal(got[0, 4:], q[1:].max(0))            # centre = max over leaves
    np.testing.assert_array_equal(got[1:, 4:], np.repeat(q[:1], 8, 0))  # leaf = centre's row
    rowptr, colidx = wl.ring_graph(12)
    q = np.random.default_rng(4).standard_normal((12, 3)).astype(np.float32)
    got = oracle.aggregate(oracle.SAGE_MAX, rowptr, colidx, q)[:, 3:]
    np.testing.assert_array_equal(got, np.maximum(np.roll(q, 1, 0), np.roll(q, -1, 0)))
    # max commutes with an increasing map; min is max of the negation
    rowptr, colidx = wl.random_small_graph(50, 45, seed=6)
    q = np.random.default_rng(6).standard_normal((50, 4)).astype(np.float32)
    deg = np.diff(rowptr)
    base = oracle.aggregate(oracle.SAGE_MAX, rowptr, colidx, q)[:, 4:]
    cubed = oracle.aggregate(oracle.SAGE_MAX, rowptr, colidx, q ** 3)[:, 4:]
    np.testing.assert_array_equal(cubed[deg > 0], (base ** 3)[deg > 0])
    mean = oracle.aggregate(oracle.SAGE_MEAN, rowptr, colidx, q)[:, 4:]
    assert np.all(base[deg > 0] >= mean[deg > 0] - 1e-6)               # max >= mean
    one = deg == 1
    assert one.any()
    np.testing.assert_allclose(base[one], mean[one], rtol=1e-6)          # single neighbour: both are its row


def test_rows_subset_equals_full_result():
    rowptr, colidx = wl.random_small_graph(64, 300, seed=9)
    q = np.random.default_rng(9).standard_normal((64, 5)).astype(np.float32)
    rows = np.array([63, 0, 17, 17, 5])
    for aggr in (oracle.GCN, oracle.SAGE_MEAN, oracle.SAGE_MAX):
        full = oracle.aggregate(aggr, rowptr, colidx, q)
        np.testing.assert_array_equal(oracle.aggregate(aggr, rowptr, colidx, q, rows=rows), full[rows])
    gat = dict(heads=1, head_dim=5, a_src=np.ones((1, 5)), a_dst=np.ones((1, 5)))
    full = oracle.aggregate(oracle.GAT, rowptr, colidx, q, gat=gat)
    np.testing.assert_array_equal(oracle.aggregate(oracle.GAT, rowptr, colidx, q, rows=rows, gat=gat), full[rows])


# ------------------------------------------------------------------ GAT
def gat_dense(rowptr, colidx, p, heads, dh, a_src, a_dst, slope, self_loop=True):
    n = p.shape[0]
    a = dense_adj(rowptr, colidx) + (np.eye(n) if self_loop else 0)
    out = np.zeros((n, heads * dh))
    alphas = np.zeros((heads, n, n))
    pd = p.astype(np.float64)
    for k in range(heads):
        pk = pd[:, k * dh:(k + 1) * dh]
        s = pk @ a_src[k].astype(np.float64)
        t = pk @ a_dst[k].astype(np.float64)
        z = t[:, None] + s[None, :]                 # z[v, u]
        e = np.where(z > 0, z, slope * z)
        e = np.where(a > 0, e, -np.inf)
        e = e - e.max(1, keepdims=True)
        w = np.exp(e)
        w = w / w.sum(1, keepdims=True)
        alphas[k] = w
        out[:, k * dh:(k + 1) * dh] = w @ pk
    return out, alphas


@pytest.mark.parametrize("name,rowptr,colidx", GRAPHS[:5], ids=[g[0] for g in GRAPHS[:5]])
def test_gat_matches_dense_masked_softmax(name, rowptr, colidx):
    n = rowptr.shape[0] - 1
    heads, dh = 3, 4
    rng = np.random.default_rng(13)
    p = rng.standard_normal((n, heads * dh)).astype(np.float32)
    a_src = rng.standard_normal((heads, dh)).astype(np.float32)
    a_dst = rng.standard_normal((heads, dh)).astype(np.float32)
    ref, alphas = gat_dense(rowptr, colidx, p, heads, dh, a_src, a_dst, 0.2)
    gat = dict(heads=heads, head_dim=dh, a_src=a_src, a_dst=a_dst, negative_slope=0.2, add_self_loop=1)
    got, ae, aself = oracle.aggregate(oracle.GAT, rowptr, colidx, p, gat=gat, return_alpha=True)
    np.testing.assert_allclose(got, ref, atol=2e-6)
    # attention weights: match the dense ones and sum to 1 per node and head
    rows = np.repeat(np.arange(n), np.diff(rowptr))
    for k in range(heads):
        np.testing.assert_allclose(ae[:, k], alphas[k][rows, colidx], atol=1e-12)
        np.testing.assert_allclose(aself[:, k], np.diag(alphas[k]), atol=1e-12)
    tot = aself.copy()
    np.add.at(tot, rows, ae)
    np.testing.assert_allclose(tot, 1.0, atol=1e-12)


def test_gat_zero_attention_vectors_give_mean_over_closed_neighbourhood():
    rowptr, colidx = wl.random_small_graph(30, 80, seed=21)
    p = np.random.default_rng(21).standard_normal((30, 8)).astype(np.float32)
    z = np.zeros((2, 4), dtype=np.float32)
    got = oracle.aggregate(oracle.GAT, rowptr, colidx, p, gat=dict(heads=2, head_dim=4, a_src=z, a_dst=z))
    a = dense_adj(rowptr, colidx) + np.eye(30)
    ref = (a @ p.astype(np.float64)) / a.sum(1, keepdims=True)
    np.testing.assert_allclose(got, ref, atol=1e-6)


def test_gat_two_way_softmax_is_logistic_and_uses_source_and_destination_sides():
    # one edge 0-1, one head of width 1: node 0 attends over {1, 0}
    rowptr, colidx = wl.csr_from_edge_list(2, [(0, 1)])
    p = np.array([[0.7], [-1.3]], dtype=np.float32)
    a_src = np.array([[2.0]], dtype=np.float32)
    a_dst = np.array([[0.5]], dtype=np.float32)
    slope = 0.2
    lrelu = lambda z: z if z > 0 else slope * z
    s = 2.0 * p[:, 0].astype(np.float64)
    t = 0.5 * p[:, 0].astype(np.float64)
    e_nb, e_self = lrelu(s[1] + t[0]), lrelu(s[0] + t[0])
    w_nb = 1.0 / (1.0 + np.exp(e_self - e_nb))
    ref0 = w_nb * p[1, 0] + (1 - w_nb) * p[0, 0]
    got = oracle.aggregate(oracle.GAT, rowptr, colidx, p,
                           gat=dict(heads=1, head_dim=1, a_src=a_src, a_dst=a_dst, negative_slope=slope))
    assert abs(got[0, 0] - ref0) < 1e-7
    # without the self loop a single neighbour takes all the weight
    got = oracle.aggregate(oracle.GAT, rowptr, colidx, p,
                           gat=dict(heads=1, head_dim=1, a_src=a_src, a_dst=a_dst, add_self_loop=0))
    np.testing.assert_array_equal(got[:, 0], p[::-1, 0])


def test_gat_destination_term_cancels_when_all_scores_are_positive():
    rowptr, colidx = wl.random_small_graph(25, 70, seed=8)
    rng = np.random.default_rng(8)
    p = np.abs(rng.standard_normal((25, 4))).astype(np.float32) + 0.1
    a_src = np.abs(rng.standard_normal((1, 4))).astype(np.float32)
    outs = []
    for scale in (0.5, 3.0):
        a_dst = np.full((1, 4), scale, dtype=np.float32)       # every s_u + t_v > 0: linear regime
        outs.append(oracle.aggregate(oracle.GAT, rowptr, colidx, p,
                                     gat=dict(heads=1, head_dim=4, a_src=a_src, a_dst=a_dst)))
    np.testing.assert_allclose(outs[0], outs[1], atol=1e-6)


def test_gat_heads_are_independent():
    rowptr, colidx = wl.random_small_graph(20, 50, seed=6)
    rng = np.random.default_rng(6)
    heads, dh = 4, 3
    p = rng.standard_normal((20, heads * dh)).astype(np.float32)
    a_src = rng.standard_normal((heads, dh)).astype(np.float32)
    a_dst = rng.standard_normal((heads, dh)).astype(np.float32)
    base = oracle.aggregate(oracle.GAT, rowptr, colidx, p, gat=dict(heads=heads, head_dim=dh, a_src=a_src, a_dst=a_dst))
    perm = np.array([2, 0, 3, 1])
    cols = (perm[:, None] * dh + np.arange(dh)[None, :]).ravel()
    got = oracle.aggregate(oracle.GAT, rowptr, colidx, np.ascontiguousarray(p[:, cols]),
                           gat=dict(heads=heads, head_dim=dh, a_src=a_src[perm], a_dst=a_dst[perm]))
    np.testing.assert_array_equal(got, base[:, cols])
