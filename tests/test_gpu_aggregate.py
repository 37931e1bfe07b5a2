"""CUDA aggregation (retexo_aggregate) against the CPU checker, element by
element, on the same seeded inputs.  Tolerance for fp32 aggregation: max-abs
error per row <= 1e-5 x the row's L2 norm; rows that are exactly zero in the
reference must be exactly zero."""
import numpy as np
import pytest
import torch

import oracle
from paper_2302_13053_b200 import workloads as wl
from gpu_util import assert_rows_close, dev

pytestmark = pytest.mark.gpu


def gpu():
    from paper_2302_13053_b200 import binding
    return binding


def run_gpu(aggr, rowptr, colidx, q, ld=None, dim=None, **kw):
    B = gpu()
    n, d = q.shape
    ld = d if ld is None else ld
    buf = torch.zeros((n, ld), dtype=torch.float32, device="cuda")
    buf[:, :d] = dev(q)
    rp, ci = dev(rowptr.astype(np.int64)), dev(colidx.astype(np.int32))
    assert B.retexo_validate_csr(rp, ci) == (0, -1)
    out, out16 = B.retexo_aggregate(aggr, rp, ci, buf, dim=d if dim is None else dim, want_bf16=True, **kw)
    torch.cuda.synchronize()
    return out.cpu().numpy(), out16.float().cpu().numpy()


LADDER = [0, 1, 2, 31, 32, 33, 63, 64, 65, 1025, 2047, 2048, 2049, 4095, 4096, 4097, 9000]   # 4096: rows cut into segments


@pytest.mark.parametrize("aggr", [oracle.GCN, oracle.SAGE_MEAN])
@pytest.mark.parametrize("dim,ld", [(1, 1), (3, 3), (4, 4), (5, 8), (100, 100), (100, 128), (127, 128), (128, 128),
                                    (129, 129), (602, 602), (602, 604), (602, 608), (256, 256), (1433, 1433),
                                    (1433, 1436), (769, 772)])
def test_degree_ladder_every_bin_and_vector_width(aggr, dim, ld):
    n, rowptr, colidx, _ = wl.degree_ladder_graph(LADDER, seed=dim)
    # Positive features: with one or a few columns a long sum of signed values can cancel to a
    # result far smaller than its terms, and then no fp32 summation can be judged against the
    # norm of the result.  (The configurations' Gaussian features are tested below.)
    q = (np.abs(np.random.default_rng(dim).standard_normal((n, dim))) + 0.5).astype(np.float32)
    ref = oracle.aggregate(aggr, rowptr, colidx, q)
    got, got16 = run_gpu(aggr, rowptr, colidx, q, ld=ld)
    assert_rows_close(got, ref, what="fp32 out")
    # the bf16 copy is the same result rounded once
    np.testing.assert_array_equal(got16[:, :got.shape[1]],
                                  torch.from_numpy(got).to(torch.bfloat16).float().numpy())
    if aggr == oracle.SAGE_MEAN:
        np.testing.assert_array_equal(got[:, :dim], q)        # self half is a bit copy


@pytest.mark.parametrize("aggr", [oracle.GCN, oracle.SAGE_MEAN])
def test_empty_and_edgeless_graphs(aggr):
    B = gpu()
    rowptr = np.zeros(6, dtype=np.int64)
    colidx = np.zeros(0, dtype=np.int32)
    q = np.random.default_rng(0).standard_normal((5, 7)).astype(np.float32)
    ref = oracle.aggregate(aggr, rowptr, colidx, q)
    got, _ = run_gpu(aggr, rowptr, colidx, q)
    assert_rows_close(got, ref)
    # zero nodes: a valid no-op
    out, _ = B.retexo_aggregate(aggr, dev(np.zeros(1, dtype=np.int64)), dev(colidx),
                                torch.zeros((0, 4), device="cuda"), dim=4)
    assert out.shape[0] == 0


@pytest.mark.parametrize("dim,ld", [(1, 1), (3, 3), (5, 8), (100, 100), (127, 128), (602, 608), (256, 256),
                                    (1433, 1436), (769, 772)])
def test_max_pooling_is_bit_exact_over_every_degree_bin(dim, ld):
    """A maximum involves no rounding: every element must equal the checker's,
    signed features included (heavy rows are cut into segments here too)."""
    n, rowptr, colidx, _ = wl.degree_ladder_graph(LADDER, seed=dim)
    q = (np.random.default_rng(dim).standard_normal((n, dim)) - 1.0).astype(np.float32)
    ref = oracle.aggregate(oracle.SAGE_MAX, rowptr, colidx, q)
    got, got16 = run_gpu(oracle.SAGE_MAX, rowptr, colidx, q, ld=ld)
    np.testing.assert_array_equal(got, ref)
    np.testing.assert_array_equal(got16[:, :got.shape[1]],
                                  torch.from_numpy(got).to(torch.bfloat16).float().numpy())
    only, _ = run_gpu(oracle.SAGE_MAX, rowptr, colidx, q, ld=ld, concat_self=False)
    np.testing.assert_array_equal(only, ref[:, dim:])


def test_max_pooling_on_a_power_law_graph_and_edgeless_rows():
    w = wl.make_config(5, scale=0.01)
    ref = oracle.aggregate(oracle.SAGE_MAX, w.rowptr, w.colidx, w.features)
    got, _ = run_gpu(oracle.SAGE_MAX, w.rowptr, w.colidx, w.features)
    np.testing.assert_array_equal(got, ref)
    rowptr = np.zeros(6, dtype=np.int64)
    q = np.random.default_rng(0).standard_normal((5, 7)).astype(np.float32)
    got, _ = run_gpu(oracle.SAGE_MAX, rowptr, np.zeros(0, dtype=np.int32), q)
    np.testing.assert_array_equal(got, np.concatenate([q, np.zeros_like(q)], 1))


def test_sage_mean_only_without_concat():
    rowptr, colidx = wl.random_small_graph(200, 900, seed=2)
    q = np.random.default_rng(2).standard_normal((200, 36)).astype(np.float32)
    ref = oracle.aggregate(oracle.SAGE_MEAN, rowptr, colidx, q)[:, 36:]
    got, _ = run_gpu(oracle.SAGE_MEAN, rowptr, colidx, q, concat_self=False)
    assert_rows_close(got, ref)


def test_results_are_bitwise_repeatable():
    w = wl.make_config(5, scale=0.01)
    a, _ = run_gpu(oracle.GCN, w.rowptr, w.colidx, w.features)
    b, _ = run_gpu(oracle.GCN, w.rowptr, w.colidx, w.features)
    np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("idx,scale", [(1, 1.0), (2, 1.0), (4, 0.02), (5, 0.02)])
def test_configs_first_round_aggregation(idx, scale):
    w = wl.make_config(idx, scale=scale)
    ref = oracle.aggregate(w.aggr, w.rowptr, w.colidx, w.features)
    got, _ = run_gpu(w.aggr, w.rowptr, w.colidx, w.features)
    assert_rows_close(got, ref, what=w.name)
    ld = (w.d0 + 31) // 32 * 32                      # the padded layout the K-round driver uses
    got, _ = run_gpu(w.aggr, w.rowptr, w.colidx, w.features, ld=ld)
    assert_rows_close(got, ref, what=w.name + " padded")


# ------------------------------------------------------------------ GAT
def gat_case(n, n_und, heads, dh, seed, slope=0.2, self_loop=1):
    rng = np.random.default_rng(seed)
    rowptr, colidx = wl.random_small_graph(n, n_und, seed=seed)
    p = rng.standard_normal((n, heads * dh)).astype(np.float32)
    if heads * dh < 16:      # few columns: keep the weighted sums from cancelling (see the ladder test)
        p = np.abs(p) + 0.5
    gat = dict(heads=heads, head_dim=dh, a_src=rng.standard_normal((heads, dh)).astype(np.float32),
               a_dst=rng.standard_normal((heads, dh)).astype(np.float32), negative_slope=slope,
               add_self_loop=self_loop)
    return rowptr, colidx, p, gat


def gat_gpu(rowptr, colidx, p, gat, ld=None):
    g = dict(gat)
    g["a_src"], g["a_dst"] = torch.from_numpy(gat["a_src"]), torch.from_numpy(gat["a_dst"])
    return run_gpu(oracle.GAT, rowptr, colidx, p, ld=ld, gat=g)


@pytest.mark.parametrize("heads,dh", [(1, 1), (1, 7), (4, 16), (2, 32), (8, 8), (3, 5), (8, 32)])
@pytest.mark.parametrize("self_loop", [0, 1])
def test_gat_random_graphs(heads, dh, self_loop):
    rowptr, colidx, p, gat = gat_case(150, 700, heads, dh, seed=heads * 100 + dh, self_loop=self_loop)
    ref = oracle.aggregate(oracle.GAT, rowptr, colidx, p, gat=gat)
    got, _ = gat_gpu(rowptr, colidx, p, gat)
    assert_rows_close(got, ref, what="gat %dx%d" % (heads, dh))


@pytest.mark.parametrize("heads,dh", [(4, 16), (8, 32), (1, 7)])
def test_gat_long_rows_isolated_nodes_and_large_scores(heads, dh):
    """Rows on both sides of the 128-entry mark, from which a whole block takes a row and merges the
    soft-max states of its eight warps (some of them without a trip below 256 entries)."""
    n, rowptr, colidx, _ = wl.degree_ladder_graph([0, 1, 31, 32, 33, 126, 127, 128, 129, 160, 255, 256, 257, 700, 3000],
                                                  seed=5)
    rng = np.random.default_rng(5)
    p = (rng.standard_normal((n, heads * dh)) * 3).astype(np.float32)
    if heads * dh < 16:
        p = np.abs(p) + 0.5
    for self_loop in (0, 1):
        gat = dict(heads=heads, head_dim=dh, a_src=(rng.standard_normal((heads, dh)) * 2).astype(np.float32),
                   a_dst=(rng.standard_normal((heads, dh)) * 2).astype(np.float32), negative_slope=0.2,
                   add_self_loop=self_loop)
        ref = oracle.aggregate(oracle.GAT, rowptr, colidx, p, gat=gat)
        got, _ = gat_gpu(rowptr, colidx, p, gat, ld=(heads * dh + 31) // 32 * 32 + 32)
        assert_rows_close(got, ref, what="gat ladder self=%d" % self_loop)
        again, _ = gat_gpu(rowptr, colidx, p, gat, ld=(heads * dh + 31) // 32 * 32 + 32)
        np.testing.assert_array_equal(again, got)        # repeatable bit for bit


def test_gat_config3_projected_input():
    w = wl.make_config(3)
    ws = wl.initial_weights(w)[0]
    rng = np.random.default_rng(1)
    p = (w.features @ ws["w_att"]).astype(np.float32)
    gat = dict(heads=4, head_dim=16, a_src=ws["a_src"], a_dst=ws["a_dst"], negative_slope=0.2, add_self_loop=1)
    ref = oracle.aggregate(oracle.GAT, w.rowptr, w.colidx, p, gat=gat)
    got, _ = gat_gpu(w.rowptr, w.colidx, p, gat)
    assert_rows_close(got, ref, what=w.name)


def ladder_in_a_large_graph(n, seed):
    """The degree ladder (hubs of every bin, isolated nodes) embedded in a graph of n nodes whose
    other nodes have a few random neighbours; node ids shuffled."""
    rng = np.random.default_rng(seed)
    edges = []
    nxt = len(LADDER)
    for h, d in enumerate(LADDER):
        edges.append(np.stack([np.full(d, h, dtype=np.int64), np.arange(nxt, nxt + d, dtype=np.int64)], axis=1))
        nxt += d
    assert nxt + 16 < n
    rest = rng.integers(nxt + 8, n, size=(3 * n, 2))          # nodes nxt .. nxt+7 stay isolated
    e = np.concatenate(edges + [rest])
    perm = rng.permutation(n)
    return wl.csr_from_edge_list(n, perm[e])


@pytest.mark.parametrize("aggr,n,dim", [(oracle.SAGE_MEAN, 120000, 850), (oracle.GCN, 170000, 602),
                                        (oracle.SAGE_MEAN, 300000, 340), (oracle.GCN, 300000, 342),
                                        (oracle.SAGE_MAX, 170000, 600)])
def test_matrices_beyond_the_cache_take_the_column_slab_variant(aggr, n, dim):
    """A feature matrix of 200 MB or more is aggregated slab of columns by slab of columns (32, 16
    or 8 vectors per slab, by the number of rows): same tolerance, every degree bin, ragged last slab."""
    rowptr, colidx = ladder_in_a_large_graph(n, seed=dim)
    rng = np.random.default_rng(dim)
    q = rng.standard_normal((n, dim)).astype(np.float32)
    if aggr != oracle.SAGE_MAX:
        q = np.abs(q) + 0.5
    ld = (dim + 3) // 4 * 4
    ref = oracle.aggregate(aggr, rowptr, colidx, q)
    got, got16 = run_gpu(aggr, rowptr, colidx, q, ld=ld)
    if aggr == oracle.SAGE_MAX:
        np.testing.assert_array_equal(got, ref)
    else:
        assert_rows_close(got, ref, what="fp32 out")
    np.testing.assert_array_equal(got16[:, :got.shape[1]], torch.from_numpy(got).to(torch.bfloat16).float().numpy())
    again, _ = run_gpu(aggr, rowptr, colidx, q, ld=ld)
    np.testing.assert_array_equal(again, got)                 # repeatable bit for bit
