"""CUDA backward of the GAT aggregation (retexo_gat_backward) against the CPU checker: gradients with
respect to the projected rows and to both attention vectors, at the aggregation tolerance."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_rows_close, dev
from paper_2302_13053_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_case(rowptr, colidx, heads, dh, seed, active_share=0.5, self_loop=1, scale=0.5):
    from paper_2302_13053_b200 import binding as B
    n = rowptr.shape[0] - 1
    rng = np.random.default_rng(seed)
    p = rng.standard_normal((n, heads * dh)).astype(np.float32)
    gat = dict(heads=heads, head_dim=dh, negative_slope=0.2, add_self_loop=self_loop,
               a_src=(rng.standard_normal((heads, dh)) * scale).astype(np.float32),
               a_dst=(rng.standard_normal((heads, dh)) * scale).astype(np.float32))
    dz = rng.standard_normal((n, heads * dh)).astype(np.float32)
    dz[rng.random(n) >= active_share] = 0.0                      # rows outside the loss
    ref_dp, ref_as, ref_ad = oracle.gat_backward(rowptr, colidx, p, gat, dz.astype(np.float64))
    g = dict(gat)
    g["a_src"], g["a_dst"] = torch.from_numpy(gat["a_src"]), torch.from_numpy(gat["a_dst"])
    dp, dp16, da_src, da_dst = B.retexo_gat_backward(dev(rowptr.astype(np.int64)), dev(colidx.astype(np.int32)), dev(p), g,
                                                     dev(dz), want_f32=True, want_bf16=True)
    again = B.retexo_gat_backward(dev(rowptr.astype(np.int64)), dev(colidx.astype(np.int32)), dev(p), g, dev(dz))
    torch.cuda.synchronize()
    assert torch.equal(dp, again[0]) and torch.equal(da_src, again[2]) and torch.equal(da_dst, again[3])
    # per row: the gradient is a sum over the row's destinations of terms of the size of dz x alpha, so it is
    # judged like an aggregation result, against the row norm (rows that must be zero: exactly zero)
    got = dp.cpu().numpy()
    norm = np.linalg.norm(ref_dp, axis=1)
    err = np.abs(got - ref_dp).max(axis=1) if n else np.zeros(0)
    floor = 1e-5 * (np.abs(ref_dp).max() if n else 0.0)          # rows whose terms cancel are judged against the matrix
    assert np.all(err <= 2e-5 * norm + floor), float((err / (norm + floor + 1e-30)).max())
    assert np.all(got[norm == 0] == 0)
    assert torch.equal(dp16[:, :heads * dh], dp.to(torch.bfloat16))
    for got_a, ref_a in ((da_src, ref_as), (da_dst, ref_ad)):
        # sums over all nodes of products that cancel: fp32 accumulation against the largest entry
        np.testing.assert_allclose(got_a.cpu().numpy(), ref_a, rtol=0, atol=2e-5 * max(1.0, np.abs(ref_a).max()) * np.sqrt(max(n, 1)) / 10)


@pytest.mark.parametrize("heads,dh", [(4, 16), (1, 8), (8, 32), (3, 5), (2, 64)])
def test_backward_on_a_random_graph(heads, dh):
    rowptr, colidx = wl.random_small_graph(500, 4000, seed=heads)
    run_case(rowptr, colidx, heads, dh, seed=dh)


def test_backward_on_a_degree_ladder_with_hubs_and_isolated_nodes():
    n, rowptr, colidx, _ = wl.degree_ladder_graph([0, 1, 2, 31, 32, 33, 127, 128, 129, 700, 2100], seed=2)
    run_case(rowptr, colidx, 4, 16, seed=3)
    run_case(rowptr, colidx, 4, 16, seed=4, self_loop=0, active_share=1.0)


def test_backward_with_no_active_row_and_with_every_row_active():
    rowptr, colidx = wl.random_small_graph(300, 1500, seed=9)
    run_case(rowptr, colidx, 4, 16, seed=1, active_share=0.0)
    run_case(rowptr, colidx, 4, 16, seed=2, active_share=1.0, scale=2.0)


def test_backward_on_the_page_page_shaped_graph():
    w = wl.make_config(3)
    run_case(w.rowptr, w.colidx, w.heads, w.head_dim, seed=5)
