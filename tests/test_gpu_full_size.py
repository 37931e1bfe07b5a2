"""Parity at the full sizes of the two large configurations, in the launch configuration the
benchmark times (128-byte feature rows, bf16 model input written by the aggregation kernel,
transposed train batch with its row of ones): outputs the CPU checker can compute one by one
are sampled (destination rows incl. the longest ones; one whole training iteration), counts
are compared exactly."""
import numpy as np
import pytest
import torch

import oracle
from paper_2302_13053_b200 import workloads as wl
from gpu_util import assert_rows_close, dev

pytestmark = pytest.mark.gpu

_cache = {}


def config(idx):
    if idx not in _cache:
        _cache.clear()                      # one large graph in host memory at a time
        _cache[idx] = wl.make_config(idx)
    return _cache[idx]


def sampled_rows(w, k=256):
    deg = np.diff(w.rowptr)
    rng = np.random.default_rng(1)
    rows = np.concatenate([np.argsort(deg)[-24:], np.argsort(deg)[:8], rng.choice(w.n_nodes, k, replace=False)])
    return np.unique(rows)


@pytest.mark.parametrize("idx", [4, 5])
def test_round_one_aggregation_on_sampled_rows(idx):
    from paper_2302_13053_b200 import binding as B
    w = config(idx)
    n, d = w.n_nodes, w.d0
    ld = (d + 31) // 32 * 32
    q = torch.zeros((n, ld), dtype=torch.float32, device="cuda")
    q[:, :d] = dev(w.features)
    rp, ci = dev(w.rowptr), dev(w.colidx)
    assert B.retexo_validate_csr(rp, ci) == (0, -1)
    out, out16 = B.retexo_aggregate(w.aggr, rp, ci, q, dim=d, want_f32=True, want_bf16=True)
    torch.cuda.synchronize()
    rows = sampled_rows(w)
    ref = oracle.aggregate(w.aggr, w.rowptr, w.colidx, w.features, rows=rows)
    got = out[torch.from_numpy(rows).cuda()].cpu().numpy()
    assert_rows_close(got, ref, what=w.name)
    width = ref.shape[1]
    assert torch.equal(out16[:, :width], out.to(torch.bfloat16))          # the bf16 copy is the same result rounded once
    # linearity of the aggregation as a whole-matrix property: A(2q) == 2 A(q) bit for bit
    out2, _ = B.retexo_aggregate(w.aggr, rp, ci, q * 2, dim=d)
    assert torch.equal(out2, out * 2)


@pytest.mark.parametrize("idx", [4, 5])
def test_cross_partition_counts_exact(idx):
    from paper_2302_13053_b200 import binding as B
    w = config(idx)
    dims = [r["rep_dim"] for r in w.round_dims()]
    ref = oracle.cross_partition(w.rowptr, w.colidx, w.part, w.n_parts, dims, 4)
    got = B.retexo_cross_partition_bytes(dev(w.rowptr), dev(w.colidx), dev(w.part), w.n_parts, dims, 4)
    for k in ("cross_edges", "boundary_pairs", "bytes_total", "dv_lazy_lt"):
        assert got[k] == ref[k], k
    np.testing.assert_array_equal(got["bytes_per_round"], ref["bytes_per_round"])
    np.testing.assert_array_equal(got["send_per_part"], ref["send_per_part"])
    np.testing.assert_array_equal(got["recv_per_part"], ref["recv_per_part"])
    if w.n_parts == w.n_nodes:
        assert got["boundary_pairs"] == w.n_edges           # node-level partition: every edge is a message


def test_one_training_iteration_of_the_reddit_shaped_round_one():
    from paper_2302_13053_b200 import binding as B
    w = config(4)
    n, d = w.n_nodes, w.d0
    ld = (d + 31) // 32 * 32
    q = torch.zeros((n, ld), dtype=torch.float32, device="cuda")
    q[:, :d] = dev(w.features)
    _, x16 = B.retexo_aggregate(w.aggr, dev(w.rowptr), dev(w.colidx), q, dim=d, want_f32=False, want_bf16=True)
    tr = dev(w.train_idx)
    xtr, _ = B.retexo_pack_rows(x16, tr, dim=2 * d, ones=True)
    y = w.labels[w.train_idx]
    wt = wl.initial_weights(w)[0]
    gpu = B.Mlp(2 * d, w.hidden, w.n_classes, wt["w1"], wt["b1"], wt["w2"], wt["b2"], lr=w.lr)
    ref = oracle.Mlp(2 * d, w.hidden, w.n_classes, wt["w1"], wt["b1"], wt["w2"], wt["b2"], lr=w.lr, round_bf16=True)
    x_host = xtr[:, :2 * d].float().cpu().numpy()           # the checker sees the very batch the GPU trains on
    given = ref.copy()
    rl, rg = ref.train_step(x_host, y, return_grad=True)
    gl, gg = B.retexo_mlp_train_step(gpu, xtr, dev(y), x_has_ones=True, return_grad=True)
    assert abs(gl.item() - rl) <= 2e-4 * max(1.0, abs(rl)), (gl.item(), rl)
    gg = gg.cpu().numpy().astype(np.float64)
    err, scale = np.abs(gg - rg), np.abs(rg).max()
    assert err.max() <= 5e-3 * scale + 1e-7, (err.max(), scale)
    assert np.median(err) <= 2e-5 * scale
    given.apply_update(gg)
    assert np.abs(gpu.theta.cpu().numpy() - given.theta).max() <= 2e-6 * max(1.0, np.abs(given.theta).max())


def round_inputs(w, m):
    """Model input of round m at full size in the benchmark's layout: round 1 aggregates the features,
    later rounds a seeded stand-in for the previous round's output (non-negative, as a ReLU leaves it)."""
    from paper_2302_13053_b200 import binding as B
    rd = w.round_dims()[m - 1]
    n, d = w.n_nodes, rd["rep_dim"]
    ld = (d + 31) // 32 * 32
    q = torch.zeros((n, ld), dtype=torch.float32, device="cuda")
    if m == 1:
        q[:, :d] = dev(w.features)
    else:
        g = torch.Generator(device="cuda")
        g.manual_seed(100 * m + d)
        q[:, :d] = torch.randn((n, d), generator=g, device="cuda").clamp_(min=0)
    _, x16 = B.retexo_aggregate(w.aggr, dev(w.rowptr), dev(w.colidx), q, dim=d, want_f32=False, want_bf16=True)
    return rd, x16


@pytest.mark.parametrize("idx,m,ln", [(4, 2, False), (4, 3, False), (5, 1, False), (5, 2, False), (5, 3, False),
                                      (4, 1, True), (5, 2, True)])
def test_one_training_iteration_and_emission_at_full_size(idx, m, ln):
    """The shapes of the two large configurations that the first-round test above does not cover: one
    whole training iteration on all train rows (loss, gradient, update) and the emission of sampled
    rows, each against the checker on the very batch the GPU works on."""
    from paper_2302_13053_b200 import binding as B
    from gpu_util import assert_logits_close
    w = config(idx)
    rd, x16 = round_inputs(w, m)
    d_in, H, O = rd["d_in"], rd["hidden"], w.n_classes
    tr = dev(w.train_idx)
    xtr, _ = B.retexo_pack_rows(x16, tr, dim=d_in, ones=True)
    y = w.labels[w.train_idx]
    wt = wl.initial_weights(w)[m - 1]
    # (ln: the same with layer normalisation inside f_theta, gamma = 1 and beta = 0 to start with)
    gpu = B.Mlp(d_in, H, O, wt["w1"], wt["b1"], wt.get("w2"), wt.get("b2"), lr=w.lr, layer_norm=ln)
    ref = oracle.Mlp(d_in, H, O, wt["w1"], wt["b1"], wt.get("w2"), wt.get("b2"), lr=w.lr, round_bf16=True,
                     layer_norm=ln)
    x_host = xtr[:, :d_in].float().cpu().numpy()
    given = ref.copy()
    rl, rg = ref.train_step(x_host, y, return_grad=True)
    gl, gg = B.retexo_mlp_train_step(gpu, xtr, dev(y), x_has_ones=True, return_grad=True)
    assert abs(gl.item() - rl) <= 2e-4 * max(1.0, abs(rl)), (gl.item(), rl)
    gg = gg.cpu().numpy().astype(np.float64)
    err, scale = np.abs(gg - rg), np.abs(rg).max()
    assert err.max() <= 5e-3 * scale + 1e-7, (err.max(), scale)
    assert np.median(err) <= 2e-5 * scale
    given.apply_update(gg)
    assert np.abs(gpu.theta.cpu().numpy() - given.theta).max() <= 2e-6 * max(1.0, np.abs(given.theta).max())
    del xtr, x_host
    # emission over all rows with the updated weights, as the K-round run calls it; 4096 sampled rows checked
    rows = np.sort(np.random.default_rng(m).choice(w.n_nodes, 4096, replace=False))
    out = B.retexo_embed(gpu, x16, want_hidden=H > 0, want_logits=True, want_pred=True)
    sel = torch.from_numpy(rows).cuda()
    xs = x16[sel][:, :d_in].float().cpu().numpy()
    ref.theta = gpu.theta.cpu().numpy().astype(np.float64)
    r = ref.embed(xs, want_hidden=H > 0)
    lg = out["logits"][sel].cpu().numpy()
    assert_logits_close(lg, r["logits"], rel=5e-3, what="vs bf16-operand checker")
    exact = ref.copy()
    exact.round_bf16 = False
    assert_logits_close(lg, exact.embed(xs)["logits"], rel=2e-2, what="vs unrounded checker")
    if H > 0:
        assert_logits_close(out["hidden"][sel].cpu().numpy(), r["hidden"], rel=1e-3, what="hidden")
    srt = np.sort(r["logits"], axis=1)
    clear = (srt[:, -1] - srt[:, -2]) > 1e-2 * np.abs(r["logits"]).max(axis=1)
    np.testing.assert_array_equal(out["pred"][sel].cpu().numpy()[clear], r["pred"][clear])


def test_whole_run_properties_on_the_products_shaped_graph():
    """At a size the checker cannot train on in reasonable time: the K-round run must be repeatable
    bit for bit, count every edge as a message, reduce the loss in every round, and beat chance."""
    from paper_2302_13053_b200 import binding as B
    w = config(5)
    ws = wl.initial_weights(w)
    res = []
    for _ in range(2):
        prob = B.LmpProblem(w.aggr, w.K, 30, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                            w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts)
        B.retexo_lmp_train(prob)
        torch.cuda.synchronize()
        res.append(prob.results())
        del prob
        torch.cuda.empty_cache()
    a, b = res
    np.testing.assert_array_equal(a["loss_history"], b["loss_history"])
    np.testing.assert_array_equal(a["final_logits"], b["final_logits"])
    assert a["counts"]["boundary_pairs"] == w.n_edges == a["counts"]["cross_edges"]
    assert np.isfinite(a["loss_history"]).all()
    assert (a["loss_history"][:, -1] < a["loss_history"][:, 0]).all()
    assert a["test_acc"] > 3.0 / w.n_classes
    for m in range(w.K):
        v = a["val_correct"][m].astype(np.int64)
        assert a["best_iter"][m] == int(np.argmax(v)) + 1


def test_gat_aggregation_on_the_products_shaped_graph():
    """The fused GAT kernel far outside L2 (2.4 M rows of 64 columns, 124 M entries, tens of thousands
    of rows long enough to be taken by whole blocks): sampled destination rows, the longest included,
    against the checker; two runs give the same bits although the list of long rows is built with
    atomics in arbitrary order."""
    from paper_2302_13053_b200 import binding as B
    w = config(5)
    heads, dh = 4, 16
    rng = np.random.default_rng(11)
    p_host = rng.standard_normal((w.n_nodes, heads * dh), dtype=np.float32)
    gat = dict(heads=heads, head_dim=dh, a_src=(rng.standard_normal((heads, dh)) * 0.5).astype(np.float32),
               a_dst=(rng.standard_normal((heads, dh)) * 0.5).astype(np.float32), negative_slope=0.2, add_self_loop=1)
    g = dict(gat)
    g["a_src"], g["a_dst"] = torch.from_numpy(gat["a_src"]), torch.from_numpy(gat["a_dst"])
    rp, ci, p = dev(w.rowptr), dev(w.colidx), dev(p_host)
    out, _ = B.retexo_aggregate(oracle.GAT, rp, ci, p, dim=heads * dh, gat=g, want_f32=True)
    again, _ = B.retexo_aggregate(oracle.GAT, rp, ci, p, dim=heads * dh, gat=g, want_f32=True)
    torch.cuda.synchronize()
    assert torch.equal(out, again)
    rows = sampled_rows(w)
    assert (np.diff(w.rowptr)[rows] >= 128).sum() >= 24 and (np.diff(w.rowptr)[rows] < 127).sum() >= 8
    ref = oracle.aggregate(oracle.GAT, w.rowptr, w.colidx, p_host, rows=rows, gat=gat)
    got = out[torch.from_numpy(rows).cuda()].cpu().numpy()
    assert_rows_close(got, ref, what="gat on " + w.name)
