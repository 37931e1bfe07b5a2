"""The K-round lazy-message-passing loop of the CPU checker (Section 3.1)."""
import numpy as np

import oracle
from paper_2302_13053_b200 import workloads as wl


def run(w, R, **kw):
    gat = dict(heads=w.heads, head_dim=w.head_dim, negative_slope=w.negative_slope,
               add_self_loop=1) if w.aggr == wl.GAT else None
    return oracle.lmp_train(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features,
                            w.labels, w.train_idx, w.val_idx, w.test_idx, wl.initial_weights(w), gat=gat,
                            part=w.part, n_parts=w.n_parts, **kw)


def test_loop_issues_k_aggregations_and_k_times_r_steps():
    for idx, scale in ((1, 0.2), (2, 0.05), (3, 0.05)):
        w = wl.make_config(idx, scale=scale)
        rep = run(w, 4)
        assert rep["n_aggregations"] == w.K          # one message-passing round per layer
        assert rep["n_steps"] == w.K * 4
        dims = [r["x"].shape[1] for r in rep["rounds"]]
        assert dims == [d["d_in"] for d in w.round_dims()]
        assert rep["rounds"][-1]["logits"].shape == (w.n_nodes, w.n_classes)
        for r in rep["rounds"][:-1]:
            assert r["q_out"].shape == (w.n_nodes, w.hidden) and (r["q_out"] >= 0).all()


def test_best_validation_iterate_is_the_earliest_maximum():
    w = wl.make_config(1, scale=0.3)
    rep = run(w, 12)
    for r in rep["rounds"]:
        assert r["best_iter"] == int(np.argmax(r["val_correct"])) + 1
        assert r["best_val_correct"] == r["val_correct"].max()


def test_more_rounds_help_when_features_are_weak_and_homophily_is_strong():
    """Qualitative claim of Sections 3.1 / 4.2: a further hop adds signal."""
    rng = np.random.default_rng(0)
    n, o = 600, 3
    labels = rng.integers(0, o, n).astype(np.int32)
    rowptr, colidx = wl.random_graph(rng, n, 2400, labels, None, 0.9, None)
    feats = (0.35 * np.eye(o)[labels] + rng.standard_normal((n, o))).astype(np.float32)
    tr, va, te = wl._split_fraction(rng, n, 0.3, 0.2)
    acc = {}
    for K in (1, 3):
        ws = []
        d = o
        for m in range(K):
            hid = 16 if m < K - 1 else 0
            r2 = np.random.default_rng(m)
            w = dict(w1=wl.glorot(r2, d, hid or o), b1=np.zeros(hid or o, dtype=np.float32))
            if hid:
                w["w2"], w["b2"] = wl.glorot(r2, hid, o), np.zeros(o, dtype=np.float32)
            ws.append(w)
            d = hid
        rep = oracle.lmp_train(oracle.GCN, K, 60, 16, o, 0.02, rowptr, colidx, feats, labels, tr, va, te, ws,
                               round_bf16=False)
        acc[K] = rep["test_acc"]
    assert acc[3] > acc[1] + 0.05, acc


def test_forced_iterate_hook_keeps_the_named_iterate():
    w = wl.make_config(1, scale=0.3)
    free = run(w, 8)
    same = run(w, 8, forced_best_iter=[r["best_iter"] for r in free["rounds"]])
    np.testing.assert_array_equal(free["rounds"][-1]["logits"], same["rounds"][-1]["logits"])
    other = run(w, 8, forced_best_iter=[8, 8, 8])
    assert [r["best_iter"] for r in other["rounds"]] == [8, 8, 8]
    assert other["rounds"][0]["test_correct_best"] == other["rounds"][0]["test_correct_last"]


def test_forced_weights_hook_feeds_the_given_weights_forward_and_leaves_the_training_alone():
    w = wl.make_config(2, scale=0.05)
    free = run(w, 6, eval_every=6)
    own = [r["model"].theta for r in free["rounds"]]
    same = run(w, 6, eval_every=6, forced_theta=own)
    np.testing.assert_array_equal(free["rounds"][-1]["logits"], same["rounds"][-1]["logits"])
    # other weights in round 1: round 1's own training is untouched, everything downstream moves
    bumped = [t.copy() for t in own]
    bumped[0] = bumped[0] * 1.5
    other = run(w, 6, eval_every=6, forced_theta=bumped)
    np.testing.assert_array_equal(other["rounds"][0]["losses"], free["rounds"][0]["losses"])
    np.testing.assert_array_equal(other["rounds"][0]["own_model"].theta, own[0])
    np.testing.assert_array_equal(other["rounds"][0]["model"].theta, bumped[0])
    assert np.abs(other["rounds"][1]["x"] - free["rounds"][1]["x"]).max() > 1e-3
    assert abs(other["rounds"][1]["losses"][0] - free["rounds"][1]["losses"][0]) > 1e-6


def test_trainable_attention_loop_retrains_the_aggregator_every_iteration():
    """RetexoGAT with its aggregator trained (Section 2.2 / 3.1): K x R local aggregations instead of K, the
    attention parameters move, and the first iteration's loss equals the frozen-attention run's (same
    initial parameters, same forward)."""
    w = wl.make_config(3, scale=0.03)
    gat = dict(heads=w.heads, head_dim=w.head_dim, negative_slope=w.negative_slope, add_self_loop=1)
    ws = wl.initial_weights(w)
    args = (w.aggr, w.K, 5, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels, w.train_idx,
            w.val_idx, w.test_idx, ws)
    frozen = oracle.lmp_train(*args, gat=gat)
    trained = oracle.lmp_train(*args, gat=gat, train_attention=True)
    assert frozen["n_aggregations"] == w.K and trained["n_aggregations"] == w.K * 5
    assert abs(trained["rounds"][0]["losses"][0] - frozen["rounds"][0]["losses"][0]) < 1e-9
    assert abs(trained["rounds"][0]["losses"][-1] - frozen["rounds"][0]["losses"][-1]) > 1e-7
    layer = trained["rounds"][0]["layer"]
    w_att, a_src, a_dst = layer.parts()
    assert np.abs(w_att - ws[0]["w_att"]).max() > 1e-4 and np.abs(a_src - ws[0]["a_src"]).max() > 1e-4
    assert trained["rounds"][-1]["logits"].shape == (w.n_nodes, w.n_classes)
    # the forcing hooks hand the given attention parameters on
    same = oracle.lmp_train(*args, gat=gat, train_attention=True,
                            forced_att=[r["layer"].att for r in trained["rounds"]],
                            forced_theta=[r["model"].theta for r in trained["rounds"]])
    np.testing.assert_array_equal(same["rounds"][-1]["logits"], trained["rounds"][-1]["logits"])
