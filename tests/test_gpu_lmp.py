"""The K-round loop on the device (retexo_lmp_train) against the CPU checker's
loop: counts exact; the emitted logits element by element against the checker's
aggregate / embed chain on the kept weights; loss curves, validation and test
counts round by round from the same start; test accuracy within 0.5 points."""
import numpy as np
import pytest
import torch

import oracle
from paper_2302_13053_b200 import workloads as wl
from gpu_util import assert_logits_close

pytestmark = pytest.mark.gpu

# Loss curves of a round that starts from the same weights and the same inputs on both sides: what is left
# is fp32-versus-fp64 arithmetic carried through R optimiser steps.
CURVE_TOL = 2e-2


def run_both(w, R, host=False, eval_every=1, force=False, freeze=False):
    from paper_2302_13053_b200 import binding as B
    ws = wl.initial_weights(w)
    gat = dict(heads=w.heads, head_dim=w.head_dim, negative_slope=w.negative_slope,
               add_self_loop=1) if w.aggr == wl.GAT else None
    prob = B.LmpProblem(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                        w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts, heads=w.heads,
                        head_dim=w.head_dim, negative_slope=w.negative_slope, eval_every=eval_every, host=host,
                        freeze_attention=freeze)
    B.retexo_lmp_train(prob)
    torch.cuda.synchronize()
    got = prob.results()
    # force=True: the checker keeps the iterate the GPU kept (an arg-max over floating-point
    # validation counts), so that everything downstream of that choice can be compared; the
    # GPU's choice itself is checked against its own validation curve by the caller.
    ref = oracle.lmp_train(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                           w.train_idx, w.val_idx, w.test_idx, ws, gat=gat, part=w.part, n_parts=w.n_parts,
                           eval_every=eval_every, forced_best_iter=list(got["best_iter"]) if force else None,
                           train_attention=w.aggr == wl.GAT and not freeze)
    return ref, got


def check_counts(ref, got):
    for k in ("cross_edges", "boundary_pairs", "bytes_total", "dv_lazy_lt"):
        assert got["counts"][k] == ref["counts"][k], k
    np.testing.assert_array_equal(got["counts"]["bytes_per_round"], ref["counts"]["bytes_per_round"])


def unpack_att(att, d, heads, dh):
    hd = heads * dh
    return att[:d * hd].reshape(d, hd), att[d * hd:d * hd + hd].reshape(heads, dh), att[d * hd + hd:].reshape(heads, dh)


def oracle_chain(w, ws, thetas, round_bf16, atts=None):
    """What the K-round run emits, recomputed by the checker without any training: the raw features
    go through aggregate -> per-node model with the given weights -> aggregate -> ... (Section 3.1:
    the kept layer's output representations are the next round's inputs, the classifier dropped)."""
    q = w.features
    out = None
    for m, (rd, wt) in enumerate(zip(w.round_dims(), ws)):
        if w.aggr == wl.GAT:
            hd = w.heads * w.head_dim
            w_att, a_src, a_dst = wt["w_att"], wt["a_src"], wt["a_dst"]
            if atts is not None:      # the aggregator parameters the run kept (trained with the round's model)
                w_att, a_src, a_dst = unpack_att(atts[m], q.shape[1], w.heads, w.head_dim)
            proj = oracle.Mlp(q.shape[1], 0, hd, w_att, np.zeros(hd), round_bf16=round_bf16)
            g = dict(heads=w.heads, head_dim=w.head_dim, negative_slope=w.negative_slope, add_self_loop=1,
                     a_src=a_src, a_dst=a_dst)
            x = oracle.aggregate(oracle.GAT, w.rowptr, w.colidx, proj.embed(q)["logits"], gat=g)
        else:
            x = oracle.aggregate(w.aggr, w.rowptr, w.colidx, q)
        model = oracle.Mlp(rd["d_in"], rd["hidden"], w.n_classes, wt["w1"], wt["b1"], wt.get("w2"), wt.get("b2"),
                           round_bf16=round_bf16)
        model.theta = np.ascontiguousarray(thetas[m], dtype=np.float64)
        if rd["hidden"] > 0:
            q = model.embed(x, want_hidden=True, want_logits=False)["hidden"]
        else:
            out = model.embed(x, want_logits=True)
    return out["logits"], out["pred"]


@pytest.mark.parametrize("idx,scale,R,freeze", [(1, 1.0, 30, False), (2, 1.0, 25, False), (3, 1.0, 30, False),
                                                (3, 1.0, 30, True), (4, 0.1, 10, False), (5, 0.05, 10, False)])
def test_emitted_logits_match_the_checkers_chain_on_the_kept_weights(idx, scale, R, freeze):
    """The weights the run kept in every round, pushed through the checker's own aggregate / embed
    chain from the raw features, must reproduce the logits the run emits element by element at the
    stated bf16 tolerance (no training happens on the checker's side, so nothing can drift)."""
    from paper_2302_13053_b200 import binding as B
    w = wl.make_config(idx, scale=scale)
    ws = wl.initial_weights(w)
    prob = B.LmpProblem(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                        w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts, heads=w.heads,
                        head_dim=w.head_dim, negative_slope=w.negative_slope, freeze_attention=freeze)
    B.retexo_lmp_train(prob)
    torch.cuda.synchronize()
    got = prob.results()
    assert all(np.abs(t).max() > 0 for t in got["theta_best"])
    atts = None
    if w.aggr == wl.GAT:
        given = [B.pack_gat(wt) for wt in ws]
        moved = [float(np.abs(a - b).max()) for a, b in zip(got["gat_best"], given)]
        assert all(d == 0 for d in moved) if freeze else all(d > 1e-4 for d in moved), moved
        atts = got["gat_best"]
    lg = got["final_logits"]
    np.testing.assert_array_equal(got["final_pred"], lg.argmax(1))
    for round_bf16 in (True, False):
        rl, rp = oracle_chain(w, ws, got["theta_best"], round_bf16, atts=atts)
        # Against the checker under the same operand-rounding contract: the stated 2e-2.  Against the
        # checker that rounds nothing, each of the K per-node models in the chain and, for GAT, each of
        # the K projections adds its own bf16 operand rounding on top of what it inherits, so the stated
        # 2e-2 (for one bf16-input model) is allowed once per rounded stage.
        stages = w.K * (2 if w.aggr == wl.GAT else 1)
        rel = 2e-2 if round_bf16 else 2e-2 * stages
        assert_logits_close(lg, rl, rel=rel, what="%s, checker %s operand rounding" % (
            w.name, "with" if round_bf16 else "without"))
        srt = np.sort(rl, axis=1)
        rms = float(np.sqrt(np.mean(rl.astype(np.float64) ** 2)))
        clear = (srt[:, -1] - srt[:, -2]) > 2 * rel * np.maximum(np.abs(rl).max(axis=1), rms)
        np.testing.assert_array_equal(got["final_pred"][clear], rp[clear])
        hits = int((rp[w.test_idx] == w.labels[w.test_idx]).sum())
        unclear = int((~clear[w.test_idx]).sum())
        assert abs(int(got["test_correct"][-1]) - hits) <= unclear


@pytest.mark.parametrize("idx,scale,R,freeze", [(1, 1.0, 30, False), (2, 1.0, 25, False), (3, 1.0, 30, False),
                                                (3, 1.0, 30, True), (4, 0.05, 20, False), (5, 0.01, 20, False)])
def test_every_round_tracks_the_checker_from_the_same_start(idx, scale, R, freeze):
    """Validation only at the last iteration, so both sides keep the last iterate; the checker hands
    the GPU's kept weights to the next round (`forced_theta`), so every round trains on the same
    inputs on both sides, each at the configuration's own learning rate, and loss curves, validation
    and test counts can be compared round by round."""
    check_rounds_from_the_same_start(wl.make_config(idx, scale=scale), R, freeze=freeze)


def test_max_pooling_rounds_track_the_checker():
    """The K-round loop with the max-pooling aggregator of Section 2.2 in place of the mean."""
    w = wl.make_config(2)
    w.aggr = wl.SAGE_MAX
    check_rounds_from_the_same_start(w, 25)


def check_rounds_from_the_same_start(w, R, freeze=False):
    from paper_2302_13053_b200 import binding as B
    ws = wl.initial_weights(w)
    gat = dict(heads=w.heads, head_dim=w.head_dim, negative_slope=w.negative_slope,
               add_self_loop=1) if w.aggr == wl.GAT else None
    prob = B.LmpProblem(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                        w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts, heads=w.heads,
                        head_dim=w.head_dim, negative_slope=w.negative_slope, eval_every=R, freeze_attention=freeze)
    B.retexo_lmp_train(prob)
    torch.cuda.synchronize()
    got = prob.results()
    trained = w.aggr == wl.GAT and not freeze      # the round trains the aggregator too: its kept parameters are handed over as well
    ref = oracle.lmp_train(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                           w.train_idx, w.val_idx, w.test_idx, ws, gat=gat, part=w.part, n_parts=w.n_parts,
                           eval_every=R, forced_theta=got["theta_best"], train_attention=trained,
                           forced_att=got["gat_best"] if trained else None)
    check_counts(ref, got)
    assert got["status"] == 0                       # written by the run: no bounded device-side wait ran out
    n_val, n_test = len(w.val_idx), len(w.test_idx)
    for m, rd in enumerate(ref["rounds"]):
        gl, rl = got["loss_history"][m], rd["losses"]
        assert abs(gl[0] - rl[0]) <= 1e-3 * max(1.0, rl[0]), (m, gl[0], rl[0])     # same weights, same inputs
        assert np.abs(gl - rl).max() <= CURVE_TOL * max(1.0, rl.max()), (m, np.abs(gl - rl).max(), rl.max())
        assert got["best_iter"][m] == R == rd["best_iter"]
        assert abs(int(got["best_val_correct"][m]) - rd["best_val_correct"]) <= max(2, 0.01 * n_val)
        # the checker's own last iterate and the GPU's, both on the test rows of the same inputs
        assert abs(int(got["test_correct"][m]) - rd["test_correct_last"]) <= max(2, 0.01 * n_test)
        assert got["test_correct"][m] == got["test_correct_last"][m]
    assert abs(got["test_acc"] - ref["test_acc_last"]) <= 0.005 + 1.0 / n_test, (got["test_acc"], ref["test_acc_last"])


@pytest.mark.parametrize("idx,scale,R", [(1, 1.0, 100), (2, 1.0, 100), (3, 1.0, 100)])
def test_best_validation_runs_reach_the_checkers_accuracy(idx, scale, R):
    """Per-iteration validation with best-iterate selection, full small configurations at the
    paper's R: final test accuracy within 0.5 points of the checker's."""
    w = wl.make_config(idx, scale=scale)
    ref, got = run_both(w, R, eval_every=1, force=True)
    check_counts(ref, got)
    n_val, n_test = len(w.val_idx), len(w.test_idx)
    rd = ref["rounds"][0]
    gl = got["loss_history"][0]
    assert abs(gl[0] - rd["losses"][0]) <= 1e-3 * max(1.0, rd["losses"][0])
    for m in range(w.K):
        gv = got["val_correct"][m].astype(np.int64)
        assert got["best_iter"][m] == int(np.argmax(gv)) + 1                        # earliest best iterate
        assert got["best_val_correct"][m] == gv.max()
    gv, rv = got["val_correct"][0].astype(np.int64), rd["val_correct"]
    assert np.abs(gv - rv).max() <= max(3, 0.04 * n_val), np.abs(gv - rv).max()
    assert abs(got["test_acc"] - ref["test_acc"]) <= 0.005 + 1.0 / n_test, (got["test_acc"], ref["test_acc"])


def test_host_buffer_run_gives_the_same_bits_as_the_device_run():
    from paper_2302_13053_b200 import binding as B
    w = wl.make_config(2, scale=0.2)
    ws = wl.initial_weights(w)
    res = []
    for host in (False, True):
        prob = B.LmpProblem(w.aggr, w.K, 6, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                            w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts, host=host)
        B.retexo_lmp_train(prob)
        torch.cuda.synchronize()
        res.append(prob.results())
    np.testing.assert_array_equal(res[0]["loss_history"], res[1]["loss_history"])
    np.testing.assert_array_equal(res[0]["final_logits"], res[1]["final_logits"])
    np.testing.assert_array_equal(res[0]["val_correct"], res[1]["val_correct"])
    assert res[0]["counts"]["boundary_pairs"] == res[1]["counts"]["boundary_pairs"]


def test_eval_every_skips_validation_and_marks_the_gaps():
    w = wl.make_config(1, scale=0.3)
    ref, got = run_both(w, 10, eval_every=4)
    check_counts(ref, got)
    v = got["val_correct"][0]
    evaluated = [i for i in range(10) if v[i] != 2 ** 64 - 1]
    assert evaluated == [3, 7, 9]
    assert got["best_iter"][0] in (4, 8, 10)


def test_a_callers_own_stream_gives_the_same_bits_and_orders_later_work():
    """The run is ordered inside the stream it is given: launched on a stream of the caller's with
    work queued before and after it, it gives the same bits as on the default stream (plain
    launches and the replayed graph alike: validation every iteration, and every third one)."""
    from paper_2302_13053_b200 import binding as B
    w = wl.make_config(2, scale=0.3)
    ws = wl.initial_weights(w)
    for eval_every in (1, 3):
        res = []
        for own in (False, True):
            prob = B.LmpProblem(w.aggr, w.K, 9, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                                w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts,
                                eval_every=eval_every)
            if own:
                s = torch.cuda.Stream()
                s.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(s):
                    busy = torch.randn(4096, 4096, device="cuda") @ torch.randn(4096, 4096, device="cuda")   # queued first
                    B.retexo_lmp_train(prob)
                    after = prob.loss_history.clone()                          # queued behind the run, same stream
                s.synchronize()
                assert torch.isfinite(busy).all()
                res.append((prob.results(), after.cpu().numpy()))
            else:
                B.retexo_lmp_train(prob)
                torch.cuda.synchronize()
                res.append((prob.results(), None))
        a, (b, after) = res[0][0], res[1]
        np.testing.assert_array_equal(a["loss_history"], b["loss_history"])
        np.testing.assert_array_equal(a["val_correct"], b["val_correct"])
        np.testing.assert_array_equal(a["final_logits"], b["final_logits"])
        np.testing.assert_array_equal(after.reshape(b["loss_history"].shape), b["loss_history"])
