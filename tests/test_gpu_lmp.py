"""The K-round loop on the device (retexo_lmp_train) against the CPU checker's
loop: counts exact, first-iteration losses tight, loss curves and accuracy
within the stated bounds (test accuracy within 0.5 points)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2302_13053_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_both(w, R, host=False, eval_every=1):
    from paper_2302_13053_b200 import binding as B
    ws = wl.initial_weights(w)
    gat = dict(heads=w.heads, head_dim=w.head_dim, negative_slope=w.negative_slope,
               add_self_loop=1) if w.aggr == wl.GAT else None
    ref = oracle.lmp_train(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                           w.train_idx, w.val_idx, w.test_idx, ws, gat=gat, part=w.part, n_parts=w.n_parts,
                           eval_every=eval_every)
    prob = B.LmpProblem(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                        w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts, heads=w.heads,
                        head_dim=w.head_dim, negative_slope=w.negative_slope, eval_every=eval_every, host=host)
    B.retexo_lmp_train(prob)
    torch.cuda.synchronize()
    return ref, prob.results()


def check(w, ref, got, R):
    for k in ("cross_edges", "boundary_pairs", "bytes_total", "dv_lazy_lt"):
        assert got["counts"][k] == ref["counts"][k], k
    np.testing.assert_array_equal(got["counts"]["bytes_per_round"], ref["counts"]["bytes_per_round"])
    n_val, n_test = len(w.val_idx), len(w.test_idx)
    for m, rd in enumerate(ref["rounds"]):
        gl, rl = got["loss_history"][m], rd["losses"]
        assert abs(gl[0] - rl[0]) <= 1e-3 * max(1.0, rl[0]), (m, gl[0], rl[0])      # same weights, same inputs
        assert np.abs(gl - rl).max() <= 0.05 * max(1.0, rl.max()), (m, np.abs(gl - rl).max())
        gv = got["val_correct"][m].astype(np.int64)
        assert np.abs(gv - rd["val_correct"]).max() <= max(3, 0.01 * n_val), m
        assert got["best_iter"][m] == int(np.argmax(gv)) + 1                        # earliest best iterate
        assert got["best_val_correct"][m] == gv.max()
        assert abs(int(got["test_correct"][m]) - rd["test_correct_best"]) <= max(3, 0.01 * n_test)
    # final accuracy within 0.5 points of the checker's
    assert abs(got["test_acc"] - ref["test_acc"]) <= 0.005 + 1.0 / n_test, (got["test_acc"], ref["test_acc"])
    assert abs(got["test_acc_last"] - ref["test_acc_last"]) <= 0.005 + 1.0 / n_test
    # final predictions agree wherever the reference margin is clear
    lg = ref["rounds"][-1]["logits"]
    srt = np.sort(lg, axis=1)
    clear = (srt[:, -1] - srt[:, -2]) > 0.05 * np.abs(lg).max(axis=1)
    agree = (got["final_pred"][clear] == ref["rounds"][-1]["pred"][clear]).mean()
    assert agree > 0.995, agree


@pytest.mark.parametrize("idx,scale,R", [(1, 1.0, 30), (2, 1.0, 25), (3, 1.0, 30), (4, 0.01, 12), (5, 0.004, 12)])
def test_device_resident_run_matches_checker(idx, scale, R):
    w = wl.make_config(idx, scale=scale)
    ref, got = run_both(w, R)
    check(w, ref, got, R)


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
    v = got["val_correct"][0]
    evaluated = [i for i in range(10) if v[i] != 2 ** 64 - 1]
    assert evaluated == [3, 7, 9]
    assert got["best_iter"][0] in (4, 8, 10)
