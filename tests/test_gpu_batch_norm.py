"""CUDA batch normalisation inside f_theta (Linear -> BatchNorm -> ReLU; paper Section 2.2 names batch and layer
normalisation among the parts of f_theta) against the CPU checker: one training step (loss, every gradient
including d gamma / d beta, the update, the running statistics), the evaluation-mode forward used for emission
and validation, the gradient with respect to the batch, and a K-round run.

Tolerances are those of the plain model (loss 2e-4, gradients 5e-3 of the largest entry with a median of 2e-5,
update 2e-6, emitted values 2e-2 of the row's largest); the running statistics, sums of fp32 values over the
batch in a fixed order against double, are held to 1e-5 of their scale."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_logits_close, dev

pytestmark = pytest.mark.gpu


def B():
    from paper_2302_13053_b200 import binding
    return binding


def make_pair(d_in, hidden, n_classes, seed, opt=oracle.ADAM, lr=1e-3, momentum=0.1):
    rng = np.random.default_rng(seed)
    w1 = (rng.standard_normal((d_in, hidden)) / np.sqrt(d_in)).astype(np.float32)
    b1 = (rng.standard_normal(hidden) * 0.1).astype(np.float32)
    w2 = (rng.standard_normal((hidden, n_classes)) / np.sqrt(hidden)).astype(np.float32)
    b2 = (rng.standard_normal(n_classes) * 0.1).astype(np.float32)
    g = (1.0 + 0.2 * rng.standard_normal(hidden)).astype(np.float32)
    be = (0.2 * rng.standard_normal(hidden)).astype(np.float32)
    rm = (0.1 * rng.standard_normal(hidden)).astype(np.float32)
    rv = (1.0 + 0.2 * rng.random(hidden)).astype(np.float32)
    kw = dict(optimizer=opt, lr=lr, batch_norm=True, ln_gamma=g, ln_beta=be, bn_mean=rm, bn_var=rv, bn_momentum=momentum)
    return oracle.Mlp(d_in, hidden, n_classes, w1, b1, w2, b2, round_bf16=True, **kw), \
        B().Mlp(d_in, hidden, n_classes, w1, b1, w2, b2, **kw)


@pytest.mark.parametrize("d_in,hidden,n_classes,n", [(33, 20, 4, 65), (64, 64, 7, 140), (100, 256, 47, 5300),
                                                     (1204, 256, 41, 513), (70, 300, 10, 257), (48, 512, 64, 129)])
@pytest.mark.parametrize("opt", [oracle.SGD, oracle.ADAM])
def test_train_steps_with_batch_norm_track_the_checker(d_in, hidden, n_classes, n, opt):
    rng = np.random.default_rng(d_in + hidden)
    x = (rng.standard_normal((n, d_in)) + 0.3).astype(np.float32)      # (a mean the statistics have to remove)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    ref, gpu = make_pair(d_in, hidden, n_classes, 1, opt=opt, lr=0.02 if opt == oracle.SGD else 1e-3)
    n_trained = (d_in + 1) * hidden + (hidden + 1) * n_classes + 2 * hidden
    assert gpu.theta.numel() == ref.theta.shape[0] == n_trained + 2 * hidden
    x16, _ = B().retexo_pack_rows(dev(x), None, ones=True, ld_multiple=8 if n % 2 else 64)
    yd = dev(y)
    for it in range(3):
        # every iteration starts from the GPU's own state, so that each step is compared on its own
        ref.theta = gpu.theta.cpu().numpy().astype(np.float64)
        ref.m = gpu.m.cpu().numpy().astype(np.float64)
        ref.v = gpu.v.cpu().numpy().astype(np.float64)
        given = ref.copy()
        rl, rg = ref.train_step(x, y, return_grad=True)
        gl, gg = B().retexo_mlp_train_step(gpu, x16, yd, x_has_ones=True, return_grad=True)
        assert abs(gl.item() - rl) <= 2e-4 * max(1.0, abs(rl)), (it, gl.item(), rl)
        gg = gg.cpu().numpy().astype(np.float64)
        scale = np.abs(rg).max()
        err = np.abs(gg - rg)
        assert err.max() <= 5e-3 * scale + 1e-7, (it, err.max(), scale, int(err.argmax()))
        assert np.median(err) <= 2e-5 * scale, (it, np.median(err), scale)
        # the normalisation's own parameters, on their own scale; the statistics' entries are exactly zero
        tail, rt = gg[n_trained - 2 * hidden:n_trained], rg[n_trained - 2 * hidden:n_trained]
        assert np.abs(tail - rt).max() <= 5e-3 * np.abs(rt).max() + 1e-7, it
        assert not gg[n_trained:].any() and not rg[n_trained:].any()
        given.apply_update(gg)
        gt = gpu.theta.cpu().numpy().astype(np.float64)
        assert np.abs(gt[:n_trained] - given.theta[:n_trained]).max() <= 2e-6 * max(1.0, np.abs(given.theta).max()), it
        # running statistics: moved like the checker's, and moved at all; the optimiser's moments never touched
        assert np.abs(gt[n_trained:] - ref.theta[n_trained:]).max() <= 1e-5 * max(1.0, np.abs(ref.theta[n_trained:]).max()), it
        assert np.abs(gt[n_trained:] - given.theta[n_trained:]).max() > 1e-4
        assert not gpu.m.cpu().numpy()[n_trained:].any() and not gpu.v.cpu().numpy()[n_trained:].any()
        assert int(gpu.status.item()) == 0


def test_a_second_run_gives_the_same_bits():
    d_in, hidden, n_classes, n = 100, 256, 47, 9000
    rng = np.random.default_rng(5)
    x = rng.standard_normal((n, d_in)).astype(np.float32)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    x16, _ = B().retexo_pack_rows(dev(x), None, ones=True)
    out = []
    for _ in range(2):
        _, gpu = make_pair(d_in, hidden, n_classes, 4)
        for _ in range(2):
            B().retexo_mlp_train_step(gpu, x16, dev(y), x_has_ones=True)
        out.append(gpu.theta.cpu().numpy().copy())
    assert np.array_equal(out[0], out[1])


def test_gradient_with_respect_to_the_batch_goes_through_the_normalisation():
    d_in, hidden, n_classes, n = 96, 64, 5, 300
    rng = np.random.default_rng(9)
    x = rng.standard_normal((n, d_in)).astype(np.float32)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    ref, gpu = make_pair(d_in, hidden, n_classes, 2, opt=oracle.SGD, lr=0.0)
    x16, _ = B().retexo_pack_rows(dev(x), None, ones=True)
    _, _, rdx = ref.train_step_dx(x, y)
    _, _, gdx = B().retexo_mlp_train_step(gpu, x16, dev(y), x_has_ones=True, return_grad=True, return_dx=True)
    err = np.abs(gdx.cpu().numpy().astype(np.float64) - rdx)
    assert err.max() <= 5e-3 * np.abs(rdx).max()


@pytest.mark.parametrize("d_in,hidden,n_classes,n", [(64, 64, 7, 500), (200, 256, 41, 700), (70, 300, 10, 257)])
@pytest.mark.parametrize("gathered", [False, True])
def test_evaluation_forward_uses_the_running_statistics(d_in, hidden, n_classes, n, gathered):
    rng = np.random.default_rng(hidden + n)
    x = rng.standard_normal((n, d_in)).astype(np.float32)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    ref, gpu = make_pair(d_in, hidden, n_classes, 3)
    idx = rng.permutation(n)[: n // 2].astype(np.int32) if gathered else None
    want = ref.embed(x, row_idx=idx, y=y if idx is None else y[idx], want_hidden=True)
    x16, _ = B().retexo_pack_rows(dev(x), None)
    got = B().retexo_embed(gpu, x16, row_idx=None if idx is None else dev(idx),
                           y=dev(y if idx is None else y[idx]), want_hidden=True, want_hidden_bf16=True,
                           want_logits=True, want_pred=True)
    assert_logits_close(got["hidden"].cpu().numpy(), want["hidden"], 2e-2)
    assert_logits_close(got["hidden_bf16"][:, :hidden].float().cpu().numpy(), want["hidden"], 2e-2)
    assert_logits_close(got["logits"].cpu().numpy(), want["logits"], 2e-2)
    lg = np.sort(want["logits"], axis=1)
    clear = (lg[:, -1] - lg[:, -2]) > 2e-2 * np.abs(lg).max(axis=1)
    assert np.array_equal(got["pred"].cpu().numpy()[clear], want["pred"][clear])
    assert abs(got["correct"] - want["correct"]) <= int((~clear).sum())


def test_a_batch_of_one_row_is_refused():
    _, gpu = make_pair(16, 8, 3, 0)
    x16, _ = B().retexo_pack_rows(dev(np.ones((1, 16), np.float32)), None, ones=True)
    with pytest.raises(B().RetexoError):
        B().retexo_mlp_train_step(gpu, x16, dev(np.zeros(1, np.int32)), x_has_ones=True)


@pytest.mark.parametrize("cfg", [1, 2])
def test_k_round_run_with_batch_norm_tracks_the_checker(cfg):
    from paper_2302_13053_b200 import workloads as wl
    w = wl.make_config(cfg, scale=0.2)
    ws = wl.initial_weights(w)
    R = 8
    prob = B().LmpProblem(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                          w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts, batch_norm=True)
    B().retexo_lmp_train(prob)
    torch.cuda.synchronize()
    got = prob.results()
    assert got["status"] == 0
    # the checker trains its own models, but hands on what the GPU kept (running statistics included): the same
    # starting point every round
    ref = oracle.lmp_train(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                           w.train_idx, w.val_idx, w.test_idx, ws, batch_norm=True,
                           forced_theta=[t.astype(np.float64) for t in got["theta_best"]])
    for m, rd in enumerate(ref["rounds"]):
        gl = np.asarray(got["loss_history"][m])
        assert abs(gl[0] - rd["losses"][0]) <= 1e-3 * max(1.0, rd["losses"][0]), (m, gl[0], rd["losses"][0])
        assert np.abs(gl - rd["losses"]).max() <= 2e-2 * max(1.0, np.abs(rd["losses"]).max()), m
    assert got["theta_best"][0].shape[0] == ref["rounds"][0]["model"].theta.shape[0]
    assert_logits_close(got["final_logits"], ref["rounds"][-1]["logits"], 2e-2 * w.K)
