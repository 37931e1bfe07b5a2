"""Dropout in the CUDA training step against the CPU checker: both sides draw the mask from the
same counter-based generator (Philox4x32-10 of (batch row, unit, update number), each written from
its published definition), so the masked steps must agree as closely as the unmasked ones do."""
import numpy as np
import pytest

import oracle
from gpu_util import dev

pytestmark = pytest.mark.gpu


def B():
    from paper_2302_13053_b200 import binding
    return binding


def pair(d_in, hidden, n_classes, seed, p, drop_seed, opt=oracle.SGD, lr=0.02):
    rng = np.random.default_rng(seed)
    w1 = (rng.standard_normal((d_in, hidden)) / np.sqrt(d_in)).astype(np.float32)
    b1 = (rng.standard_normal(hidden) * 0.1).astype(np.float32)
    w2 = (rng.standard_normal((hidden, n_classes)) / np.sqrt(hidden)).astype(np.float32)
    b2 = (rng.standard_normal(n_classes) * 0.1).astype(np.float32)
    ref = oracle.Mlp(d_in, hidden, n_classes, w1, b1, w2, b2, optimizer=opt, lr=lr, round_bf16=True)
    gpu = B().Mlp(d_in, hidden, n_classes, w1, b1, w2, b2, optimizer=opt, lr=lr, dropout=p, dropout_seed=drop_seed)
    return ref, gpu


@pytest.mark.parametrize("d_in,hidden,n_classes,n,p", [(33, 20, 4, 65, 0.5), (64, 64, 7, 140, 0.25),
                                                       (100, 256, 47, 300, 0.5), (70, 130, 5, 513, 0.3),
                                                       (1204, 256, 41, 700, 0.5)])
def test_masked_steps_track_the_checker(d_in, hidden, n_classes, n, p):
    p = float(np.float32(p))                   # the rate both sides see
    drop_seed = 0x9e3779b97f4a7c15 ^ n
    rng = np.random.default_rng(d_in + hidden)
    x = rng.standard_normal((n, d_in)).astype(np.float32)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    ref, gpu = pair(d_in, hidden, n_classes, 1, p, drop_seed)
    x16, _ = B().retexo_pack_rows(dev(x), None, ones=True, ld_multiple=8 if n % 2 else 64)
    x_host = x16[:, :d_in].float().cpu().numpy()
    losses = []
    for it in range(3):
        # each iteration starts from the GPU's state (see test_gpu_mlp.py); update numbers stay in step
        ref.theta = gpu.theta.cpu().numpy().astype(np.float64)
        rl, rg = ref.train_step(x_host, y, return_grad=True, dropout=p, dropout_seed=drop_seed)
        gl, gg = B().retexo_mlp_train_step(gpu, x16, dev(y), x_has_ones=True, return_grad=True)
        gg = gg.cpu().numpy().astype(np.float64)
        assert ref.step == gpu.step == it + 1
        assert abs(gl.item() - rl) <= 2e-4 * max(1.0, abs(rl)), (it, gl.item(), rl)
        err, scale = np.abs(gg - rg), np.abs(rg).max()
        assert err.max() <= 5e-3 * scale + 1e-7, (it, err.max(), scale)
        assert np.median(err) <= 2e-5 * scale
        losses.append(gl.item())
    assert len(set(losses)) == 3               # another mask every update
    # without dropout the same weights give another loss: the mask is really applied
    plain = oracle.Mlp(d_in, hidden, n_classes, **ref.unpack(), optimizer=oracle.SGD, lr=0.0, round_bf16=True)
    plain.theta = gpu.theta.cpu().numpy().astype(np.float64)
    assert abs(plain.train_step(x_host, y) - losses[-1]) > 1e-3


def test_rate_zero_is_bit_for_bit_the_plain_step_and_bad_rates_are_rejected():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((200, 48)).astype(np.float32)
    y = rng.integers(0, 5, 200).astype(np.int32)
    x16, _ = B().retexo_pack_rows(dev(x), None, ones=True)
    _, a = pair(48, 64, 5, 3, 0.0, 0)
    _, b = pair(48, 64, 5, 3, 0.0, 12345)
    la = B().retexo_mlp_train_step(a, x16, dev(y), x_has_ones=True)
    lb = B().retexo_mlp_train_step(b, x16, dev(y), x_has_ones=True)
    assert la.item() == lb.item()
    assert (a.theta == b.theta).all()
    for bad in (1.0, -0.1, float("nan")):
        _, c = pair(48, 64, 5, 3, bad, 1)
        with pytest.raises(B().RetexoError):
            B().retexo_mlp_train_step(c, x16, dev(y), x_has_ones=True)


def lmp_both(w, R, p, seed, eval_every):
    import torch
    from paper_2302_13053_b200 import workloads as wl
    ws = wl.initial_weights(w)
    prob = B().LmpProblem(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                          w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts,
                          eval_every=eval_every, dropout=p, dropout_seed=seed)
    B().retexo_lmp_train(prob)
    torch.cuda.synchronize()
    return prob.results(), ws


@pytest.mark.parametrize("idx,scale,R,eval_every", [(1, 1.0, 12, 1), (2, 1.0, 12, 12), (4, 0.05, 10, 1)])
def test_k_round_run_with_dropout_tracks_the_checker(idx, scale, R, eval_every):
    """The whole loop with dropout 0.5: with validation every iteration the iterations are replayed
    from a recorded graph and the update number that keys the mask lives on the device, so the first
    iterations' losses (same weights up to rounding, same masks) pin that bookkeeping."""
    from paper_2302_13053_b200 import workloads as wl
    w = wl.make_config(idx, scale=scale)
    p, seed = 0.5, 0xfeedfacecafebeef
    got, ws = lmp_both(w, R, p, seed, eval_every)
    ref = oracle.lmp_train(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                           w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts,
                           eval_every=eval_every, forced_best_iter=list(got["best_iter"]), dropout=p,
                           dropout_seed=seed, forced_theta=got["theta_best"])
    rl, gl = ref["rounds"][0]["losses"], got["loss_history"][0]
    assert abs(gl[0] - rl[0]) <= 1e-3 * max(1.0, rl[0]), (gl[0], rl[0])
    assert np.abs(gl[:4] - rl[:4]).max() <= 1e-2 * max(1.0, rl[:4].max()), (gl[:4], rl[:4])
    for m, rd in enumerate(ref["rounds"]):
        g = got["loss_history"][m]
        assert np.isfinite(g).all()
        # (every round starts from the GPU's kept weights on both sides, at the configuration's own learning rate)
        assert np.abs(g - rd["losses"]).max() <= 2e-2 * max(1.0, rd["losses"].max()), (m, np.abs(g - rd["losses"]).max())
    # the run without dropout is a different run, the same seed the same bits, another seed other masks
    plain, _ = lmp_both(w, R, 0.0, seed, eval_every)
    assert np.abs(plain["loss_history"][0] - gl).max() > 1e-3
    again, _ = lmp_both(w, R, p, seed, eval_every)
    np.testing.assert_array_equal(again["loss_history"], got["loss_history"])
    np.testing.assert_array_equal(again["val_correct"], got["val_correct"])
    other, _ = lmp_both(w, R, p, seed + 1, eval_every)
    assert np.abs(other["loss_history"][0][1:] - gl[1:]).max() > 1e-4
