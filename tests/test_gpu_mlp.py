"""CUDA per-node model (retexo_pack_rows, retexo_mlp_train_step, retexo_embed)
against the CPU checker.

Both sides round the operands of every matrix product to bf16 and accumulate
wider (GPU fp32, checker double), so against the checker run with the same
operand rounding the logits agree far inside the stated 2e-2 relative
tolerance; the unrounded checker is compared at 2e-2 as well."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_logits_close, dev

pytestmark = pytest.mark.gpu


def B():
    from paper_2302_13053_b200 import binding
    return binding


def make_pair(d_in, hidden, n_classes, seed, opt=oracle.ADAM, lr=0.01):
    rng = np.random.default_rng(seed)
    out1 = hidden if hidden > 0 else n_classes
    w1 = (rng.standard_normal((d_in, out1)) / np.sqrt(d_in)).astype(np.float32)
    b1 = (rng.standard_normal(out1) * 0.1).astype(np.float32)
    w2 = (rng.standard_normal((hidden, n_classes)) / np.sqrt(max(hidden, 1))).astype(np.float32) if hidden else None
    b2 = (rng.standard_normal(n_classes) * 0.1).astype(np.float32) if hidden else None
    ref = oracle.Mlp(d_in, hidden, n_classes, w1, b1, w2, b2, optimizer=opt, lr=lr, round_bf16=True)
    gpu = B().Mlp(d_in, hidden, n_classes, w1, b1, w2, b2, optimizer=opt, lr=lr)
    return ref, gpu


def test_pack_rows_gathers_rounds_and_transposes():
    rng = np.random.default_rng(0)
    src = rng.standard_normal((70, 37)).astype(np.float32)
    idx = rng.integers(0, 70, 45).astype(np.int32)
    want = torch.from_numpy(src[idx]).to(torch.bfloat16)
    dst, dst_t = B().retexo_pack_rows(dev(src), dev(idx), transpose=True)
    assert dst.shape == (45, 64) and dst_t.shape == (37, 64)          # default: rows on 128-byte lines
    for source in (dev(src), dev(src).to(torch.bfloat16)):
        dst, dst_t = B().retexo_pack_rows(source, dev(idx), transpose=True, ld_multiple=8)
        assert dst.shape == (45, 40) and dst_t.shape == (37, 48)
        ref = want if source.dtype == torch.float32 else want
        assert torch.equal(dst[:, :37].cpu(), ref)
        assert torch.equal(dst_t[:, :45].cpu(), ref.T)
        assert dst[:, 37:].abs().sum() == 0 and dst_t[:, 45:].abs().sum() == 0
    dst, _ = B().retexo_pack_rows(dev(src), None, dim=20)
    assert torch.equal(dst[:, :20].cpu(), torch.from_numpy(src[:, :20]).to(torch.bfloat16))
    # the ones that carry the bias gradient through the weight-gradient product: a column behind the batch,
    # a row under its transpose
    dst, dst_t = B().retexo_pack_rows(dev(src), dev(idx), transpose=True, ones=True, ld_multiple=8)
    assert dst.shape == (45, 40) and dst_t.shape == (38, 48)
    assert torch.equal(dst[:, :37].cpu(), want) and torch.equal(dst_t[:37, :45].cpu(), want.T)
    assert torch.equal(dst[:, 37].float().cpu(), torch.ones(45)) and dst[:, 38:].abs().sum() == 0
    assert torch.equal(dst_t[37].float().cpu(), torch.cat([torch.ones(45), torch.zeros(3)]))
    dst, _ = B().retexo_pack_rows(dev(src)[:, :32].contiguous(), None, ones=True)      # a full last line: one more line
    assert dst.shape == (70, 64) and torch.equal(dst[:, 32].float().cpu(), torch.ones(70)) and dst[:, 33:].abs().sum() == 0


@pytest.mark.parametrize("d_in,hidden,n_classes,n", [(5, 0, 3, 17), (64, 64, 7, 140), (33, 20, 4, 65),
                                                     (1433, 64, 7, 140), (100, 256, 47, 300), (1204, 256, 41, 513),
                                                     (256, 0, 3, 60), (70, 512, 64, 129)])
@pytest.mark.parametrize("opt", [oracle.SGD, oracle.ADAM])
def test_train_steps_track_the_checker(d_in, hidden, n_classes, n, opt):
    rng = np.random.default_rng(d_in + hidden)
    x = rng.standard_normal((n, d_in)).astype(np.float32)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    # Adam's first steps move every weight by about lr whatever the gradient's size, so weights whose
    # gradient is at rounding level take a different step in fp32 and fp64: keep that step small.
    ref, gpu = make_pair(d_in, hidden, n_classes, 1, opt=opt, lr=0.02 if opt == oracle.SGD else 1e-3)
    x16, _ = B().retexo_pack_rows(dev(x), None, ones=True, ld_multiple=8 if n % 2 else 64)
    yd = dev(y)
    for it in range(4):
        # Every iteration starts from the GPU's own state, so that each step is compared on its
        # own: an optimiser turns rounding-level gradient differences on near-zero gradients into
        # full-size steps (Adam moves a weight by about lr whatever the gradient's size), and the
        # two trajectories would otherwise drift apart for reasons that are not errors.
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
        assert err.max() <= 5e-3 * scale + 1e-7, (it, err.max(), scale)
        assert np.median(err) <= 2e-5 * scale, (it, np.median(err), scale)
        assert gpu.step == ref.step == it + 1
        # the update itself: the checker's optimiser fed with the GPU's gradient
        given.apply_update(gg)
        gt = gpu.theta.cpu().numpy().astype(np.float64)
        assert np.abs(gt - given.theta).max() <= 2e-6 * max(1.0, np.abs(given.theta).max()), it
        assert int(gpu.status.item()) == 0          # the status word reaches the caller: no bounded wait ran out


def test_zero_weights_give_log_of_class_count():
    n, d, h, o = 50, 12, 8, 5
    x = np.random.default_rng(3).standard_normal((n, d)).astype(np.float32)
    y = np.random.default_rng(4).integers(0, o, n).astype(np.int32)
    gpu = B().Mlp(d, h, o, np.zeros((d, h)), np.zeros(h), np.zeros((h, o)), np.zeros(o), optimizer=oracle.SGD, lr=0.1)
    x16, _ = B().retexo_pack_rows(dev(x))
    loss = B().retexo_mlp_train_step(gpu, x16, dev(y))      # no column of ones given: the call adds it itself
    assert abs(loss.item() - np.log(o)) < 1e-6


@pytest.mark.parametrize("d_in,hidden,n_classes,n", [(64, 64, 7, 500), (1000, 128, 3, 300), (33, 0, 5, 200),
                                                     (602, 256, 41, 257)])
def test_embed_matches_checker_and_stated_tolerance(d_in, hidden, n_classes, n):
    rng = np.random.default_rng(7)
    x = rng.standard_normal((n, d_in)).astype(np.float32)
    ref, gpu = make_pair(d_in, hidden, n_classes, 2)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    x16, _ = B().retexo_pack_rows(dev(x))
    out = B().retexo_embed(gpu, x16, y=dev(y), want_hidden=hidden > 0, want_hidden_bf16=hidden > 0,
                           want_logits=True, want_pred=True)
    r = ref.embed(x, y=y, want_hidden=hidden > 0)
    lg = out["logits"].cpu().numpy()
    # 5e-3: one hidden unit whose fp32 and fp64 pre-activations straddle a bf16 rounding boundary
    # differs by a bf16 ulp (2^-8 relative) and moves a logit by up to |w2| x that
    assert_logits_close(lg, r["logits"], rel=5e-3, what="vs bf16-operand checker")
    exact = oracle.Mlp(d_in, hidden, n_classes, **{k: v for k, v in ref.unpack().items()}, round_bf16=False)
    assert_logits_close(lg, exact.embed(x)["logits"], rel=2e-2, what="vs unrounded checker")
    if hidden > 0:
        h = out["hidden"].cpu().numpy()
        assert_logits_close(h, r["hidden"], rel=1e-3, what="hidden")
        assert torch.equal(out["hidden_bf16"][:, :hidden].cpu(), out["hidden"].to(torch.bfloat16).cpu())
    # predictions: exact wherever the reference margin is clear of the tolerance
    srt = np.sort(r["logits"], axis=1)
    clear = (srt[:, -1] - srt[:, -2]) > 4e-3 * np.abs(r["logits"]).max(axis=1)
    pred = out["pred"].cpu().numpy()
    np.testing.assert_array_equal(pred[clear], r["pred"][clear])
    np.testing.assert_array_equal(pred, lg.argmax(1))            # argmax of its own logits, lowest index on ties
    assert out["correct"] == int((pred == y).sum())
    # row gather
    idx = rng.integers(0, n, 77).astype(np.int32)
    sub = B().retexo_embed(gpu, x16, row_idx=dev(idx), want_logits=True)
    # (gathered rows take the CUDA-core product, dense ones the tensor cores: same values up to
    # summation order and the bf16 rounding of the hidden layer that follows it)
    assert_logits_close(sub["logits"].cpu().numpy(), lg[idx], rel=5e-3, what="row gather")


def test_argmax_tie_rule_lowest_index():
    gpu = B().Mlp(8, 0, 4, np.zeros((8, 4)), np.array([1.0, 3.0, 3.0, 3.0]))
    x16, _ = B().retexo_pack_rows(dev(np.ones((5, 8), dtype=np.float32)))
    out = B().retexo_embed(gpu, x16, want_pred=True)
    assert out["pred"].cpu().tolist() == [1] * 5


@pytest.mark.parametrize("d_in,hidden,n_classes,n", [(64, 64, 4, 300), (64, 0, 4, 300), (33, 20, 5, 129), (128, 256, 41, 513)])
def test_input_gradient_matches_the_checker(d_in, hidden, n_classes, n):
    """dLoss / dx, the extra output a round with a trained aggregator needs."""
    rng = np.random.default_rng(n + hidden)
    x = rng.standard_normal((n, d_in)).astype(np.float32)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    ref, gpu = make_pair(d_in, hidden, n_classes, 3, opt=oracle.SGD, lr=0.01)
    x16, _ = B().retexo_pack_rows(dev(x), None, ones=True)
    x_host = x16[:, :d_in].float().cpu().numpy()
    rl, rg, rdx = ref.train_step_dx(x_host, y)
    gl, gg, gdx = B().retexo_mlp_train_step(gpu, x16, dev(y), x_has_ones=True, return_grad=True, return_dx=True)
    assert abs(gl.item() - rl) <= 2e-4 * max(1.0, abs(rl))
    gdx = gdx.cpu().numpy().astype(np.float64)
    err, scale = np.abs(gdx - rdx), np.abs(rdx).max()
    assert err.max() <= 5e-3 * scale + 1e-9, (err.max(), scale)
    assert np.median(err) <= 1e-4 * scale
    # asking for it changes nothing else
    _, gpu2 = make_pair(d_in, hidden, n_classes, 3, opt=oracle.SGD, lr=0.01)
    gl2, gg2 = B().retexo_mlp_train_step(gpu2, x16, dev(y), x_has_ones=True, return_grad=True)
    assert gl2.item() == gl.item() and torch.equal(gg, gg2) and torch.equal(gpu.theta, gpu2.theta)


@pytest.mark.parametrize("d_in,hidden,n_classes,n", [(200, 256, 10, 5000), (72, 192, 5, 4224), (1204, 256, 41, 9000)])
def test_wide_forward_over_many_rows_runs_in_block_pairs_and_matches_the_checker(d_in, hidden, n_classes, n):
    """Forward products with more than 128 output columns and at least 4096 rows run on pairs of thread
    blocks (256-row tiles, odd tails included): hidden representation, logits and one training step."""
    rng = np.random.default_rng(n)
    x = rng.standard_normal((n, d_in)).astype(np.float32)
    y = rng.integers(0, n_classes, n).astype(np.int32)
    ref, gpu = make_pair(d_in, hidden, n_classes, 5, opt=oracle.SGD, lr=0.01)
    x16, _ = B().retexo_pack_rows(dev(x), None, ones=True)
    x_host = x16[:, :d_in].float().cpu().numpy()
    out = B().retexo_embed(gpu, x16, want_hidden=True, want_hidden_bf16=True, want_logits=True)
    r = ref.embed(x_host, want_hidden=True)
    assert_logits_close(out["hidden"].cpu().numpy(), r["hidden"], rel=1e-3, what="hidden")
    assert torch.equal(out["hidden_bf16"][:, :hidden].cpu(), out["hidden"].to(torch.bfloat16).cpu())
    assert_logits_close(out["logits"].cpu().numpy(), r["logits"], rel=5e-3, what="logits")
    rl, rg = ref.train_step(x_host, y, return_grad=True)
    gl, gg = B().retexo_mlp_train_step(gpu, x16, dev(y), x_has_ones=True, return_grad=True)
    assert abs(gl.item() - rl) <= 2e-4 * max(1.0, abs(rl))
    err, scale = np.abs(gg.cpu().numpy().astype(np.float64) - rg), np.abs(rg).max()
    assert err.max() <= 5e-3 * scale + 1e-7 and np.median(err) <= 2e-5 * scale
    assert int(gpu.status.item()) == 0
