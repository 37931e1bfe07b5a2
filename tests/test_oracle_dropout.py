"""Pins of the CPU checker's dropout (Appendix B lists dropout among the hyper-parameters):
the generator against its published known-answer vectors, the mask against the generator, the
masked step against closed forms, finite differences and the step without dropout."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_known_answers.txt")


def make(d_in, hidden, n_classes, seed, **kw):
    rng = np.random.default_rng(seed)
    return oracle.Mlp(d_in, hidden, n_classes, rng.standard_normal((d_in, hidden)) * 0.4,
                      rng.standard_normal(hidden) * 0.1, rng.standard_normal((hidden, n_classes)) * 0.3,
                      rng.standard_normal(n_classes) * 0.1, **kw)


def test_generator_reproduces_the_published_known_answers():
    n = 0
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        ctr, key, out = [[int(v, 16) for v in part.split()] for part in line.split("|")]
        assert oracle.philox4x32_10(ctr, key) == out
        n += 1
    assert n == 3


def test_mask_is_the_generator_word_compared_with_the_threshold():
    p, seed, hidden = 0.3, 0x1234567890abcdef, 11
    thresh = int(np.floor(p * 2.0 ** 32))
    for row, step in [(0, 1), (5, 1), (5, 2), (70000, 199)]:
        keep = oracle.dropout_mask(row, step, hidden, p, seed)
        for j in range(hidden):
            w = oracle.philox4x32_10([row, j // 4, step, 0], [seed & 0xffffffff, seed >> 32])[j % 4]
            assert keep[j] == (1.0 / (1.0 - p) if w >= thresh else 0.0)


def test_keep_rate_scale_and_independence_of_rows_steps_and_seeds():
    p, hidden = 0.5, 256
    rows = np.stack([oracle.dropout_mask(i, 3, hidden, p, 7) for i in range(400)])
    assert set(np.unique(rows)) == {0.0, 2.0}
    kept = (rows > 0).mean()
    assert abs(kept - 0.5) < 4 * np.sqrt(0.25 / rows.size)
    assert abs(rows.mean() - 1.0) < 0.02                         # E[keep] = 1: the expectation of Hd is unchanged
    np.testing.assert_array_equal(rows[0], oracle.dropout_mask(0, 3, hidden, p, 7))      # a pure function
    for other in (oracle.dropout_mask(1, 3, hidden, p, 7), oracle.dropout_mask(0, 4, hidden, p, 7),
                  oracle.dropout_mask(0, 3, hidden, p, 8)):
        assert 0.3 < ((rows[0] > 0) != (other > 0)).mean() < 0.7
    # rate 0.25: three quarters kept
    q = np.stack([oracle.dropout_mask(i, 1, hidden, 0.25, 1) for i in range(400)])
    assert abs((q > 0).mean() - 0.75) < 4 * np.sqrt(0.1875 / q.size)


def test_rate_zero_is_the_plain_step_bit_for_bit():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((12, 5)).astype(np.float32)
    y = rng.integers(0, 3, 12).astype(np.int32)
    a, b = make(5, 6, 3, 1, lr=0.05), make(5, 6, 3, 1, lr=0.05)
    la = a.train_step(x, y)
    lb = b.train_step(x, y, dropout=0.0, dropout_seed=99)
    assert la == lb
    np.testing.assert_array_equal(a.theta, b.theta)


def test_masked_forward_loss_and_gradient_against_numpy_closed_form():
    """Loss and gradient written out with the mask as a constant matrix."""
    n, d, h, o, p, seed = 7, 4, 8, 3, 0.4, 42
    rng = np.random.default_rng(3)
    x = rng.standard_normal((n, d)).astype(np.float32)
    y = rng.integers(0, o, n).astype(np.int32)
    m = make(d, h, o, 2, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    u = m.unpack()
    loss, grad = m.copy().train_step(x, y, return_grad=True, dropout=p, dropout_seed=seed)
    keep = np.stack([oracle.dropout_mask(i, 1, h, p, seed) for i in range(n)])       # update number 1
    a1 = x.astype(np.float64) @ u["w1"] + u["b1"]
    hd = np.maximum(a1, 0.0) * keep
    lg = hd @ u["w2"] + u["b2"]
    lg = lg - lg.max(axis=1, keepdims=True)
    prob = np.exp(lg) / np.exp(lg).sum(axis=1, keepdims=True)
    ref_loss = -np.log(prob[np.arange(n), y]).mean()
    assert abs(loss - ref_loss) < 1e-12
    dl = prob.copy()
    dl[np.arange(n), y] -= 1.0
    dl /= n
    d1 = (dl @ u["w2"].T) * (a1 > 0) * keep
    ref = np.concatenate([(x.astype(np.float64).T @ d1).ravel(), d1.sum(0), (hd.T @ dl).ravel(), dl.sum(0)])
    np.testing.assert_allclose(grad, ref, rtol=0, atol=1e-12)


def test_gradient_with_a_fixed_mask_matches_central_finite_differences():
    n, d, h, o, p, seed = 9, 4, 6, 3, 0.5, 5
    rng = np.random.default_rng(4)
    x = rng.standard_normal((n, d)).astype(np.float32)
    y = rng.integers(0, o, n).astype(np.int32)
    base = make(d, h, o, 6, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    _, grad = base.copy().train_step(x, y, return_grad=True, dropout=p, dropout_seed=seed)

    def loss_at(theta):
        m = base.copy()                 # same update number, so the same mask
        m.theta = theta.copy()
        return m.train_step(x, y, dropout=p, dropout_seed=seed)

    eps = 1e-6
    for q in rng.choice(base.theta.shape[0], size=25, replace=False):
        tp, tm = base.theta.copy(), base.theta.copy()
        tp[q] += eps
        tm[q] -= eps
        assert abs((loss_at(tp) - loss_at(tm)) / (2 * eps) - grad[q]) < 1e-7


def test_the_mask_changes_with_the_update_number_and_evaluation_ignores_it():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((20, 4)).astype(np.float32)
    y = rng.integers(0, 3, 20).astype(np.int32)
    m = make(4, 16, 3, 7, optimizer=oracle.SGD, lr=0.0, round_bf16=False)
    l1 = m.train_step(x, y, dropout=0.5, dropout_seed=1)       # update 1
    l2 = m.train_step(x, y, dropout=0.5, dropout_seed=1)       # update 2: lr = 0, same weights, other mask
    assert l1 != l2
    plain = m.copy().train_step(x, y)
    out = m.embed(x, y=y)                                       # evaluation: no dropout
    lg = out["logits"].astype(np.float64)
    lg = lg - lg.max(axis=1, keepdims=True)
    ev = -np.log(np.exp(lg)[np.arange(20), y] / np.exp(lg).sum(axis=1)).mean()
    assert abs(ev - plain) < 1e-5
