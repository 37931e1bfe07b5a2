"""Structure of the seeded synthetic inputs (no arithmetic of the method)."""
import numpy as np
import pytest

from paper_2302_13053_b200 import workloads as wl


@pytest.mark.parametrize("idx,scale", [(1, 1.0), (2, 1.0), (3, 1.0), (4, 0.01), (5, 0.01)])
def test_graph_is_symmetric_sorted_loop_free_and_seeded(idx, scale):
    w = wl.make_config(idx, scale=scale)
    n, deg = w.n_nodes, np.diff(w.rowptr)
    assert w.rowptr[0] == 0 and w.rowptr[-1] == w.n_edges and (deg >= 0).all()
    rows = np.repeat(np.arange(n), deg)
    assert (rows != w.colidx).all()
    key = rows.astype(np.int64) * n + w.colidx
    assert (np.diff(key) > 0).all()                       # sorted rows, no duplicates
    assert np.array_equal(np.sort(w.colidx.astype(np.int64) * n + rows), key)   # symmetric
    assert w.features.dtype == np.float32 and w.features.shape[0] == n
    assert w.labels.min() >= 0 and w.labels.max() < w.n_classes
    allidx = np.concatenate([w.train_idx, w.val_idx, w.test_idx])
    assert np.unique(allidx).shape[0] == allidx.shape[0]
    assert w.part.min() >= 0 and w.part.max() < w.n_parts
    w2 = wl.make_config(idx, scale=scale)
    assert np.array_equal(w.colidx, w2.colidx) and np.array_equal(w.features, w2.features)


def test_full_size_shapes_of_the_three_small_configs():
    w1, w2, w3 = wl.make_config(1), wl.make_config(2), wl.make_config(3)
    assert (w1.n_nodes, w1.n_edges, w1.d0, len(w1.train_idx)) == (2708, 10556, 1433, 140)
    assert (w2.n_nodes, w2.n_edges, w2.d0, len(w2.train_idx)) == (19717, 88648, 500, 60)
    assert (w3.n_nodes, w3.n_edges, w3.d0) == (22470, 342004, 128)
    assert 600 <= np.diff(w3.rowptr).max() <= 800
    assert abs((w1.features != 0).mean() - 0.013) < 0.002
    np.testing.assert_allclose(np.linalg.norm(w2.features, axis=1), 1.0, atol=1e-5)
    assert [d["d_in"] for d in w2.round_dims()] == [1000, 256, 256]
    assert [d["hidden"] for d in w1.round_dims()] == [64, 64, 0]
