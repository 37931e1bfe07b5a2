"""CUDA cross-partition count (retexo_cross_partition_bytes) against the CPU
checker: every value bit-exact."""
import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from paper_2302_13053_b200 import workloads as wl
from gpu_util import dev

pytestmark = pytest.mark.gpu


def compare(rowptr, colidx, part, n_parts, dims=(7, 3), elem_bytes=4):
    from paper_2302_13053_b200 import binding as B
    ref = oracle.cross_partition(rowptr, colidx, part, n_parts, dims, elem_bytes)
    got = B.retexo_cross_partition_bytes(dev(rowptr.astype(np.int64)), dev(colidx.astype(np.int32)),
                                         dev(part.astype(np.int32)), n_parts, dims, elem_bytes)
    for k in ("cross_edges", "boundary_pairs", "bytes_total", "dv_lazy_lt"):
        assert got[k] == ref[k], k
    np.testing.assert_array_equal(got["bytes_per_round"], ref["bytes_per_round"])
    np.testing.assert_array_equal(got["send_per_part"], ref["send_per_part"])
    np.testing.assert_array_equal(got["recv_per_part"], ref["recv_per_part"])
    # the per-partition tallies are optional
    lean = B.retexo_cross_partition_bytes(dev(rowptr.astype(np.int64)), dev(colidx.astype(np.int32)),
                                          dev(part.astype(np.int32)), n_parts, dims, elem_bytes, per_part=False)
    assert lean["boundary_pairs"] == ref["boundary_pairs"] and lean["cross_edges"] == ref["cross_edges"]
    return ref


@pytest.mark.parametrize("n_parts", [1, 2, 31, 32, 33, 100, 1000, 8192, 8193, 50000])
def test_random_partitions_on_a_heavy_tailed_graph(n_parts):
    w = wl.make_config(5, scale=0.005)
    part = np.random.default_rng(n_parts).integers(0, n_parts, w.n_nodes).astype(np.int32)
    compare(w.rowptr, w.colidx, part, n_parts)


def test_node_level_partition_and_single_partition():
    w = wl.make_config(3)
    ref = compare(w.rowptr, w.colidx, np.arange(w.n_nodes, dtype=np.int32), w.n_nodes, dims=(128, 64))
    assert ref["boundary_pairs"] == w.n_edges == ref["cross_edges"]
    ref = compare(w.rowptr, w.colidx, np.zeros(w.n_nodes, dtype=np.int32), 1)
    assert ref["boundary_pairs"] == 0


def test_every_dedup_path_of_the_many_partition_kernel():
    """Node-level ids scrambled (rows not ordered -> hash set), a long scrambled
    row (> 512 entries -> global bitmap), range partitions (ordered rows)."""
    n, rowptr, colidx, _ = wl.degree_ladder_graph([3, 40, 900, 1500, 6000], seed=4)
    rng = np.random.default_rng(4)
    n_parts = 20000
    compare(rowptr, colidx, rng.permutation(n).astype(np.int32) % n_parts, n_parts)
    compare(rowptr, colidx, rng.integers(0, 9000, n).astype(np.int32), 9000)       # many duplicates per row
    compare(rowptr, colidx, (np.arange(n) // 3).astype(np.int32), n // 3 + 1 if n // 3 + 1 > 8192 else 8200)


def test_empty_graph_and_configs():
    compare(np.zeros(4, dtype=np.int64), np.zeros(0, dtype=np.int32), np.array([0, 1, 2], dtype=np.int32), 3)
    for idx, scale in ((1, 1.0), (2, 1.0), (4, 0.02)):
        w = wl.make_config(idx, scale=scale)
        dims = [d["rep_dim"] for d in w.round_dims()]
        compare(w.rowptr, w.colidx, w.part, w.n_parts, dims=dims)


def test_out_of_range_partition_id_poisons_the_result_without_faulting():
    from paper_2302_13053_b200 import binding as B
    rowptr, colidx = wl.ring_graph(8)
    part = np.array([0, 1, 2, 3, 99, 1, 2, 3], dtype=np.int32)
    got = B.retexo_cross_partition_bytes(dev(rowptr), dev(colidx), dev(part), 4, [5])
    assert got["cross_edges"] == 2 ** 64 - 1 and got["boundary_pairs"] == 2 ** 64 - 1


@settings(max_examples=25, deadline=None)
@given(st.integers(2, 80), st.integers(0, 400), st.integers(1, 40), st.integers(0, 10 ** 6))
def test_hypothesis_random_csr_and_partitions(n, n_und, n_parts, seed):
    rowptr, colidx = wl.random_small_graph(n, n_und, seed=seed)
    part = np.random.default_rng(seed).integers(0, n_parts, n).astype(np.int32)
    compare(rowptr, colidx, part, n_parts, dims=(3,), elem_bytes=2)
