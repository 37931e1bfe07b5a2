"""Pins for the CPU checker's cross-partition message/byte count
(Section 2.1 boundary nodes, Appendix A.1 data volume)."""
import os

import numpy as np
import pytest

import oracle
from paper_2302_13053_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "cross_partition_hand_cases.txt")


def hand_cases():
    cases = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = [c.strip() for c in line.split("|")]
        edges = [tuple(int(t) for t in e.split("-")) for e in f[2].split()]
        ints = lambda s: [int(t) for t in s.split()]
        cases.append((f[0], int(f[1]), edges, ints(f[3]), int(f[4]), int(f[5]), int(f[6]), ints(f[7]), ints(f[8])))
    return cases


@pytest.mark.parametrize("case", hand_cases(), ids=lambda c: c[0])
def test_hand_worked_cases(case):
    name, n, edges, part, n_parts, ce, bp, send, recv = case
    rowptr, colidx = wl.csr_from_edge_list(n, edges)
    out = oracle.cross_partition(rowptr, colidx, np.array(part), n_parts, [7, 3], 4)
    assert out["cross_edges"] == ce
    assert out["boundary_pairs"] == bp
    assert list(out["send_per_part"]) == send
    assert list(out["recv_per_part"]) == recv
    assert list(out["bytes_per_round"]) == [bp * 7 * 4, bp * 3 * 4]
    assert out["bytes_total"] == bp * 10 * 4
    # Appendix A.1: DV^lazy_lt = 2 * (sum_i B_i) * (H_0 + sum H_m) bytes
    assert out["dv_lazy_lt"] == 2 * bp * (7 + 3) * 4


def brute(rowptr, colidx, part, n_parts):
    pairs = set()
    ce = 0
    n = rowptr.shape[0] - 1
    for u in range(n):
        for v in colidx[rowptr[u]:rowptr[u + 1]]:
            if part[u] != part[v]:
                ce += 1
                pairs.add((u, int(part[v])))
    send = np.zeros(n_parts, dtype=np.uint64)
    recv = np.zeros(n_parts, dtype=np.uint64)
    for u, p in pairs:
        send[part[u]] += 1
        recv[p] += 1
    return ce, len(pairs), send, recv


@pytest.mark.parametrize("seed", range(6))
def test_random_graphs_match_set_based_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(5, 120))
    rowptr, colidx = wl.random_small_graph(n, int(rng.integers(0, 4 * n)), seed=seed)
    n_parts = int(rng.integers(1, 9))
    part = rng.integers(0, n_parts, n).astype(np.int32)
    out = oracle.cross_partition(rowptr, colidx, part, n_parts, [5], 2)
    ce, bp, send, recv = brute(rowptr, colidx, part, n_parts)
    assert (out["cross_edges"], out["boundary_pairs"]) == (ce, bp)
    np.testing.assert_array_equal(out["send_per_part"], send)
    np.testing.assert_array_equal(out["recv_per_part"], recv)
    assert out["boundary_pairs"] <= out["cross_edges"]
    assert out["send_per_part"].sum() == out["recv_per_part"].sum() == bp
    assert out["bytes_total"] == bp * 5 * 2


def test_single_partition_is_zero_and_node_level_is_twice_the_undirected_edges():
    w = wl.make_config(1)
    n_und = w.n_edges // 2
    one = oracle.cross_partition(w.rowptr, w.colidx, np.zeros(w.n_nodes, dtype=np.int32), 1, [1433, 64, 64])
    assert one["cross_edges"] == 0 and one["boundary_pairs"] == 0 and one["bytes_total"] == 0
    node = oracle.cross_partition(w.rowptr, w.colidx, np.arange(w.n_nodes, dtype=np.int32), w.n_nodes,
                                  [1433, 64, 64])
    assert node["cross_edges"] == 2 * n_und == node["boundary_pairs"]
    assert node["bytes_total"] == 2 * n_und * (1433 + 64 + 64) * 4
    np.testing.assert_array_equal(node["send_per_part"], np.diff(w.rowptr).astype(np.uint64))
    np.testing.assert_array_equal(node["recv_per_part"], np.diff(w.rowptr).astype(np.uint64))


def test_relabelling_partitions_keeps_totals():
    w = wl.make_config(2, scale=0.1)
    a = oracle.cross_partition(w.rowptr, w.colidx, w.part, w.n_parts, [500, 128, 128])
    perm = np.random.default_rng(0).permutation(w.n_parts).astype(np.int32)
    b = oracle.cross_partition(w.rowptr, w.colidx, perm[w.part], w.n_parts, [500, 128, 128])
    assert (a["cross_edges"], a["boundary_pairs"], a["bytes_total"]) == \
           (b["cross_edges"], b["boundary_pairs"], b["bytes_total"])
    np.testing.assert_array_equal(a["send_per_part"], b["send_per_part"][perm])
    np.testing.assert_array_equal(a["recv_per_part"], b["recv_per_part"][perm])
