"""Host-side plan of the sharded round (node-range partition, boundary-row exchange once per round, Section
3.3 / 3.4 and Appendix A.1): the rows exchanged are exactly the messages the cross-partition count counts,
and a rank that aggregates over [owned rows | received rows] gets the single-worker result bit for bit.
Two gloo ranks on CPU carry out the exchange itself."""
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2302_13053_b200 import partition as pt
from paper_2302_13053_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("world", [1, 2, 3, 5])
def test_plans_send_what_the_peers_receive_and_match_the_message_count(world):
    w = wl.make_config(2, scale=0.1)
    n = w.n_nodes
    plans = [pt.build_plan(w.rowptr, w.colidx, r, world) for r in range(world)]
    for r, p in enumerate(plans):
        assert p.lo == pt.node_ranges(n, world)[r] and p.n_owned == p.hi - p.lo
        for s, q in enumerate(plans):
            np.testing.assert_array_equal(p.send_ids[s], q.recv_ids[r])      # what r sends to s is what s expects from r
        assert p.recv_ids[r].shape[0] == 0 and p.send_ids[r].shape[0] == 0
    ref = oracle.cross_partition(w.rowptr, w.colidx, pt.owner_of(n, world), world, [w.d0, w.hidden, w.hidden], 4)
    assert sum(p.n_halo for p in plans) == ref["boundary_pairs"]
    np.testing.assert_array_equal([p.n_halo for p in plans], ref["recv_per_part"])
    np.testing.assert_array_equal([sum(p.send_counts()) for p in plans], ref["send_per_part"])
    for m, d in enumerate([w.d0, w.hidden, w.hidden]):
        assert sum(pt.exchanged_bytes(p, d) for p in plans) == int(ref["bytes_per_round"][m])


@pytest.mark.parametrize("aggr", [oracle.GCN, oracle.SAGE_MEAN, oracle.SAGE_MAX, oracle.GAT])
def test_aggregating_over_owned_plus_received_rows_equals_the_whole_graph_result(aggr):
    w = wl.make_config(3, scale=0.05)
    rng = np.random.default_rng(3)
    q = rng.standard_normal((w.n_nodes, 8)).astype(np.float32)
    gat = dict(heads=2, head_dim=4, a_src=rng.standard_normal((2, 4)).astype(np.float32),
               a_dst=rng.standard_normal((2, 4)).astype(np.float32)) if aggr == oracle.GAT else None
    whole = oracle.aggregate(aggr, w.rowptr, w.colidx, q, gat=gat)
    world = 3
    for r in range(world):
        p = pt.build_plan(w.rowptr, w.colidx, r, world, halo_rows_carry_degree=aggr == oracle.GCN)
        q_local = np.concatenate([q[p.lo:p.hi], q[p.halo_ids]])                 # what the exchange delivers
        got = oracle.aggregate(aggr, p.rowptr, p.colidx, q_local, rows=np.arange(p.n_owned), gat=gat)
        np.testing.assert_array_equal(got, whole[p.lo:p.hi])


WORKER = r"""
import os, sys
import numpy as np
sys.path.insert(0, %r)
import torch.distributed as dist
import oracle
from paper_2302_13053_b200 import partition as pt
from paper_2302_13053_b200 import workloads as wl
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = wl.make_config(2, scale=0.1)                     # every rank draws the same seeded graph
q = w.features
whole = oracle.aggregate(w.aggr, w.rowptr, w.colidx, q)
plan = pt.build_plan(w.rowptr, w.colidx, rank, world)
q_local = pt.exchange_rows(plan, np.ascontiguousarray(q[plan.lo:plan.hi]), dist)      # the round's one exchange
assert q_local.shape[0] == plan.n_owned + plan.n_halo
assert np.array_equal(q_local[plan.n_owned:], q[plan.halo_ids])
got = oracle.aggregate(w.aggr, plan.rowptr, plan.colidx, q_local, rows=np.arange(plan.n_owned))
assert np.array_equal(got, whole[plan.lo:plan.hi])                                    # bit for bit
# bytes on the wire against the count: sum over ranks of received rows x width x 4
import torch
t = torch.tensor([plan.n_halo * q.shape[1] * 4], dtype=torch.int64)
dist.all_reduce(t)
ref = oracle.cross_partition(w.rowptr, w.colidx, pt.owner_of(w.n_nodes, world), world, [q.shape[1]], 4)
assert int(t.item()) == ref["bytes_total"], (int(t.item()), ref["bytes_total"])
# the per-iteration gradient average (the paper's reducer): row-weighted mean of the ranks' gradients; checked
# without operand rounding, because dL = (softmax - onehot) / n_rows is rounded after the division and
# n_rows differs between a rank's share and the whole batch
tr = w.train_idx[(w.train_idx >= plan.lo) & (w.train_idx < plan.hi)]
ws = wl.initial_weights(w)[0]
def grad_on(x, idx):
    m = oracle.Mlp(x.shape[1], w.hidden, w.n_classes, ws["w1"], ws["b1"], ws["w2"], ws["b2"], optimizer=oracle.SGD, lr=0.0,
                   round_bf16=False)
    return m.train_step(x, w.labels[idx], row_idx=None, return_grad=True)[1]
local = grad_on(np.ascontiguousarray(whole[tr]), tr) * len(tr) if len(tr) else np.zeros(oracle.Mlp(whole.shape[1], w.hidden, w.n_classes, ws["w1"], ws["b1"], ws["w2"], ws["b2"]).theta.shape[0])
g = torch.from_numpy(local.copy())
dist.all_reduce(g)
n_all = torch.tensor([len(tr)], dtype=torch.int64)
dist.all_reduce(n_all)
assert int(n_all.item()) == len(w.train_idx)
want = grad_on(np.ascontiguousarray(whole[w.train_idx]), w.train_idx)
assert np.abs(g.numpy() / len(w.train_idx) - want).max() <= 1e-12 * max(1.0, np.abs(want).max())
dist.barrier()
dist.destroy_process_group()
print("rank %%d ok" %% rank)
""" % ROOT


def test_two_gloo_ranks_exchange_boundary_rows_once_and_reproduce_the_round(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29531", str(script)],
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-3000:]
    assert "rank 0 ok" in out.stdout and "rank 1 ok" in out.stdout
