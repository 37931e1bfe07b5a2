"""Device data plane of a sharded round (paper Section 3.3 / 3.4: one exchange of boundary rows per round, then
local aggregation): the rows a rank packs for its peers and the aggregation over [owned | received] rows on the
GPU against the CPU checker's whole-graph result, first with the exchange emulated inside one process (any
number of ranks), then with two ranks that share the GPU and exchange through `gloo` (their kernels are
independent of each other: nothing on the device waits for the other rank).  The local CSR orders a row's
neighbours by local index, so sums are taken in another order than on one worker: tolerance as for any fp32
aggregation (1e-5 of the row's norm)."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _close(got, want):
    norm = np.linalg.norm(want.astype(np.float64), axis=1, keepdims=True)
    assert np.all(np.abs(got.astype(np.float64) - want) <= 1e-5 * norm + 1e-30)


@pytest.mark.parametrize("aggr", [oracle.GCN, oracle.SAGE_MEAN, oracle.SAGE_MAX])
@pytest.mark.parametrize("world", [1, 3])
def test_packed_rows_and_local_aggregation_match_the_whole_graph(aggr, world):
    from paper_2302_13053_b200 import binding as B, partition as pt, workloads as wl
    w = wl.make_config(2, scale=0.2)
    rng = np.random.default_rng(1)
    q = rng.standard_normal((w.n_nodes, 40)).astype(np.float32)
    whole = oracle.aggregate(aggr, w.rowptr, w.colidx, q)
    plans = [pt.build_plan(w.rowptr, w.colidx, r, world, halo_rows_carry_degree=aggr == oracle.GCN) for r in range(world)]
    rounds = [pt.DeviceRound(p) for p in plans]
    packed = []
    for p, rd in zip(plans, rounds):      # what every rank would hand to the transport, peer by peer
        sent = B.retexo_gather_rows(dev(q[p.lo:p.hi]), rd.send_local).cpu().numpy() if rd.n_send else np.zeros((0, 40), np.float32)
        want = np.concatenate([q[ids] for ids in p.send_ids]) if world > 1 else np.zeros((0, 40), np.float32)
        assert np.array_equal(sent, want)
        packed.append(np.split(sent, np.cumsum(p.send_counts())[:-1]) if world > 1 else [])
    for r, (p, rd) in enumerate(zip(plans, rounds)):
        recv = [packed[s][r] for s in range(world)] if world > 1 else []      # the all-to-all, emulated
        q_local = np.concatenate([q[p.lo:p.hi]] + recv)
        got = rd.aggregate(aggr, dev(q_local)).cpu().numpy()
        _close(got, whole[p.lo:p.hi])


WORKER = r"""
import os, sys
import numpy as np
sys.path.insert(0, %r)
sys.path.insert(0, os.path.join(%r, "tests"))
import torch
import torch.distributed as dist
import oracle
from paper_2302_13053_b200 import binding as B, partition as pt, workloads as wl
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
torch.cuda.set_device(0)                               # both ranks share the one GPU; their kernels are independent
w = wl.make_config(4, scale=0.02)                      # every rank draws the same seeded graph
q = w.features
whole = oracle.aggregate(w.aggr, w.rowptr, w.colidx, q)
plan = pt.build_plan(w.rowptr, w.colidx, rank, world)
rd = pt.DeviceRound(plan)
q_owned = torch.from_numpy(np.ascontiguousarray(q[plan.lo:plan.hi])).cuda()
q_local = rd.exchange(q_owned, dist)
assert np.array_equal(q_local[plan.n_owned:].cpu().numpy(), q[plan.halo_ids])
got = rd.aggregate(w.aggr, q_local).cpu().numpy()
want = whole[plan.lo:plan.hi]
norm = np.linalg.norm(want.astype(np.float64), axis=1, keepdims=True)
assert np.all(np.abs(got.astype(np.float64) - want) <= 1e-5 * norm + 1e-30)
t = torch.tensor([plan.n_halo * q.shape[1] * 4], dtype=torch.int64)
dist.all_reduce(t)
ref = oracle.cross_partition(w.rowptr, w.colidx, pt.owner_of(w.n_nodes, world), world, [q.shape[1]], 4)
assert int(t.item()) == ref["bytes_total"]
torch.cuda.synchronize()
dist.barrier()
dist.destroy_process_group()
print("rank %%d ok" %% rank)
""" % (ROOT, ROOT)


def test_two_ranks_sharing_the_gpu_exchange_once_and_aggregate_locally(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-3000:]
    assert "rank 0 ok" in out.stdout and "rank 1 ok" in out.stdout
