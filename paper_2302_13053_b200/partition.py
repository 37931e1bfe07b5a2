"""Host-side plan for running one lazy-message-passing round on several workers (Section 3.3 / 3.4:
each worker owns a block of nodes, and before a round it receives the representations of its boundary
nodes once; Appendix A.1 counts exactly those messages).

This module only builds index structures (numpy): which rows a rank owns, which rows it must receive from
and send to every peer, and a local CSR over [owned rows | received rows].  It holds none of the method's
arithmetic.  The exchange itself is one all-to-all of rows per round (torch.distributed); the kernels then
work on local memory only.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np


def node_ranges(n_nodes: int, world: int) -> np.ndarray:
    """Contiguous node ranges, as even as possible: rank r owns [bounds[r], bounds[r + 1])."""
    return (np.arange(world + 1, dtype=np.int64) * n_nodes) // world


def owner_of(n_nodes: int, world: int) -> np.ndarray:
    """Partition id per node for the node-range partition (the `part` array of the count entry point)."""
    b = node_ranges(n_nodes, world)
    return np.repeat(np.arange(world, dtype=np.int32), np.diff(b))


@dataclass
class RankPlan:
    rank: int
    world: int
    lo: int                       # first owned node
    hi: int                       # one past the last owned node
    recv_ids: List[np.ndarray]    # per peer: global ids of the boundary rows this rank receives (ascending)
    send_ids: List[np.ndarray]    # per peer: global ids of owned rows that peer needs (ascending)
    halo_ids: np.ndarray          # all received ids, peer by peer: local index = n_owned + position
    rowptr: np.ndarray            # int64 [n_owned + n_halo + 1]: owned rows first, then one row per received node
    colidx: np.ndarray            # int32, local indices; columns ascending inside an owned row
    halo_degree: np.ndarray       # int64 [n_halo]: the received nodes' degrees in the whole graph

    @property
    def n_owned(self) -> int:
        return self.hi - self.lo

    @property
    def n_halo(self) -> int:
        return int(self.halo_ids.shape[0])

    def recv_counts(self) -> List[int]:
        return [int(a.shape[0]) for a in self.recv_ids]

    def send_counts(self) -> List[int]:
        return [int(a.shape[0]) for a in self.send_ids]


def build_plan(rowptr: np.ndarray, colidx: np.ndarray, rank: int, world: int,
               halo_rows_carry_degree: bool = False) -> RankPlan:
    """The plan of `rank` for the node-range partition of a symmetric CSR graph.

    halo_rows_carry_degree: give every received node a local row as long as its row in the whole graph
    (filled with its own index), so that code which reads a neighbour's degree off the CSR (the GCN
    normalisation) sees the true degree; those rows are never aggregated."""
    n = rowptr.shape[0] - 1
    bounds = node_ranges(n, world)
    lo, hi = int(bounds[rank]), int(bounds[rank + 1])
    owner = owner_of(n, world)
    cols = colidx[rowptr[lo]:rowptr[hi]].astype(np.int64)
    outside = (cols < lo) | (cols >= hi)
    need = np.unique(cols[outside])                                   # boundary nodes of this rank, ascending
    need_owner = owner[need]
    recv_ids = [need[need_owner == s] for s in range(world)]
    # rows of mine that peer s needs: my nodes with a neighbour owned by s (the graph is symmetric, so they
    # are read off my own rows)
    row_of = np.repeat(np.arange(lo, hi, dtype=np.int64), np.diff(rowptr[lo:hi + 1]))
    send_ids = []
    col_owner = owner[cols]
    for s in range(world):
        send_ids.append(np.unique(row_of[col_owner == s]) if s != rank else np.zeros(0, dtype=np.int64))
    halo = np.concatenate(recv_ids) if world > 1 else np.zeros(0, dtype=np.int64)
    n_owned, n_halo = hi - lo, halo.shape[0]
    # global id -> local index: owned rows keep their order, received rows follow peer by peer
    local = np.full(n, -1, dtype=np.int64)
    local[lo:hi] = np.arange(n_owned)
    local[halo] = n_owned + np.arange(n_halo)
    halo_degree = (rowptr[halo + 1] - rowptr[halo]).astype(np.int64)
    owned_ptr = (rowptr[lo:hi + 1] - rowptr[lo]).astype(np.int64)
    owned_cols = local[cols]
    # columns ascending inside a row, in local numbering
    order = np.lexsort((owned_cols, np.repeat(np.arange(n_owned), np.diff(owned_ptr))))
    owned_cols = owned_cols[order]
    if halo_rows_carry_degree:
        tail_len = halo_degree
        tail_cols = np.repeat(n_owned + np.arange(n_halo), halo_degree)
    else:
        tail_len = np.zeros(n_halo, dtype=np.int64)
        tail_cols = np.zeros(0, dtype=np.int64)
    rp = np.concatenate([owned_ptr, owned_ptr[-1] + np.cumsum(tail_len)]).astype(np.int64)
    ci = np.concatenate([owned_cols, tail_cols]).astype(np.int32)
    return RankPlan(rank, world, lo, hi, recv_ids, send_ids, halo, rp, ci, halo_degree)


def exchange_rows(plan: RankPlan, q_owned: np.ndarray, dist) -> np.ndarray:
    """The round's one exchange (`sync_embeddings` in the paper's Section 3.4): every rank sends each peer the
    owned rows that peer needs and receives its own boundary rows, as one all-to-all with per-peer counts.
    q_owned: fp32 [n_owned x d].  Returns [n_owned + n_halo, d]: owned rows, then received rows."""
    import torch
    d = q_owned.shape[1]
    send = [q_owned[ids - plan.lo] for ids in plan.send_ids]
    send_t = torch.from_numpy(np.ascontiguousarray(np.concatenate(send) if send else np.zeros((0, d), np.float32)))
    recv_t = torch.empty((plan.n_halo, d), dtype=send_t.dtype)
    dist.all_to_all_single(recv_t, send_t, output_split_sizes=plan.recv_counts(), input_split_sizes=plan.send_counts())
    return np.concatenate([q_owned, recv_t.numpy()])


def exchanged_bytes(plan: RankPlan, dim: int, elem_bytes: int = 4) -> int:
    """Bytes this rank receives in one round of width `dim` (summed over ranks: boundary_pairs x dim x elem_bytes)."""
    return plan.n_halo * dim * elem_bytes


# ---------------------------------------------------------------- device data plane
class DeviceRound:
    """What a rank keeps on its GPU to run the aggregation of a sharded round: the local CSR over
    [owned rows | received rows], the local indices of the owned rows each peer needs, and a buffer for
    [owned | received] rows.  The exchange writes into this GPU's own memory; the aggregation kernel then reads
    local memory only (no kernel reads a peer's memory)."""

    def __init__(self, plan: RankPlan, device="cuda"):
        import torch
        self.plan = plan
        self.device = torch.device(device)
        self.rowptr = torch.from_numpy(plan.rowptr.astype(np.int64)).to(self.device)
        self.colidx = torch.from_numpy(plan.colidx.astype(np.int32)).to(self.device)
        send = np.concatenate([ids - plan.lo for ids in plan.send_ids]) if plan.world > 1 else np.zeros(0, np.int64)
        self.send_local = torch.from_numpy(send.astype(np.int32)).to(self.device)      # peer by peer
        self.n_send = int(send.shape[0])

    def exchange(self, q_owned, dist=None):
        """The round's one exchange on device tensors.  q_owned: fp32 [n_owned x d] on this GPU.  Returns fp32
        [n_owned + n_halo, d]: the owned rows, then the received rows peer by peer.  With the `nccl` backend the
        all-to-all moves device memory directly; with any other backend (`gloo`: tests on one GPU) the packed rows
        are staged through host memory."""
        import torch
        from . import binding as B
        p = self.plan
        d = q_owned.shape[1]
        q_local = torch.empty((p.n_owned + p.n_halo, d), dtype=torch.float32, device=self.device)
        q_local[:p.n_owned].copy_(q_owned)
        if p.world == 1:
            return q_local
        send = B.retexo_gather_rows(q_owned, self.send_local) if self.n_send else \
            torch.empty((0, d), dtype=torch.float32, device=self.device)
        recv = q_local[p.n_owned:]
        if dist.get_backend() == "nccl":
            dist.all_to_all_single(recv, send, output_split_sizes=p.recv_counts(), input_split_sizes=p.send_counts())
        else:
            recv_h = torch.empty((p.n_halo, d), dtype=torch.float32)
            dist.all_to_all_single(recv_h, send.cpu(), output_split_sizes=p.recv_counts(), input_split_sizes=p.send_counts())
            recv.copy_(recv_h)
        return q_local

    def aggregate(self, aggr: int, q_local, gat=None, want_bf16: bool = False):
        """AGGR (+ COMBINE) over [owned | received] rows with the library's kernel; returns the owned rows' part
        (fp32 [n_owned x width], and the bf16 copy if asked)."""
        from . import binding as B
        out, out16 = B.retexo_aggregate(aggr, self.rowptr, self.colidx, q_local, gat=gat, want_bf16=want_bf16)
        n = self.plan.n_owned
        return (out[:n], out16[:n]) if want_bf16 else out[:n]


def sharded_aggregate(round_: DeviceRound, aggr: int, q_owned, dist=None, gat=None):
    """One message-passing round of a sharded run on this rank: exchange, then local aggregation."""
    return round_.aggregate(aggr, round_.exchange(q_owned, dist), gat=gat)
