"""CPU checker (test infrastructure, not part of the product) of *standard* full-graph GNN training, the scheme
lazy message passing is compared with (Section 2.3): one model of K layers,
    H^0 = F,   X^m = COMBINE(H^{m-1}, AGGR(H^{m-1}))  (Eq. 1),   H^m = ReLU(X^m W_m + b_m)  for m < K,
    logits = X^K W_K + b_K,
trained end to end: every iteration runs the K aggregations forward and carries the gradient back through
them (the transposed aggregation), so a partitioned run exchanges boundary rows once per layer and direction
in every iteration instead of once per layer in all.

Plain numpy in double.  The aggregation is a sparse matrix written out from its definition and applied with
the library's sparse product; its backward pass applies the transpose of that same matrix (nothing assumes
the graph to be symmetric).  The last layer, the loss and the optimiser are those of the per-node model
checker (`oracle.Mlp` with hidden = 0).

Operand rounding (round_bf16 = True) follows the rule of the per-node model: both operands of every matrix
product are rounded to bf16, sums are wide; an aggregation takes and returns fp32 values (its output is
rounded where a product reads it); the ReLU gate is decided on the unrounded pre-activation; a bias gradient
is the product of the all-ones vector with the rounded output gradient.

Pins: tests/test_oracle_standard.py (autograd of a dense-adjacency model, the adjoint identity against the
aggregation checker, the one-layer case against oracle.Mlp)."""
from typing import Dict, List, Optional, Sequence

import numpy as np
import scipy.sparse as sp

from . import ADAM, GCN, SAGE_MEAN, Mlp, bf16_round_array


def aggregation_matrices(aggr: int, rowptr: np.ndarray, colidx: np.ndarray):
    """(S, M): X = [S H | M H] without the first block where S is None.
    GCN: M = D^-1/2 (A + I) D^-1/2 with D = degree + 1, no self block.
    SAGE mean with self-concat: S = I, M = D^-1 A (zero rows where the degree is 0)."""
    n = rowptr.shape[0] - 1
    rowptr = np.asarray(rowptr, dtype=np.int64)
    a = sp.csr_matrix((np.ones(colidx.shape[0]), np.asarray(colidx, dtype=np.int64), rowptr), shape=(n, n))
    deg = np.diff(rowptr).astype(np.float64)
    if aggr == GCN:
        nrm = sp.diags(1.0 / np.sqrt(deg + 1.0))
        return None, (nrm @ (a + sp.identity(n, format="csr")) @ nrm).tocsr()
    if aggr == SAGE_MEAN:
        inv = np.where(deg > 0, 1.0 / np.maximum(deg, 1.0), 0.0)
        return sp.identity(n, format="csr"), (sp.diags(inv) @ a).tocsr()
    raise ValueError("standard training is defined here for GCN and SAGE-mean")


def _opnd(a: np.ndarray, rounded: bool) -> np.ndarray:
    return bf16_round_array(a.astype(np.float32)).astype(np.float64) if rounded else a


class StandardGnn:
    """The K-layer model and one full-batch training iteration of it."""

    def __init__(self, aggr: int, rowptr, colidx, weights: Sequence[Dict[str, np.ndarray]], optimizer: int = ADAM,
                 lr: float = 0.003, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, round_bf16: bool = True):
        self.aggr, self.K, self.round_bf16 = aggr, len(weights), bool(round_bf16)
        self.S, self.M = aggregation_matrices(aggr, rowptr, colidx)
        # a layer's [W | b] with its optimiser state: a per-node model without hidden layer
        self.layers: List[Mlp] = []
        for w in weights:
            w1 = np.asarray(w["w1"], dtype=np.float64)
            self.layers.append(Mlp(w1.shape[0], 0, w1.shape[1], w1, w["b1"], optimizer=optimizer, lr=lr, beta1=beta1,
                                   beta2=beta2, eps=eps, round_bf16=round_bf16))

    def copy(self) -> "StandardGnn":
        o = StandardGnn.__new__(StandardGnn)
        o.__dict__.update(self.__dict__)
        o.layers = [l.copy() for l in self.layers]
        return o

    # ---- Eq. 1 and its transpose
    def aggregate(self, h: np.ndarray) -> np.ndarray:
        z = self.M @ h
        x = z if self.S is None else np.concatenate([self.S @ h, z], axis=1)
        return x.astype(np.float32).astype(np.float64) if self.round_bf16 else x      # (handed on as fp32 values)

    def aggregate_transposed(self, g: np.ndarray) -> np.ndarray:
        if self.S is None:
            d = self.M.T @ g
        else:
            half = g.shape[1] // 2
            d = self.S.T @ g[:, :half] + self.M.T @ g[:, half:]
        return d.astype(np.float32).astype(np.float64) if self.round_bf16 else d

    def _wb(self, m: int):
        u = self.layers[m].unpack()
        return u["w1"], u["b1"]

    def forward(self, features: np.ndarray):
        """All layers over all nodes; returns (X^1..X^K, pre-activations Z^1..Z^{K-1}, logits)."""
        h = np.asarray(features, dtype=np.float64)
        xs, zs = [], []
        for m in range(self.K):
            x = self.aggregate(h)
            xs.append(x)
            w, b = self._wb(m)
            z = _opnd(x, self.round_bf16) @ _opnd(w, self.round_bf16) + b
            if m < self.K - 1:
                zs.append(z)
                h = np.maximum(z, 0.0)
                if self.round_bf16:
                    h = h.astype(np.float32).astype(np.float64)
        return xs, zs, z

    def evaluate(self, features, rows, y) -> int:
        logits = self.forward(features)[2][np.asarray(rows, dtype=np.int64)]
        return int((np.argmax(logits, axis=1) == np.asarray(y)).sum())

    def train_step(self, features, labels, train_idx, return_grad: bool = False):
        """One full-batch iteration (forward, mean soft-max cross-entropy over the train rows, backward through
        every layer and aggregation, update).  Returns the loss before the update (and the gradients, one flat
        [dW | db] per layer, if asked)."""
        tr = np.asarray(train_idx, dtype=np.int64)
        y = np.ascontiguousarray(np.asarray(labels)[tr], dtype=np.int32)
        xs, zs, _ = self.forward(features)
        n = xs[0].shape[0]
        rd = self.round_bf16
        # last layer, loss and that layer's update: the per-node model checker on the train rows of X^K (it applies
        # the update itself and returns the gradients taken before it, dLoss / dX^K of those rows among them);
        # the rows of all other nodes have no gradient
        last = self.layers[-1]
        loss, g_last, dx_tr = last.train_step_dx(xs[-1][tr].astype(np.float32), y)
        grads = [None] * self.K
        grads[-1] = g_last
        g = np.zeros((n, xs[-1].shape[1]))
        g[tr] = dx_tr
        for m in range(self.K - 2, -1, -1):
            dh = self.aggregate_transposed(g)                      # gradient at H^{m+1} (0-based m: the output of layer m)
            dz = _opnd(dh * (zs[m] > 0.0), rd)                     # through the ReLU, then an operand of two products
            w, _ = self._wb(m)
            dw = _opnd(xs[m], rd).T @ dz
            db = dz.sum(axis=0)
            grads[m] = np.concatenate([dw.ravel(), db])
            if m > 0:
                g = dz @ _opnd(w, rd).T
                if rd:
                    g = g.astype(np.float32).astype(np.float64)
        for m in range(self.K - 1):
            self.layers[m].apply_update(grads[m])
        return (loss, grads) if return_grad else loss


def standard_train(aggr: int, R: int, rowptr, colidx, features, labels, train_idx, val_idx, test_idx,
                   weights: Sequence[Dict[str, np.ndarray]], optimizer: int = ADAM, lr: float = 0.003,
                   round_bf16: bool = True, forced_best_iter: Optional[int] = None) -> Dict:
    """R iterations of standard training; validation after every iteration, the earliest best iterate kept
    (forced_best_iter, a test hook: keep that 1-based iterate instead).  Per iteration a partitioned run would
    exchange boundary rows of H^1 .. H^{K-1} forward and as many gradient rows backward (Appendix A.1)."""
    labels = np.asarray(labels)
    model = StandardGnn(aggr, rowptr, colidx, weights, optimizer=optimizer, lr=lr, round_bf16=round_bf16)
    best, best_correct, best_iter = None, -1, -1
    losses, val_hist = [], []
    for r in range(1, R + 1):
        losses.append(model.train_step(features, labels, train_idx))
        c = model.evaluate(features, val_idx, labels[val_idx]) if len(val_idx) else 0
        val_hist.append(c)
        if (forced_best_iter == r) if forced_best_iter is not None else (c > best_correct):
            best, best_correct, best_iter = model.copy(), c, r
    logits = best.forward(features)[2]
    te = np.asarray(test_idx, dtype=np.int64)
    return dict(losses=np.asarray(losses), val_correct=np.asarray(val_hist), best_iter=best_iter,
                best_val_correct=best_correct, model=best, last_model=model, logits=logits,
                pred=np.argmax(logits, axis=1).astype(np.int32),
                test_correct_best=int((np.argmax(logits[te], axis=1) == labels[te]).sum()),
                test_correct_last=model.evaluate(features, te, labels[te]) if len(te) else 0,
                n_aggregations_forward=R * (model.K - 1) + 1, n_aggregations_backward=R * (model.K - 1))
