"""ctypes binding of libretexo.so: argument marshalling only.

Every function has the name of the C entry point it calls (see
include/retexo.h).  Tensors are torch CUDA tensors (torch is used for device
memory and streams, nothing else); all arithmetic of the path happens in the
library's kernels.  There is no fallback: if the library is missing or a call
fails, a RuntimeError is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libretexo.so")
_lib = None

GCN, SAGE_MEAN, GAT, SAGE_MAX = 0, 1, 2, 3
NORM_NONE, NORM_LAYER, NORM_BATCH = 0, 1, 2
SGD, ADAM = 0, 1


class RetexoError(RuntimeError):
    pass


class _Csr(C.Structure):
    _fields_ = [("n_nodes", C.c_int64), ("n_edges", C.c_int64), ("rowptr", C.c_void_p), ("colidx", C.c_void_p)]


class _GatParams(C.Structure):
    _fields_ = [("heads", C.c_int32), ("head_dim", C.c_int32), ("a_src", C.c_void_p), ("a_dst", C.c_void_p),
                ("negative_slope", C.c_float), ("add_self_loop", C.c_int32)]


class _Mlp(C.Structure):
    _fields_ = [("d_in", C.c_int32), ("hidden", C.c_int32), ("n_classes", C.c_int32),
                ("theta", C.c_void_p), ("adam_m", C.c_void_p), ("adam_v", C.c_void_p),
                ("optimizer", C.c_int32), ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
                ("eps", C.c_float), ("step", C.c_int64), ("dropout", C.c_float), ("dropout_seed", C.c_uint64),
                ("status_out", C.c_void_p), ("norm", C.c_int32), ("norm_eps", C.c_float), ("bn_momentum", C.c_float)]


class _LmpConfig(C.Structure):
    _fields_ = [("aggr", C.c_int32), ("K", C.c_int32), ("R", C.c_int32), ("d0", C.c_int32), ("hidden", C.c_int32),
                ("n_classes", C.c_int32), ("optimizer", C.c_int32), ("lr", C.c_float), ("beta1", C.c_float),
                ("beta2", C.c_float), ("eps", C.c_float), ("eval_every", C.c_int32), ("gat_heads", C.c_int32),
                ("gat_head_dim", C.c_int32), ("gat_negative_slope", C.c_float), ("memory_is_host", C.c_int32),
                ("dropout", C.c_float), ("dropout_seed", C.c_uint64), ("gat_freeze_attention", C.c_int32),
                ("norm", C.c_int32), ("norm_eps", C.c_float), ("bn_momentum", C.c_float)]


class _LmpInputs(C.Structure):
    _fields_ = [("graph", _Csr), ("features", C.c_void_p), ("ld_features", C.c_int64), ("labels", C.c_void_p),
                ("train_idx", C.c_void_p), ("n_train", C.c_int64), ("val_idx", C.c_void_p), ("n_val", C.c_int64),
                ("test_idx", C.c_void_p), ("n_test", C.c_int64), ("part", C.c_void_p), ("n_parts", C.c_int32),
                ("theta0", C.POINTER(C.c_void_p)), ("gat_w", C.POINTER(C.c_void_p))]


class _StandardConfig(C.Structure):
    _fields_ = [("aggr", C.c_int32), ("K", C.c_int32), ("R", C.c_int32), ("d0", C.c_int32), ("hidden", C.c_int32),
                ("n_classes", C.c_int32), ("optimizer", C.c_int32), ("lr", C.c_float), ("beta1", C.c_float),
                ("beta2", C.c_float), ("eps", C.c_float)]


class _StandardOutputs(C.Structure):
    _fields_ = [("loss_history", C.c_void_p), ("val_correct", C.c_void_p), ("best_val_correct", C.c_void_p),
                ("best_iter", C.c_void_p), ("test_correct", C.c_void_p), ("test_correct_last", C.c_void_p),
                ("final_logits", C.c_void_p), ("ld_logits", C.c_int64), ("final_pred", C.c_void_p),
                ("theta_best", C.POINTER(C.c_void_p)), ("grad_last", C.POINTER(C.c_void_p)), ("status", C.c_void_p)]


class _DataVolume(C.Structure):
    _fields_ = [("lazy_lt", C.c_double), ("standard_lt", C.c_double), ("lazy_reduce", C.c_double),
                ("standard_reduce", C.c_double), ("gamma", C.c_double), ("model_size", C.c_double)]


class _LmpOutputs(C.Structure):
    _fields_ = [("loss_history", C.c_void_p), ("val_correct", C.c_void_p), ("best_val_correct", C.c_void_p),
                ("best_iter", C.c_void_p), ("test_correct", C.c_void_p), ("test_correct_last", C.c_void_p),
                ("counts", C.c_void_p), ("final_logits", C.c_void_p), ("ld_logits", C.c_int64),
                ("final_pred", C.c_void_p), ("theta_best", C.POINTER(C.c_void_p)), ("gat_best", C.POINTER(C.c_void_p)),
                ("status", C.c_void_p)]


EXPORTS = ["retexo_status_string", "retexo_version", "retexo_validate_csr", "retexo_aggregate_workspace_size",
           "retexo_aggregate", "retexo_gat_backward_workspace_size", "retexo_gat_backward", "retexo_theta_size", "retexo_theta_size_norm", "retexo_pack_rows",
           "retexo_mlp_train_step_workspace_size", "retexo_mlp_train_step_workspace_size_norm",
           "retexo_mlp_train_step", "retexo_embed_workspace_size", "retexo_embed_workspace_size_norm", "retexo_embed",
           "retexo_cross_partition_workspace_size", "retexo_cross_partition_bytes",
           "retexo_cross_partition_static_scratch_bytes", "retexo_cross_partition_bytes_static",
           "retexo_data_volume", "retexo_lmp_workspace_size", "retexo_standard_workspace_size", "retexo_standard_train",
           "retexo_gather_rows",
           "retexo_lmp_train"]


def lib():
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RetexoError("libretexo.so is missing: build it with `python -m paper_2302_13053_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.retexo_status_string.restype = C.c_char_p
        L.retexo_status_string.argtypes = [C.c_int]
        for name in ("retexo_aggregate_workspace_size", "retexo_gat_backward_workspace_size",
                     "retexo_mlp_train_step_workspace_size", "retexo_mlp_train_step_workspace_size_norm",
                     "retexo_embed_workspace_size", "retexo_embed_workspace_size_norm", "retexo_cross_partition_workspace_size",
                     "retexo_lmp_workspace_size", "retexo_cross_partition_static_scratch_bytes",
                     "retexo_standard_workspace_size"):
            getattr(L, name).restype = C.c_size_t
        L.retexo_theta_size.restype = C.c_int64
        L.retexo_theta_size_norm.restype = C.c_int64
        _lib = L
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        raise RetexoError("%s failed: %s (status %d)" % (what, lib().retexo_status_string(rc).decode(), rc))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def _csr(rowptr: torch.Tensor, colidx: torch.Tensor) -> _Csr:
    assert rowptr.dtype == torch.int64 and colidx.dtype == torch.int32
    assert rowptr.is_contiguous() and colidx.is_contiguous()
    return _Csr(rowptr.numel() - 1, colidx.numel(), rowptr.data_ptr(), colidx.data_ptr() if colidx.numel() else 0)


def retexo_version() -> int:
    return int(lib().retexo_version())


def retexo_validate_csr(rowptr: torch.Tensor, colidx: torch.Tensor):
    """Returns (number of violations, index of one of them or -1)."""
    g = _csr(rowptr, colidx)
    status = torch.zeros(2, dtype=torch.int64, device=rowptr.device)
    _check(lib().retexo_validate_csr(C.byref(g), _ptr(status), _stream()), "retexo_validate_csr")
    s = status.cpu()
    return int(s[0]), int(s[1])


def retexo_aggregate(aggr: int, rowptr: torch.Tensor, colidx: torch.Tensor, q: torch.Tensor, dim: Optional[int] = None,
                     gat: Optional[Dict] = None, concat_self: bool = True, want_f32: bool = True,
                     want_bf16: bool = False, out: Optional[torch.Tensor] = None,
                     out_bf16: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    """One message-passing round (Eq. 1).  q: fp32 [n, ld] (stride(0) is the
    leading dimension), `dim` columns are aggregated (default: all).
    Returns (out_f32 or None, out_bf16 or None)."""
    assert q.dtype == torch.float32 and q.stride(1) == 1
    n = rowptr.numel() - 1
    dim = int(q.shape[1] if dim is None else dim)
    width = 2 * dim if (aggr in (SAGE_MEAN, SAGE_MAX) and concat_self) else dim
    dev = q.device
    if want_f32 and out is None:
        out = torch.empty((n, width), dtype=torch.float32, device=dev)
    if want_bf16 and out_bf16 is None:
        out_bf16 = torch.empty((n, (width + 63) // 64 * 64), dtype=torch.bfloat16, device=dev)
    g = _csr(rowptr, colidx)
    gp = None
    keep = []
    heads = 0
    if aggr == GAT:
        a_src = gat["a_src"].to(device=dev, dtype=torch.float32).contiguous()
        a_dst = gat["a_dst"].to(device=dev, dtype=torch.float32).contiguous()
        keep += [a_src, a_dst]
        heads = int(gat["heads"])
        gp = _GatParams(heads, int(gat["head_dim"]), a_src.data_ptr(), a_dst.data_ptr(),
                        float(gat.get("negative_slope", 0.2)), int(gat.get("add_self_loop", 1)))
    need = lib().retexo_aggregate_workspace_size(C.c_int64(n), C.c_int64(colidx.numel()), C.c_int32(aggr),
                                                 C.c_int32(dim), C.c_int32(heads))
    ws = workspace if workspace is not None else _workspace(need, dev)
    rc = lib().retexo_aggregate(C.byref(g), C.c_int32(aggr), _ptr(q), C.c_int64(q.stride(0) if n > 0 else dim),
                                C.c_int32(dim), C.byref(gp) if gp is not None else None,
                                _ptr(out), C.c_int64(out.stride(0) if out is not None and n > 0 else width),
                                C.c_int32(1 if concat_self else 0),
                                _ptr(out_bf16),
                                C.c_int64(out_bf16.stride(0) if out_bf16 is not None and n > 0 else width),
                                _ptr(ws), C.c_size_t(ws.numel()), _stream())
    _check(rc, "retexo_aggregate")
    return out, out_bf16


def retexo_gat_backward(rowptr: torch.Tensor, colidx: torch.Tensor, p: torch.Tensor, gat: Dict, dz: torch.Tensor,
                        want_f32: bool = True, want_bf16: bool = False):
    """Backward of the GAT aggregation: returns (dp fp32 or None, dp bf16 or None, da_src, da_dst)."""
    assert p.dtype == torch.float32 and dz.dtype == torch.float32 and p.stride(1) == 1 and dz.stride(1) == 1
    n = rowptr.numel() - 1
    dev = p.device
    heads, dh = int(gat["heads"]), int(gat["head_dim"])
    dim = heads * dh
    a_src = gat["a_src"].to(device=dev, dtype=torch.float32).contiguous()
    a_dst = gat["a_dst"].to(device=dev, dtype=torch.float32).contiguous()
    gp = _GatParams(heads, dh, a_src.data_ptr(), a_dst.data_ptr(), float(gat.get("negative_slope", 0.2)),
                    int(gat.get("add_self_loop", 1)))
    dp = torch.empty((n, dim), dtype=torch.float32, device=dev) if want_f32 else None
    dp16 = torch.empty((n, (dim + 63) // 64 * 64), dtype=torch.bfloat16, device=dev) if want_bf16 else None
    da_src = torch.empty((heads, dh), dtype=torch.float32, device=dev)
    da_dst = torch.empty((heads, dh), dtype=torch.float32, device=dev)
    g = _csr(rowptr, colidx)
    need = lib().retexo_gat_backward_workspace_size(C.c_int64(n), C.c_int64(colidx.numel()), C.c_int32(heads), C.c_int32(dim))
    ws = _workspace(need, dev)
    rc = lib().retexo_gat_backward(C.byref(g), _ptr(p), C.c_int64(p.stride(0) if n > 0 else dim), C.byref(gp), _ptr(dz),
                                   C.c_int64(dz.stride(0) if n > 0 else dim), _ptr(dp), C.c_int64(dim), _ptr(dp16),
                                   C.c_int64(dp16.stride(0) if dp16 is not None else 0), _ptr(da_src), _ptr(da_dst),
                                   _ptr(ws), C.c_size_t(ws.numel()), _stream())
    _check(rc, "retexo_gat_backward")
    return dp, dp16, da_src, da_dst


def retexo_pack_rows(src: torch.Tensor, idx: Optional[torch.Tensor] = None, dim: Optional[int] = None,
                     transpose: bool = False, ones: bool = False, ld_multiple: int = 64):
    """bf16 batch of the rows src[idx] (all rows if idx is None).  Returns
    (dst [n_rows, round_up(dim (+1 with ones), ld_multiple)], dst_t [dim (+1 with ones), round_up(n_rows, ld_multiple)]
    or None).  With `ones`, column `dim` of dst (and row `dim` of dst_t) holds 1: the form
    retexo_mlp_train_step takes with x_has_ones.  The library needs leading dimensions that are
    multiples of 8; multiples of 64 put every row on a 128-byte line, which its bulk tensor loads prefer."""
    assert ld_multiple % 8 == 0 and ld_multiple > 0
    assert src.dtype in (torch.float32, torch.bfloat16) and src.stride(1) == 1
    dim = int(src.shape[1] if dim is None else dim)
    n_rows = int(src.shape[0] if idx is None else idx.numel())
    dev = src.device
    ld = (dim + (1 if ones else 0) + ld_multiple - 1) // ld_multiple * ld_multiple
    dst = torch.empty((n_rows, ld), dtype=torch.bfloat16, device=dev)
    dst_t = None
    ld_t = 0
    if transpose:
        ld_t = (n_rows + ld_multiple - 1) // ld_multiple * ld_multiple
        dst_t = torch.empty((dim + (1 if ones else 0), ld_t), dtype=torch.bfloat16, device=dev)
    if idx is not None:
        assert idx.dtype == torch.int32
    rc = lib().retexo_pack_rows(_ptr(src), C.c_int32(1 if src.dtype == torch.bfloat16 else 0),
                                C.c_int64(src.stride(0)), C.c_int32(dim), _ptr(idx), C.c_int64(n_rows),
                                _ptr(dst), C.c_int64(ld), _ptr(dst_t), C.c_int64(ld_t),
                                C.c_int32(1 if ones else 0), _stream())
    _check(rc, "retexo_pack_rows")
    return dst, dst_t


class Mlp:
    """Device-side state of one round's per-node model (theta, Adam moments)."""

    def __init__(self, d_in: int, hidden: int, n_classes: int, w1, b1, w2=None, b2=None, optimizer: int = ADAM,
                 lr: float = 0.003, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 device: str = "cuda", dropout: float = 0.0, dropout_seed: int = 0, layer_norm: bool = False,
                 ln_eps: float = 1e-5, ln_gamma=None, ln_beta=None, batch_norm: bool = False, bn_momentum: float = 0.1,
                 bn_mean=None, bn_var=None):
        """layer_norm: f_theta = Linear -> LayerNorm -> ReLU, gamma (default ones) and beta (default zeros) trained
        and stored at the end of theta.  batch_norm: Linear -> BatchNorm -> ReLU instead (eps = ln_eps); the running
        mean (default zeros) and variance (default ones) follow gamma and beta in theta."""
        self.d_in, self.hidden, self.n_classes = int(d_in), int(hidden), int(n_classes)
        assert not (layer_norm and batch_norm)
        self.layer_norm = bool(layer_norm) and hidden > 0
        self.batch_norm = bool(batch_norm) and hidden > 0
        self.norm = NORM_LAYER if self.layer_norm else (NORM_BATCH if self.batch_norm else NORM_NONE)
        parts = [np.asarray(w1, dtype=np.float32).ravel(), np.asarray(b1, dtype=np.float32).ravel()]
        if hidden > 0:
            parts += [np.asarray(w2, dtype=np.float32).ravel(), np.asarray(b2, dtype=np.float32).ravel()]
        if self.norm:
            parts += [np.ones(hidden, np.float32) if ln_gamma is None else np.asarray(ln_gamma, dtype=np.float32).ravel(),
                      np.zeros(hidden, np.float32) if ln_beta is None else np.asarray(ln_beta, dtype=np.float32).ravel()]
        if self.batch_norm:
            parts += [np.zeros(hidden, np.float32) if bn_mean is None else np.asarray(bn_mean, dtype=np.float32).ravel(),
                      np.ones(hidden, np.float32) if bn_var is None else np.asarray(bn_var, dtype=np.float32).ravel()]
        theta = np.concatenate(parts)
        assert theta.shape[0] == lib().retexo_theta_size_norm(C.c_int32(d_in), C.c_int32(hidden), C.c_int32(n_classes),
                                                              C.c_int32(self.norm))
        self.theta = torch.from_numpy(theta).to(device)
        self.m = torch.zeros_like(self.theta)
        self.v = torch.zeros_like(self.theta)
        self.status = torch.full((1,), -1, dtype=torch.int32, device=device)      # written by every step / embed call
        self.c = _Mlp(self.d_in, self.hidden, self.n_classes, self.theta.data_ptr(), self.m.data_ptr(),
                      self.v.data_ptr(), optimizer, lr, beta1, beta2, eps, 0, dropout, dropout_seed,
                      self.status.data_ptr(), self.norm, ln_eps, bn_momentum)

    @property
    def step(self) -> int:
        return int(self.c.step)

    def unpack(self, flat: Optional[torch.Tensor] = None) -> Dict[str, np.ndarray]:
        t = (self.theta if flat is None else flat).detach().cpu().numpy()
        out1 = self.hidden if self.hidden > 0 else self.n_classes
        o = self.d_in * out1
        d = {"w1": t[:o].reshape(self.d_in, out1), "b1": t[o:o + out1]}
        o += out1
        if self.hidden > 0:
            d["w2"] = t[o:o + self.hidden * self.n_classes].reshape(self.hidden, self.n_classes)
            o += self.hidden * self.n_classes
            d["b2"] = t[o:o + self.n_classes]
            o += self.n_classes
        if self.norm:
            d["ln_gamma"], d["ln_beta"] = t[o:o + self.hidden], t[o + self.hidden:o + 2 * self.hidden]
        if self.batch_norm:
            d["bn_mean"], d["bn_var"] = t[o + 2 * self.hidden:o + 3 * self.hidden], t[o + 3 * self.hidden:o + 4 * self.hidden]
        return d


def retexo_mlp_train_step(model: Mlp, x: torch.Tensor, y: torch.Tensor, x_has_ones: bool = False,
                          return_grad: bool = False, workspace: Optional[torch.Tensor] = None, return_dx: bool = False):
    """One full-batch iteration on the bf16 batch x [n_rows, ld] with labels y.
    x_has_ones: column d_in of x holds 1 in every row (retexo_pack_rows(ones=True)).
    Returns the loss before the update as a 0-dim device tensor (and the
    gradient, and dLoss/dx [n_rows, d_in], if asked: (loss, grad, dx) with None for what was not)."""
    assert x.dtype == torch.bfloat16 and y.dtype == torch.int32 and x.stride(1) == 1
    n_rows = x.shape[0]
    dev = x.device
    loss = torch.zeros((), dtype=torch.float32, device=dev)
    grad = torch.zeros_like(model.theta) if return_grad else None
    dx = torch.empty((n_rows, model.d_in), dtype=torch.float32, device=dev) if return_dx else None
    need = lib().retexo_mlp_train_step_workspace_size_norm(C.c_int32(model.d_in), C.c_int32(model.hidden),
                                                         C.c_int32(model.n_classes), C.c_int64(n_rows),
                                                         C.c_int32(model.norm))
    ws = workspace if workspace is not None else _workspace(need, dev)
    rc = lib().retexo_mlp_train_step(C.byref(model.c), _ptr(x), C.c_int64(x.stride(0)),
                                     C.c_int32(1 if x_has_ones else 0), _ptr(y),
                                     C.c_int64(n_rows), _ptr(loss), _ptr(grad), _ptr(dx), C.c_int64(model.d_in),
                                     _ptr(ws), C.c_size_t(ws.numel()), _stream())
    _check(rc, "retexo_mlp_train_step")
    if return_dx:
        return loss, grad, dx
    return (loss, grad) if return_grad else loss


def retexo_embed(model: Mlp, x: torch.Tensor, row_idx: Optional[torch.Tensor] = None,
                 y: Optional[torch.Tensor] = None, want_hidden: bool = False, want_hidden_bf16: bool = False,
                 want_logits: bool = False, want_pred: bool = False, workspace: Optional[torch.Tensor] = None) -> Dict:
    """Forward over rows of the bf16 matrix x; returns a dict with the
    requested outputs (`correct` is a python int when y is given)."""
    assert x.dtype == torch.bfloat16 and x.stride(1) == 1
    dev = x.device
    n_rows = int(x.shape[0] if row_idx is None else row_idx.numel())
    H, O = model.hidden, model.n_classes
    hid = torch.empty((n_rows, H), dtype=torch.float32, device=dev) if want_hidden else None
    hid16 = torch.empty((n_rows, (H + 7) // 8 * 8), dtype=torch.bfloat16, device=dev) if want_hidden_bf16 else None
    lg = torch.empty((n_rows, O), dtype=torch.float32, device=dev) if want_logits else None
    pred = torch.empty(n_rows, dtype=torch.int32, device=dev) if want_pred else None
    correct = torch.zeros(1, dtype=torch.int64, device=dev) if y is not None else None
    need = lib().retexo_embed_workspace_size_norm(C.c_int32(model.d_in), C.c_int32(H), C.c_int32(O), C.c_int64(n_rows),
                                                C.c_int32(model.norm))
    ws = workspace if workspace is not None else _workspace(need, dev)
    rc = lib().retexo_embed(C.byref(model.c), _ptr(x), C.c_int64(x.stride(0)), _ptr(row_idx), C.c_int64(n_rows),
                            _ptr(hid), C.c_int64(H), _ptr(hid16), C.c_int64(hid16.stride(0) if hid16 is not None else 0),
                            _ptr(lg), C.c_int64(O), _ptr(pred), _ptr(y), _ptr(correct), _ptr(ws),
                            C.c_size_t(ws.numel()), _stream())
    _check(rc, "retexo_embed")
    return dict(hidden=hid, hidden_bf16=hid16, logits=lg, pred=pred,
                correct=None if correct is None else int(correct.item()))


def retexo_cross_partition_bytes(rowptr: torch.Tensor, colidx: torch.Tensor, part: torch.Tensor, n_parts: int,
                                 dims: Sequence[int], elem_bytes: int = 4, per_part: bool = True) -> Dict:
    assert part.dtype == torch.int32
    dev = rowptr.device
    n = rowptr.numel() - 1
    K = len(dims)
    g = _csr(rowptr, colidx)
    scal = torch.zeros(3 + max(K, 1), dtype=torch.int64, device=dev)   # cross, pairs, total, per round...
    send = torch.zeros(n_parts, dtype=torch.int64, device=dev) if per_part else None
    recv = torch.zeros(n_parts, dtype=torch.int64, device=dev) if per_part else None
    dims_a = (C.c_int32 * max(K, 1))(*[int(d) for d in dims])
    need = lib().retexo_cross_partition_workspace_size(C.c_int64(n), C.c_int64(colidx.numel()), C.c_int32(n_parts))
    ws = _workspace(need, dev)
    base = scal.data_ptr()
    rc = lib().retexo_cross_partition_bytes(C.byref(g), _ptr(part), C.c_int32(n_parts), C.c_int32(K), dims_a,
                                            C.c_int32(elem_bytes), C.c_void_p(base), C.c_void_p(base + 8),
                                            C.c_void_p(base + 24), C.c_void_p(base + 16), _ptr(send), _ptr(recv),
                                            _ptr(ws), C.c_size_t(ws.numel()), _stream())
    _check(rc, "retexo_cross_partition_bytes")
    s = scal.cpu().numpy().view(np.uint64)
    return dict(cross_edges=int(s[0]), boundary_pairs=int(s[1]), bytes_total=int(s[2]),
                bytes_per_round=s[3:3 + K].copy(), dv_lazy_lt=2 * int(s[2]),
                send_per_part=None if send is None else send.cpu().numpy().view(np.uint64),
                recv_per_part=None if recv is None else recv.cpu().numpy().view(np.uint64))


def retexo_cross_partition_bytes_static(rowptr: torch.Tensor, colidx: torch.Tensor, part: torch.Tensor, n_parts: int,
                                        dims: Sequence[int], out: torch.Tensor, elem_bytes: int = 4) -> None:
    """The count through the entry point that allocates nothing.  This wrapper allocates nothing
    either: `out` is a caller-provided int64 device tensor of 3 + len(dims) elements that receives
    cross_edges, boundary_pairs, bytes_total and then the bytes of each round (read them as
    uint64 after synchronising)."""
    assert part.dtype == torch.int32 and out.dtype == torch.int64 and out.numel() >= 3 + len(dims)
    K = len(dims)
    g = _csr(rowptr, colidx)
    dims_a = (C.c_int32 * max(K, 1))(*[int(d) for d in dims])
    base = out.data_ptr()
    rc = lib().retexo_cross_partition_bytes_static(C.byref(g), _ptr(part), C.c_int32(n_parts), C.c_int32(K), dims_a,
                                                   C.c_int32(elem_bytes), C.c_void_p(base), C.c_void_p(base + 8),
                                                   C.c_void_p(base + 24), C.c_void_p(base + 16), None, None,
                                                   _stream())
    _check(rc, "retexo_cross_partition_bytes_static")


def retexo_gather_rows(src: torch.Tensor, idx: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """out[i] = src[idx[i]] for a fp32 matrix src (rows contiguous) and int32 row indices idx, on the device."""
    assert src.dtype == torch.float32 and idx.dtype == torch.int32 and src.stride(1) == 1
    n, dim = idx.numel(), src.shape[1]
    if out is None:
        out = torch.empty((n, dim), dtype=torch.float32, device=src.device)
    assert out.shape[0] >= n and out.shape[1] == dim and out.stride(1) == 1
    rc = lib().retexo_gather_rows(_ptr(src), C.c_int64(src.stride(0)), C.c_int32(dim), _ptr(idx), C.c_int64(n), _ptr(out),
                                  C.c_int64(out.stride(0)), _stream())
    _check(rc, "retexo_gather_rows")
    return out


def pack_theta(w: Dict[str, np.ndarray], layer_norm: bool = False, batch_norm: bool = False) -> np.ndarray:
    """theta of one round as the library lays it out; with layer_norm or batch_norm (and a hidden layer) it ends in
    [gamma | beta], taken from w["ln_gamma"], w["ln_beta"] or, if absent, ones and zeros; with batch_norm the running
    statistics follow (w["bn_mean"], w["bn_var"], else zeros and ones)."""
    parts = [np.asarray(w["w1"], dtype=np.float32).ravel(), np.asarray(w["b1"], dtype=np.float32).ravel()]
    if "w2" in w:
        parts += [np.asarray(w["w2"], dtype=np.float32).ravel(), np.asarray(w["b2"], dtype=np.float32).ravel()]
        h = np.asarray(w["b1"]).shape[0]
        if layer_norm or batch_norm:
            parts += [np.asarray(w.get("ln_gamma", np.ones(h)), dtype=np.float32).ravel(),
                      np.asarray(w.get("ln_beta", np.zeros(h)), dtype=np.float32).ravel()]
        if batch_norm:
            parts += [np.asarray(w.get("bn_mean", np.zeros(h)), dtype=np.float32).ravel(),
                      np.asarray(w.get("bn_var", np.ones(h)), dtype=np.float32).ravel()]
    return np.ascontiguousarray(np.concatenate(parts))


def pack_gat(w: Dict[str, np.ndarray]) -> np.ndarray:
    return np.ascontiguousarray(np.concatenate([np.asarray(w["w_att"], dtype=np.float32).ravel(),
                                                np.asarray(w["a_src"], dtype=np.float32).ravel(),
                                                np.asarray(w["a_dst"], dtype=np.float32).ravel()]))


class LmpProblem:
    """Inputs of a K-round run, resident either on the device (torch CUDA
    tensors) or in pinned host memory, plus the preallocated workspace and
    output buffers, so that repeated runs allocate nothing."""

    def __init__(self, aggr: int, K: int, R: int, hidden: int, n_classes: int, lr: float,
                 rowptr: np.ndarray, colidx: np.ndarray, features: np.ndarray, labels: np.ndarray,
                 train_idx: np.ndarray, val_idx: np.ndarray, test_idx: np.ndarray,
                 weights: List[Dict[str, np.ndarray]], part: Optional[np.ndarray] = None, n_parts: int = 0,
                 heads: int = 0, head_dim: int = 0, negative_slope: float = 0.2, optimizer: int = ADAM,
                 beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, eval_every: int = 1,
                 host: bool = False, want_logits: bool = True, device: str = "cuda", dropout: float = 0.0,
                 dropout_seed: int = 0, freeze_attention: bool = False, layer_norm: bool = False,
                 ln_eps: float = 1e-5, batch_norm: bool = False, bn_momentum: float = 0.1):
        self.host = bool(host)
        self.device = torch.device(device)
        n, e = rowptr.shape[0] - 1, colidx.shape[0]
        self.n, self.e, self.K, self.R, self.n_classes = n, e, K, R, n_classes
        self.cfg = _LmpConfig(aggr, K, R, features.shape[1], hidden, n_classes, optimizer, lr, beta1, beta2, eps,
                              eval_every, heads, head_dim, negative_slope, 1 if host else 0, dropout, dropout_seed,
                              1 if freeze_attention else 0,
                              NORM_LAYER if layer_norm else (NORM_BATCH if batch_norm else NORM_NONE), ln_eps, bn_momentum)

        def put(a: np.ndarray) -> torch.Tensor:
            t = torch.from_numpy(np.ascontiguousarray(a))
            return t.pin_memory() if host else t.to(self.device)

        self.rowptr, self.colidx = put(rowptr.astype(np.int64)), put(colidx.astype(np.int32))
        self.features = put(features.astype(np.float32))
        self.labels = put(labels.astype(np.int32))
        self.train_idx, self.val_idx, self.test_idx = (put(a.astype(np.int32)) for a in (train_idx, val_idx, test_idx))
        self.part = put(part.astype(np.int32)) if part is not None else None
        self.theta0 = [put(pack_theta(w, layer_norm, batch_norm)) for w in weights]
        self.gat_w = [put(pack_gat(w)) for w in weights] if aggr == GAT else None
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in
                             [self.rowptr, self.colidx, self.features, self.labels, self.train_idx, self.val_idx,
                              self.test_idx] + ([self.part] if self.part is not None else []) + self.theta0 +
                             (self.gat_w or []))

        def out(shape, dtype) -> torch.Tensor:
            t = torch.zeros(shape, dtype=dtype)
            return t.pin_memory() if host else t.to(self.device)

        self.loss_history = out((K * R,), torch.float32)
        self.val_correct = out((K * R,), torch.int64)
        self.best_val = out((K,), torch.int64)
        self.best_iter = out((K,), torch.int32)
        self.test_correct = out((K,), torch.int64)
        self.test_last = out((K,), torch.int64)
        self.counts = out((4 + K,), torch.int64)
        self.final_logits = out((n, n_classes), torch.float32) if want_logits else None
        self.final_pred = out((n,), torch.int32) if want_logits else None
        self.theta_best = [out(t.shape, torch.float32) for t in self.theta0]
        self.gat_best = [out(t.shape, torch.float32) for t in self.gat_w] if self.gat_w else None
        self.status = out((1,), torch.int32)
        self.status.fill_(-1)
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in
                             [self.loss_history, self.val_correct, self.best_val, self.best_iter, self.test_correct,
                              self.test_last, self.counts] + self.theta_best + (self.gat_best or []) +
                             ([self.final_logits, self.final_pred] if want_logits else []))

        self._theta0_arr = (C.c_void_p * K)(*[t.data_ptr() for t in self.theta0])
        self._gat_arr = (C.c_void_p * K)(*[t.data_ptr() for t in self.gat_w]) if self.gat_w else None
        self._best_arr = (C.c_void_p * K)(*[t.data_ptr() for t in self.theta_best])
        self._gat_best_arr = (C.c_void_p * K)(*[t.data_ptr() for t in self.gat_best]) if self.gat_best else None
        g = _Csr(n, e, self.rowptr.data_ptr(), self.colidx.data_ptr())
        self.inputs = _LmpInputs(g, self.features.data_ptr(), features.shape[1], self.labels.data_ptr(),
                                 self.train_idx.data_ptr(), self.train_idx.numel(),
                                 self.val_idx.data_ptr() if self.val_idx.numel() else None, self.val_idx.numel(),
                                 self.test_idx.data_ptr() if self.test_idx.numel() else None, self.test_idx.numel(),
                                 self.part.data_ptr() if self.part is not None else None, n_parts,
                                 C.cast(self._theta0_arr, C.POINTER(C.c_void_p)),
                                 C.cast(self._gat_arr, C.POINTER(C.c_void_p)) if self._gat_arr else None)
        self.outputs = _LmpOutputs(self.loss_history.data_ptr(), self.val_correct.data_ptr(),
                                   self.best_val.data_ptr(), self.best_iter.data_ptr(),
                                   self.test_correct.data_ptr(), self.test_last.data_ptr(), self.counts.data_ptr(),
                                   self.final_logits.data_ptr() if want_logits else None, n_classes,
                                   self.final_pred.data_ptr() if want_logits else None,
                                   C.cast(self._best_arr, C.POINTER(C.c_void_p)),
                                   C.cast(self._gat_best_arr, C.POINTER(C.c_void_p)) if self._gat_best_arr else None,
                                   self.status.data_ptr())
        need = lib().retexo_lmp_workspace_size(C.byref(self.cfg), C.c_int64(n), C.c_int64(e),
                                               C.c_int64(self.train_idx.numel()), C.c_int64(self.val_idx.numel()),
                                               C.c_int64(self.test_idx.numel()),
                                               C.c_int32(n_parts if part is not None else 0))
        if need == 0:
            raise RetexoError("retexo_lmp_workspace_size rejected the configuration")
        self.workspace_bytes = int(need)
        self.workspace = _workspace(need, self.device)

    def results(self) -> Dict:
        K, R = self.K, self.R
        cpu = lambda t: t.cpu().numpy()
        counts = cpu(self.counts).view(np.uint64)
        n_test = max(1, self.test_idx.numel())
        return dict(loss_history=cpu(self.loss_history).reshape(K, R),
                    val_correct=cpu(self.val_correct).view(np.uint64).reshape(K, R),
                    best_val_correct=cpu(self.best_val).view(np.uint64), best_iter=cpu(self.best_iter),
                    test_correct=cpu(self.test_correct).view(np.uint64),
                    test_correct_last=cpu(self.test_last).view(np.uint64),
                    test_acc=float(cpu(self.test_correct)[-1]) / n_test,
                    test_acc_last=float(cpu(self.test_last)[-1]) / n_test,
                    counts=dict(cross_edges=int(counts[0]), boundary_pairs=int(counts[1]),
                                bytes_total=int(counts[2]), dv_lazy_lt=int(counts[3]),
                                bytes_per_round=counts[4:4 + K].copy()),
                    final_logits=None if self.final_logits is None else cpu(self.final_logits),
                    final_pred=None if self.final_pred is None else cpu(self.final_pred),
                    theta_best=[cpu(t) for t in self.theta_best],
                    gat_best=[cpu(t) for t in self.gat_best] if self.gat_best else None,
                    status=int(cpu(self.status)[0]))


def retexo_lmp_train(problem: LmpProblem) -> None:
    """Runs the K-round loop on the current stream.  Device-resident problems
    are only enqueued; host-resident ones are copied in, run, copied out and
    synchronised by the library."""
    rc = lib().retexo_lmp_train(C.byref(problem.cfg), C.byref(problem.inputs), C.byref(problem.outputs),
                                _ptr(problem.workspace), C.c_size_t(problem.workspace.numel()), _stream())
    _check(rc, "retexo_lmp_train")


class StandardProblem:
    """Inputs, workspace and outputs of a standard (end-to-end) training run of the K-layer GNN, all on the device.
    weights[m] holds "w1" [d_m, out_m] and "b1" of layer m (other keys are ignored)."""

    def __init__(self, aggr: int, R: int, hidden: int, n_classes: int, lr: float, rowptr: np.ndarray,
                 colidx: np.ndarray, features: np.ndarray, labels: np.ndarray, train_idx: np.ndarray,
                 val_idx: np.ndarray, test_idx: np.ndarray, weights: List[Dict[str, np.ndarray]], optimizer: int = ADAM,
                 beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, want_logits: bool = True,
                 want_grad: bool = False, device: str = "cuda"):
        dev = torch.device(device)
        K = len(weights)
        n, e = rowptr.shape[0] - 1, colidx.shape[0]
        self.K, self.R, self.n = K, R, n
        self.cfg = _StandardConfig(aggr, K, R, features.shape[1], hidden, n_classes, optimizer, lr, beta1, beta2, eps)
        put = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.rowptr, self.colidx = put(rowptr.astype(np.int64)), put(colidx.astype(np.int32))
        self.features, self.labels = put(features.astype(np.float32)), put(labels.astype(np.int32))
        self.train_idx, self.val_idx, self.test_idx = (put(a.astype(np.int32)) for a in (train_idx, val_idx, test_idx))
        self.theta0 = [put(np.concatenate([np.asarray(w["w1"], dtype=np.float32).ravel(),
                                           np.asarray(w["b1"], dtype=np.float32).ravel()])) for w in weights]
        zeros = lambda shape, dtype: torch.zeros(shape, dtype=dtype, device=dev)
        self.loss_history, self.val_correct = zeros((R,), torch.float32), zeros((R,), torch.int64)
        self.best_val, self.best_iter = zeros((1,), torch.int64), zeros((1,), torch.int32)
        self.test_correct, self.test_last = zeros((1,), torch.int64), zeros((1,), torch.int64)
        self.final_logits = zeros((n, n_classes), torch.float32) if want_logits else None
        self.final_pred = zeros((n,), torch.int32) if want_logits else None
        self.theta_best = [torch.zeros_like(t) for t in self.theta0]
        self.grad_last = [torch.zeros_like(t) for t in self.theta0] if want_grad else None
        self.status = torch.full((1,), -1, dtype=torch.int32, device=dev)
        arr = lambda ts: (C.c_void_p * K)(*[t.data_ptr() for t in ts])
        self._theta0_arr, self._best_arr = arr(self.theta0), arr(self.theta_best)
        self._grad_arr = arr(self.grad_last) if want_grad else None
        g = _Csr(n, e, self.rowptr.data_ptr(), self.colidx.data_ptr())
        ptr = lambda t: t.data_ptr() if t is not None and t.numel() else None
        self.inputs = _LmpInputs(g, self.features.data_ptr(), features.shape[1], self.labels.data_ptr(),
                                 self.train_idx.data_ptr(), self.train_idx.numel(), ptr(self.val_idx), self.val_idx.numel(),
                                 ptr(self.test_idx), self.test_idx.numel(), None, 0,
                                 C.cast(self._theta0_arr, C.POINTER(C.c_void_p)), None)
        self.outputs = _StandardOutputs(self.loss_history.data_ptr(), self.val_correct.data_ptr(), self.best_val.data_ptr(),
                                        self.best_iter.data_ptr(), self.test_correct.data_ptr(), self.test_last.data_ptr(),
                                        ptr(self.final_logits), n_classes, ptr(self.final_pred),
                                        C.cast(self._best_arr, C.POINTER(C.c_void_p)),
                                        C.cast(self._grad_arr, C.POINTER(C.c_void_p)) if want_grad else None,
                                        self.status.data_ptr())
        need = lib().retexo_standard_workspace_size(C.byref(self.cfg), C.c_int64(n), C.c_int64(e),
                                                    C.c_int64(self.train_idx.numel()), C.c_int64(self.val_idx.numel()),
                                                    C.c_int64(self.test_idx.numel()))
        if need == 0:
            raise RetexoError("retexo_standard_workspace_size: configuration not supported")
        self.workspace = _workspace(need, dev)

    def results(self) -> Dict:
        cpu = lambda t: t.cpu().numpy()
        n_test = max(1, self.test_idx.numel())
        return dict(loss_history=cpu(self.loss_history), val_correct=cpu(self.val_correct).view(np.uint64),
                    best_val_correct=int(cpu(self.best_val)[0]), best_iter=int(cpu(self.best_iter)[0]),
                    test_correct=int(cpu(self.test_correct)[0]), test_correct_last=int(cpu(self.test_last)[0]),
                    test_acc=float(cpu(self.test_correct)[0]) / n_test,
                    final_logits=None if self.final_logits is None else cpu(self.final_logits),
                    final_pred=None if self.final_pred is None else cpu(self.final_pred),
                    theta_best=[cpu(t) for t in self.theta_best],
                    grad_last=[cpu(t) for t in self.grad_last] if self.grad_last else None,
                    status=int(cpu(self.status)[0]))


def retexo_standard_train(problem: StandardProblem) -> None:
    """Enqueues R iterations of standard training on the current stream."""
    rc = lib().retexo_standard_train(C.byref(problem.cfg), C.byref(problem.inputs), C.byref(problem.outputs),
                                     _ptr(problem.workspace), C.c_size_t(problem.workspace.numel()), _stream())
    _check(rc, "retexo_standard_train")


def retexo_data_volume(H, L, n_workers: float, B: float, R: float) -> dict:
    """Closed-form data volumes and gamma (Eq. 2); H = [H_0..H_K], L = [L_1..L_K].  Host only."""
    K = len(L)
    if len(H) != K + 1:
        raise RetexoError("H must hold K + 1 widths")
    h = (C.c_int64 * (K + 1))(*[int(x) for x in H])
    l = (C.c_int64 * K)(*[int(x) for x in L])
    out = _DataVolume()
    _check(lib().retexo_data_volume(C.c_int32(K), h, l, C.c_double(n_workers), C.c_double(B), C.c_double(R),
                                    C.byref(out)), "retexo_data_volume")
    return {k: getattr(out, k) for k, _ in _DataVolume._fields_}
