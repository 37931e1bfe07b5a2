#!/usr/bin/env python
"""Benchmark of the lazy-message-passing hot path on B200.

One "step" is one pass of the whole hot path over one synthetic workload: the
cross-partition count, then for each of the K rounds one full-graph
aggregation, R training iterations of the round's per-node model (with
validation every iteration and best-iterate tracking) and the emission of the
next representations — i.e. one end-to-end K-round training run.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl reference]

Prints one JSON line.  `value` = edges aggregated per second of whole-job time
(K rounds x directed edges / step time, summed over replicas); `ms_per_step`
is the end-to-end K-round train time.  With --gpus N > 1 (under torchrun) every
rank runs an independent replica: the path is specified for one GPU, without
sharding or collectives.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "edges aggregated/s"
UNIT = "edges/s"

import hashlib

CSRC = os.path.join(ROOT, "paper_2302_13053_b200", "csrc")


def source_fingerprint(names) -> str:
    """First 12 hex digits of the SHA-256 of the named kernel sources: the counters below are only valid
    for the kernels they were captured from."""
    h = hashlib.sha256()
    for name in names:
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


# DRAM bytes (read + write) per launch, from one-pass ncu captures summarised under profiles/.  Each table names
# the sources of the kernels it was captured from and their fingerprint at capture time; where the sources
# have changed since, `traffic` is reported as null.
AGG_SOURCES = ("aggregate.cu",)
AGG_DRAM_TRAFFIC = {
    "fingerprint": "b169e13d7982",      # profiles/agg_kernels_cfg4.txt, profiles/agg_rows_kernel_cfg5.txt
    "bytes": {("cfg4_sage_reddit_like", 1): 14.68e9, ("cfg4_sage_reddit_like", 2): 6.24e9,
              ("cfg4_sage_reddit_like", 3): 5.99e9, ("cfg5_gcn_products_like", 1): 46.68e9,
              ("cfg5_gcn_products_like", 2): 102.92e9, ("cfg5_gcn_products_like", 3): 102.93e9}}
# one stand-alone training iteration (its tensor-core launches and reduce_update_kernel): profiles/mlp_iteration_cfg4.txt
STEP_SOURCES = ("gemm_tc.cu", "mlp_fused.cu", "mlp.cu", "mlp_kernels.cuh", "tc_common.cuh", "launch_overlap.cuh")
STEP_DRAM_TRAFFIC = {
    "fingerprint": "16175fb90a45",
    "bytes": {("cfg4_sage_reddit_like", 1): 1.241e9, ("cfg4_sage_reddit_like", 2): 0.823e9,
              ("cfg4_sage_reddit_like", 3): 0.3415e9}}


# Peak of the L2 -> SM path in GB/s, as the profiler normalises it: in the section capture of the slab gather
# (profiles/agg_kernels_cfg4.txt) the kernel delivered 15.6 / 16.7 TB/s of neighbour rows, all of them out of L2
# (L1 hit rate 2 %), at lts__throughput = 68.3 / 72.5 % of peak; both give 22.9 TB/s for 100 %.
L2_PEAK_GBS = 22900.0


def measured_traffic(table, sources, key):
    if table["fingerprint"] is None or table["fingerprint"] != source_fingerprint(sources):
        return None
    return table["bytes"].get(key)


def min_time_roofline(flops: float, nbytes: float, ms: float, peaks) -> dict:
    """Min-time roofline of a dense product (or a chain of them): the slower of flops / tensor peak
    and bytes / HBM peak is the bound; `achieved` is quoted in that bound's unit."""
    t_tensor = flops / (peaks["bf16_sustained"] * 1e12) * 1e3
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e3
    if t_hbm >= t_tensor:
        return dict(bound="hbm", achieved=nbytes / ms / 1e6, peak=peaks["hbm_gbs"], unit="GB/s",
                    algorithmic_bytes=nbytes, flops=flops, tflops=flops / ms / 1e9, min_ms=t_hbm)
    return dict(bound="tensor", achieved=flops / ms / 1e9, peak=peaks["bf16_sustained"], unit="TFLOP/s",
                algorithmic_bytes=nbytes, flops=flops, gbs=nbytes / ms / 1e6, min_ms=t_tensor)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm), window="last warm-up step and timed region, 100 ms period")


def max_over_ranks(value: float, world: int, device: str = "cuda") -> float:
    """The slowest rank's time: what a multi-replica step takes."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(edges_per_step: int, world: int, ms_per_step: float) -> float:
    """Replicas only: every rank aggregates its own copy of the graph, so the job's throughput is
    world x the per-replica edges over the slowest replica's step time."""
    return world * edges_per_step / (ms_per_step * 1e-3)


def build_workload(index: int, scale: float):
    from paper_2302_13053_b200 import workloads as wl
    t = time.time()
    w = wl.make_config(index, scale=scale)
    ws = wl.initial_weights(w)
    return w, ws, time.time() - t


FREEZE_ATTENTION = False      # --freeze-attention: GAT with its aggregator's parameters fixed (one aggregation per round)


def make_problem(w, ws, host: bool, R: int):
    from paper_2302_13053_b200 import binding as B
    return B.LmpProblem(w.aggr, w.K, R, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                        w.train_idx, w.val_idx, w.test_idx, ws, part=w.part, n_parts=w.n_parts, heads=w.heads,
                        head_dim=w.head_dim, negative_slope=w.negative_slope, host=host,
                        freeze_attention=FREEZE_ATTENTION)


def launches_per_step(w, R: int) -> int:
    """Kernels the library launches in one K-round run (memsets and copies not counted)."""
    from paper_2302_13053_b200 import workloads as wl
    total = 3 + 1                                    # label gathers, history fill
    n_parts = w.n_parts
    total += (2 if n_parts <= 8192 else 3) + 1       # count kernels + finalize + pack
    for rd in w.round_dims():
        h = rd["hidden"]
        gat_forward = 1 + 1 + 2                      # W_att^T copy, projection, scores + rows
        trained_gat = w.aggr == wl.GAT and not FREEZE_ATTENTION
        if trained_gat:
            total += 1                               # the round's input as a bf16 operand
            total += 3 * gat_forward                 # last and kept iterate for the test rows, kept iterate for the emission
        elif w.aggr == wl.GAT:
            total += 1 + gat_forward + 2             # input operand, one aggregation; train / val batches
        else:
            total += 3 + 2                           # prep, warp rows, block rows; train / val batches
        step = 5 if h > 0 else 3                     # products, fused middle, reduce + update (+ weight copies once)
        if trained_gat:
            # the aggregator is trained with the model: per iteration projection + aggregation + batches before
            # the step, input gradient inside it, kept copy + scatter + backward (4) + dW_att + update after it
            step += gat_forward + 2 + 1 + 8
            total += gat_forward + 2                 # the last iterate's own validation pass
        total += R * step + 1 + (2 if h > 0 else 1)       # (the update kernel's last block books the validation count
                                                          #  that rides along; the last iterate's is booked by a kernel of its own)
        total += (2 if h > 0 else 1) + 1             # stand-alone validation of the last iterate + snapshot
        total += 1 + 2 * (4 if h > 0 else 2)         # test rows gathered, then kept and last iterate (weight copies + products)
        total += 3 if h > 0 else 2                   # emission of Q^m / final logits
    return total


def time_calls(fn, reps: int, warm: int = 3):
    import torch
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in evs:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    ts = [a.elapsed_time(b) for a, b in evs]
    return statistics.mean(ts), min(ts)


def measure_l2_gather_peak(rp, ci, n: int, e: int) -> float:
    """Ceiling of the L2 -> SM path for a CSR gather, measured with the library's own gather on a matrix
    that fits L2 whole (64 fp32 columns: 256-byte rows, every neighbour row a hit): bytes delivered to
    the SMs per second, in GB/s."""
    import torch
    from paper_2302_13053_b200 import binding as B
    d = 64
    q = torch.rand((n, d), dtype=torch.float32, device="cuda")
    out = torch.empty((n, 64), dtype=torch.bfloat16, device="cuda")
    fn = lambda: B.retexo_aggregate(B.SAGE_MEAN, rp, ci, q, dim=d, concat_self=False, want_f32=False, out_bf16=out)
    _, best_ms = time_calls(fn, 5)
    return (e * (4 * d + 4) + 8 * (n + 1) + n * d * 2) / best_ms / 1e6


def aggregation_phases(w, ws, peaks, rp, ci, l2_peak):
    """Times every round's aggregation alone, in the launch configuration of the K-round run, and says
    which ceiling binds: the L2 -> SM path where the kernel gathers from L2-resident column slabs (its DRAM
    traffic is a small fraction of the bytes it delivers), HBM otherwise."""
    import torch
    from paper_2302_13053_b200 import binding as B
    from paper_2302_13053_b200 import workloads as wl
    dev = "cuda"
    n, e = w.n_nodes, w.n_edges
    out = []
    for rd, wt in zip(w.round_dims(), ws):
        m, d = rd["round"], rd["agg_dim"]
        ld = (rd["rep_dim"] + 31) // 32 * 32
        if m == 1:
            q = torch.zeros((n, ld), dtype=torch.float32, device=dev)
            q[:, :w.d0] = torch.from_numpy(w.features).to(dev)
        else:
            q = torch.rand((n, ld), dtype=torch.float32, device=dev)
        width = rd["d_in"]
        x16 = torch.empty((n, (width + 63) // 64 * 64), dtype=torch.bfloat16, device=dev)
        if w.aggr == wl.GAT:
            hd = w.heads * w.head_dim
            p = torch.randn((n, (hd + 31) // 32 * 32), dtype=torch.float32, device=dev)
            gat = dict(heads=w.heads, head_dim=w.head_dim, a_src=torch.from_numpy(wt["a_src"]),
                       a_dst=torch.from_numpy(wt["a_dst"]), negative_slope=w.negative_slope, add_self_loop=1)
            fn = lambda: B.retexo_aggregate(w.aggr, rp, ci, p, dim=hd, gat=gat, want_f32=False, out_bf16=x16)
            alg = e * (4 * hd + 4 * w.heads + 4) + 8 * (n + 1) + n * hd * 2
        else:
            fn = lambda: B.retexo_aggregate(w.aggr, rp, ci, q, dim=d, want_f32=False, out_bf16=x16)
            alg = e * (4 * d + 4) + 8 * (n + 1) + n * width * 2
        mean_ms, best_ms = time_calls(fn, 5)
        traffic = measured_traffic(AGG_DRAM_TRAFFIC, AGG_SOURCES, (w.name, m))
        alg_gbs = alg / mean_ms / 1e6
        ph = dict(kernel="aggregate", workload=w.name, round=m, calls_per_step=1, ms=mean_ms, best_ms=best_ms,
                  algorithmic_bytes=alg, algorithmic_gbs=alg_gbs, edges_per_s=e / mean_ms * 1e3, traffic=traffic,
                  dram_gbs=(traffic / mean_ms / 1e6) if traffic else None,
                  dram_frac=(traffic / mean_ms / 1e6 / peaks["hbm_gbs"]) if traffic else None, x16=x16)
        if traffic and traffic < 0.25 * alg:
            ph.update(bound="l2", achieved=alg_gbs, peak=L2_PEAK_GBS, unit="GB/s",
                      ceiling="L2 -> SM path: neighbour rows gathered from L2-resident column slabs (DRAM traffic is %.2f "
                              "of the bytes delivered); peak = 100 %% of the profiler's lts__throughput, from the "
                              "section capture of this kernel; the plain kernel on a 64-column matrix that fits L2 "
                              "whole delivers %.1f TB/s in this run" % (traffic / alg, (l2_peak or 0.0) / 1e3))
        elif traffic:
            ph.update(bound="hbm", achieved=traffic / mean_ms / 1e6, peak=peaks["hbm_gbs"], unit="GB/s",
                      ceiling="HBM: achieved = DRAM bytes (ncu) / time; L2 serves the rest of the %.1f TB/s delivered"
                              % (alg_gbs / 1e3))
        else:
            # no DRAM counters for this workload / these sources: the bytes delivered are an upper bound of the
            # DRAM bytes, so this fraction can exceed 1 where L2 serves part of the gather
            ph.update(bound="hbm", achieved=alg_gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                      ceiling="HBM (no DRAM counters for this workload: achieved = bytes delivered / time)")
        out.append(ph)
    return out


def phase_breakdown(w, ws, R: int, peaks, l2_peak=None):
    """Times each entry point alone, at the shapes and launch configuration the
    K-round run uses, and derives the roofline figures per kernel."""
    import torch
    from paper_2302_13053_b200 import binding as B
    dev = "cuda"
    rp = torch.from_numpy(w.rowptr).to(dev)
    ci = torch.from_numpy(w.colidx).to(dev)
    n, e = w.n_nodes, w.n_edges
    tr = torch.from_numpy(w.train_idx).to(dev)
    va = torch.from_numpy(w.val_idx).to(dev)
    y = torch.from_numpy(w.labels).to(dev)
    y_tr, y_va = y[tr.long()].contiguous(), y[va.long()].contiguous()
    if l2_peak is None and n * 64 * 4 < 100e6:
        l2_peak = measure_l2_gather_peak(rp, ci, n, e)
    agg = aggregation_phases(w, ws, peaks, rp, ci, l2_peak)
    phases = []
    for rd, wt, ag in zip(w.round_dims(), ws, agg):
        m = rd["round"]
        width = rd["d_in"]
        x16 = ag.pop("x16")
        phases.append(ag)
        # the round's model at its training / validation / full shapes
        model = B.Mlp(rd["d_in"], rd["hidden"], w.n_classes, wt["w1"], wt["b1"], wt.get("w2"), wt.get("b2"), lr=w.lr)
        xtr, _ = B.retexo_pack_rows(x16, tr, dim=width, ones=True)
        xva, _ = B.retexo_pack_rows(x16, va, dim=width)
        H, O = rd["hidden"], w.n_classes
        n_tr, n_va = tr.numel(), va.numel()
        # Algorithmic bytes, counted per product: every product reads each operand once and writes its result
        # once (bf16 activations and gradients, fp32 weight gradients).  chain_bytes counts the launch sequence
        # as it is built instead: the class product, the loss and the gated back-propagation are one kernel
        # (Hd read once, no logits), the ReLU bits replace the gate operand, and the weight-gradient products
        # re-read X, Hd, dL and dHd.
        if H > 0:
            flops_step = 2.0 * n_tr * (2 * width * H + 3 * H * O)
            flops_fwd = lambda rows: 2.0 * rows * (width * H + H * O)
            bytes_fwd = lambda rows: 2.0 * (rows * width + width * H + rows * H) + 2.0 * (rows * H + H * O) + 4.0 * rows
            opt = 7 * 4.0 * (width * H + H * O)                                  # theta, m, v in and out, gradient in
            bytes_step = (2.0 * (n_tr * width + width * H + n_tr * H)            # Hd = ReLU(X W1 + b1)
                          + 2.0 * (n_tr * H + H * O + n_tr * O)                   # logits, loss, dL
                          + 2.0 * (n_tr * O + H * O + 2 * n_tr * H)               # dHd = (dL W2^T) gated by Hd
                          + 2.0 * (n_tr * H + n_tr * O) + 4.0 * H * O             # dW2
                          + 2.0 * (n_tr * width + n_tr * H) + 4.0 * width * H     # dW1
                          + opt)
            chain_bytes = (2.0 * (n_tr * width + width * H + n_tr * H) + n_tr * H / 8.0      # forward: X, W1 in; Hd and its bits out
                           + 2.0 * (n_tr * H + H * O) + n_tr * H / 8.0 + 2.0 * n_tr * 64 + 2.0 * n_tr * H   # fused middle
                           + 2.0 * (n_tr * H + n_tr * 64) + 2.0 * (n_tr * width + n_tr * H)   # the two weight-gradient products
                           + opt)
        else:
            flops_step = 2.0 * n_tr * 2 * width * O
            flops_fwd = lambda rows: 2.0 * rows * width * O
            bytes_fwd = lambda rows: 2.0 * (rows * width + width * O) + 4.0 * rows
            bytes_step = (2.0 * (n_tr * width + width * O + n_tr * O) + 2.0 * (n_tr * width + n_tr * O)
                          + 4.0 * width * O + 7 * 4.0 * width * O)
            chain_bytes = bytes_step + 2.0 * n_tr * (64 - O) * 2
        import ctypes as C
        need = B.lib().retexo_mlp_train_step_workspace_size(C.c_int32(width), C.c_int32(H), C.c_int32(O),
                                                            C.c_int64(n_tr))
        ws_step = torch.empty(int(need), dtype=torch.uint8, device=dev)
        mean_ms, best_ms = time_calls(lambda: B.retexo_mlp_train_step(model, xtr, y_tr, x_has_ones=True, workspace=ws_step), 10)
        phases.append(dict(kernel="mlp_train_step", round=m, calls_per_step=R, ms=mean_ms, best_ms=best_ms,
                           traffic=measured_traffic(STEP_DRAM_TRAFFIC, STEP_SOURCES, (w.name, m)),
                           chain_bytes=chain_bytes, chain_min_ms=chain_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3,
                           tensor_min_ms=flops_step / (peaks["bf16_sustained"] * 1e12) * 1e3,
                           **min_time_roofline(flops_step, bytes_step, mean_ms, peaks)))
        mean_ms, best_ms = time_calls(lambda: B.retexo_embed(model, xva, y=y_va), 10)
        phases.append(dict(kernel="embed_validation", round=m, calls_per_step=0, ms=mean_ms, best_ms=best_ms,
                           note="stand-alone call; inside the K-round run validation rides along in the training forward",
                           **min_time_roofline(flops_fwd(n_va), bytes_fwd(n_va), mean_ms, peaks)))
        if H > 0:
            mean_ms, best_ms = time_calls(lambda: B.retexo_embed(model, x16, want_hidden=True), 3, warm=1)
            fl = 2.0 * n * width * H
            nb = 2.0 * (n * width + width * H) + 4.0 * n * H          # fp32 Q^m out
        else:
            mean_ms, best_ms = time_calls(lambda: B.retexo_embed(model, x16, want_logits=True, want_pred=True), 3, warm=1)
            fl = 2.0 * n * width * O
            nb = 2.0 * (n * width + width * O) + 4.0 * n * O + 4.0 * n
        phases.append(dict(kernel="embed_all_rows", round=m, calls_per_step=1, ms=mean_ms, best_ms=best_ms,
                           **min_time_roofline(fl, nb, mean_ms, peaks)))
        del model, xtr, xva, ws_step, x16
    part = torch.from_numpy(w.part).to(dev)
    dims = [rd["rep_dim"] for rd in w.round_dims()]
    mean_ms, best_ms = time_calls(lambda: B.retexo_cross_partition_bytes(rp, ci, part, w.n_parts, dims, 4,
                                                                         per_part=False), 5)
    alg = 8 * e + 8 * (n + 1) + 4 * n
    phases.append(dict(kernel="cross_partition_count", round=0, calls_per_step=1, ms=mean_ms, best_ms=best_ms,
                       bound="hbm", algorithmic_bytes=alg, achieved=alg / mean_ms / 1e6, peak=peaks["hbm_gbs"],
                       unit="GB/s"))
    for p in phases:
        p["frac"] = p["achieved"] / p["peak"]
    return phases, l2_peak


def iteration_only(w, ws, m: int, calls: int = 12):
    """Runs `calls` stand-alone training iterations of round m's model at the shapes phase_breakdown times
    (training rows only, column of ones in the batch) and nothing else after the round's input is built:
    what a profiler capture of the iteration wants (`--iteration-only M`).  The batch holds synthetic
    values of the aggregated rows' shape: the kernels' work does not depend on them."""
    import torch
    from paper_2302_13053_b200 import binding as B
    rd, wt = w.round_dims()[m - 1], ws[m - 1]
    tr = torch.from_numpy(w.train_idx).to("cuda")
    y_tr = torch.from_numpy(w.labels).to("cuda")[tr.long()].contiguous()
    g = torch.Generator(device="cuda").manual_seed(m)
    x = torch.randn((tr.numel(), rd["d_in"]), generator=g, device="cuda", dtype=torch.float32)
    xtr, _ = B.retexo_pack_rows(x, None, ones=True)
    del x
    model = B.Mlp(rd["d_in"], rd["hidden"], w.n_classes, wt["w1"], wt["b1"], wt.get("w2"), wt.get("b2"), lr=w.lr)
    for _ in range(calls):
        B.retexo_mlp_train_step(model, xtr, y_tr, x_has_ones=True)
    torch.cuda.synchronize()
    print(json.dumps(dict(iteration_only=m, calls=calls, rows=int(tr.numel()), d_in=rd["d_in"], hidden=rd["hidden"],
                          status=int(model.status.item()))))


def second_large_graph_aggregation(peaks, l2_peak):
    """The aggregation rounds of the other of the two largest graphs (the products-shaped GCN run), timed
    alone like the rounds of the benchmarked workload, so that one run reports both."""
    import torch
    w5, ws5, gen_s = build_workload(5, 1.0)
    rp = torch.from_numpy(w5.rowptr).to("cuda")
    ci = torch.from_numpy(w5.colidx).to("cuda")
    out = aggregation_phases(w5, ws5, peaks, rp, ci, l2_peak)
    for p in out:
        p.pop("x16", None)
        p["frac"] = p["achieved"] / p["peak"]
    return out


def standard_training(w, ws, R: int, lazy_ms_per_step: float, counts: dict):
    """Standard (end-to-end) training of the same K-layer model on the same kernels (Section 2.3), timed beside
    the lazy run: the time of one iteration is the difference between a run of 12 and a run of 4 iterations
    (set-up, X^1 = AGGR(F) and the closing evaluation passes cancel), and the bytes a partitioned run would
    exchange follow from the cross-partition count: per iteration K - 1 forward and K - 1 gradient exchanges of
    the boundary rows at the hidden width, against one exchange per layer in all for the lazy run."""
    import torch
    from paper_2302_13053_b200 import binding as B

    def run(iters):
        prob = B.StandardProblem(w.aggr, iters, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features, w.labels,
                                 w.train_idx, w.val_idx, w.test_idx, ws, want_logits=False)
        B.retexo_standard_train(prob)                 # warm-up
        torch.cuda.synchronize()
        ms, _ = time_calls(lambda: B.retexo_standard_train(prob), 2, warm=0)
        res = prob.results()
        del prob
        torch.cuda.empty_cache()
        return ms, res
    short, _ = run(4)
    long, res = run(12)
    per_iter = (long - short) / 8.0
    fixed = max(short - 4 * per_iter, 0.0)
    pairs = int(counts["boundary_pairs"])
    lazy_bytes = int(counts["bytes_total"])
    std_bytes = pairs * 4 * (w.d0 + R * 2 * (w.K - 1) * w.hidden)
    est = fixed + R * per_iter
    return dict(ms_per_iteration=per_iter, fixed_ms=fixed, est_ms_for_R_iterations=est, R=R,
                aggregations_per_iteration=2 * (w.K - 1), lazy_ms_per_step=lazy_ms_per_step,
                time_ratio_standard_over_lazy=est / lazy_ms_per_step,
                exchanged_bytes_standard=std_bytes, exchanged_bytes_lazy=lazy_bytes,
                gamma_messages=std_bytes / lazy_bytes if lazy_bytes else None, status=res["status"],
                loss_first_last=[float(res["loss_history"][0]), float(res["loss_history"][-1])],
                note="one GPU, no exchange: the time ratio compares computation only; gamma_messages counts the "
                     "boundary rows a partitioned run of either scheme would send (one direction, features included "
                     "once), without the gradient all-reduce")


def oracle_sample(w, ws, R: int, budget_s: float = 75.0, budget_train: int = 2048):
    """Times the CPU checker on the workload within about budget_s seconds and scales to one full step
    (K rounds).  Every round's aggregation and the cross-partition count run in full where a short probe
    says they fit the budget (otherwise on sampled destination rows, scaled by edges); the training
    iteration and the forward pass are always timed on budget_train rows and scaled by rows."""
    import oracle
    rng = np.random.default_rng(0)
    n, e = w.n_nodes, w.n_edges
    deg = np.diff(w.rowptr)
    gat_of = lambda wt: dict(heads=w.heads, head_dim=w.head_dim, a_src=wt["a_src"], a_dst=wt["a_dst"])

    def aggregate(q, wt, rows):
        t = time.time()
        if w.aggr == 2:
            oracle.aggregate(2, w.rowptr, w.colidx, q, rows=rows, gat=gat_of(wt))
        else:
            oracle.aggregate(w.aggr, w.rowptr, w.colidx, q, rows=rows)
        return time.time() - t

    inputs = []
    for rd in w.round_dims():
        d = w.heads * w.head_dim if w.aggr == 2 else rd["rep_dim"]
        inputs.append(w.features if (rd["round"] == 1 and w.aggr != 2) else rng.standard_normal((n, d)).astype(np.float32))
    probe_rows = np.sort(rng.choice(n, size=min(n, 512), replace=False))
    probe_edges = max(1, int(deg[probe_rows].sum()))
    est = [aggregate(q, wt, probe_rows) * e / probe_edges for q, wt in zip(inputs, ws)]
    est_count = e / 8e6                                           # the count walks every entry once on one core
    full = sum(est) + est_count <= 0.75 * budget_s
    rows = None if full else np.sort(rng.choice(n, size=min(n, 1536), replace=False))
    sample_edges = e if full else int(deg[rows].sum())
    total = 0.0
    detail = []
    for rd, wt, q in zip(w.round_dims(), ws, inputs):
        t_agg = aggregate(q, wt, rows) * (e / max(1, sample_edges))
        n_tr = len(w.train_idx)
        sub = min(n_tr, budget_train)
        x = rng.standard_normal((sub, rd["d_in"])).astype(np.float32)
        y = w.labels[w.train_idx[:sub]]
        m = oracle.Mlp(rd["d_in"], rd["hidden"], w.n_classes, wt["w1"], wt["b1"], wt.get("w2"), wt.get("b2"), lr=w.lr)
        t = time.time()
        m.train_step(x, y)
        t_step = (time.time() - t) * (n_tr / sub)
        t = time.time()
        m.embed(x, y=y, want_logits=False)
        t_fwd_row = (time.time() - t) / sub
        t_round = t_agg + R * (t_step + t_fwd_row * len(w.val_idx)) + t_fwd_row * (n + 2 * len(w.test_idx))
        detail.append(dict(round=rd["round"], aggregate_s=t_agg, train_step_s=t_step, round_s=t_round))
        total += t_round
    count_s = None
    if full:
        t = time.time()
        oracle.cross_partition(w.rowptr, w.colidx, w.part, w.n_parts, [rd["rep_dim"] for rd in w.round_dims()], 4)
        count_s = time.time() - t
        total += count_s
    else:
        total += est_count
    detail.append(dict(count_s=count_s if count_s is not None else est_count))
    what = ("every round's aggregation and the cross-partition count in full" if full else
            "aggregation of %d sampled rows (%d edges), scaled by edges; the count estimated" % (len(rows), sample_edges))
    sample = "%s; one training iteration + forward on %d train rows per round, scaled by rows to %d rows and R=%d" % (
        what, min(len(w.train_idx), budget_train), len(w.train_idx), R)
    kind = ("oracle, aggregation and count in full, training step extrapolated from %d rows" % min(len(w.train_idx), budget_train)
            if full else "oracle, aggregation and training step extrapolated from samples")
    return total, detail, sample, kind


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w, ws, _ = build_workload(args.config, args.scale)
    R = args.iters or w.R
    times = []
    sample = kind = ""
    # the whole run (warm-up and timed steps) is kept to a few minutes: each step gets its share of ~150 s
    per_step = max(4.0, 150.0 / max(1, args.steps + args.warmup))
    for _ in range(args.warmup):
        oracle_sample(w, ws, R, budget_s=min(per_step, 8.0), budget_train=256)
    for _ in range(args.steps):
        t, detail, sample, kind = oracle_sample(w, ws, R, budget_s=per_step)
        times.append(t)
    step_s = statistics.mean(times)
    value = w.K * w.n_edges / step_s
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=step_s * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=w.name, n_nodes=w.n_nodes, n_edges=w.n_edges, K=w.K, R=R,
                            note="CPU checker; each step is a bounded sample of the workload, scaled to the whole"),
                cpu_baseline=dict(value=value, unit=UNIT, cores=oracle.n_threads(), kind=kind, sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4, help="workload 1..5 (default 4: the Reddit-shaped SAGE run)")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the workload (profiling captures only)")
    ap.add_argument("--iters", type=int, default=0, help="override R, the iterations per round")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-breakdown", action="store_true")
    ap.add_argument("--freeze-attention", action="store_true",
                    help="GAT workloads: keep the aggregator's parameters fixed (the round aggregates once)")
    ap.add_argument("--iteration-only", type=int, default=0, metavar="M",
                    help="run a dozen stand-alone training iterations of round M's model and exit (profiler captures)")
    ap.add_argument("--standard-only", type=int, default=0, metavar="ITERS",
                    help="run ITERS iterations of standard training twice and nothing else (profiler captures)")
    ap.add_argument("--no-standard", action="store_true",
                    help="skip the standard-training comparison (same model trained end to end on the same kernels)")
    ap.add_argument("--no-second-graph", action="store_true",
                    help="with the default workload, do not time the products-shaped graph's aggregation rounds as well")
    args = ap.parse_args()
    global FREEZE_ATTENTION
    FREEZE_ATTENTION = bool(args.freeze_attention)
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2302_13053_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl")
    peaks = load_peaks()

    w, ws, gen_s = build_workload(args.config, args.scale)
    if args.iteration_only:
        iteration_only(w, ws, args.iteration_only)
        return
    if args.standard_only:
        sp = B.StandardProblem(w.aggr, args.standard_only, w.hidden, w.n_classes, w.lr, w.rowptr, w.colidx, w.features,
                               w.labels, w.train_idx, w.val_idx, w.test_idx, ws, want_logits=False)
        for _ in range(2):
            B.retexo_standard_train(sp)
        torch.cuda.synchronize()
        r = sp.results()
        print(json.dumps(dict(standard_only=args.standard_only, status=r["status"], loss=[float(x) for x in r["loss_history"]])))
        return
    R = args.iters or w.R
    prob = make_problem(w, ws, host=False, R=R)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    n_warm = max(args.warmup, 3)
    for _ in range(n_warm - 1):
        B.retexo_lmp_train(prob)
    barrier()
    # nvidia-smi needs a few hundred ms before its first sample: it is started ahead of the last warm-up
    # step (the same load as the timed steps), so that the timed region is covered from its start
    sampler = ClockSampler(local)
    sampler.start()
    B.retexo_lmp_train(prob)
    barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(args.steps):
        B.retexo_lmp_train(prob)
    stop.record()
    barrier()
    clocks = sampler.stop()
    ms = max_over_ranks(start.elapsed_time(stop), world)
    ms_per_step = ms / args.steps
    edges_per_step = w.K * w.n_edges
    value = whole_job_value(edges_per_step, world, ms_per_step)
    res = prob.results()

    # ---- end to end through the host-buffer entry point: H2D of all inputs and D2H of results inside
    e2e = None
    if not args.no_e2e:
        del prob
        torch.cuda.empty_cache()
        hprob = make_problem(w, ws, host=True, R=R)
        for _ in range(2):
            B.retexo_lmp_train(hprob)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            B.retexo_lmp_train(hprob)          # synchronises the stream before returning
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0, world)
        e2e = dict(value=world * edges_per_step * args.steps / dt, unit=UNIT, ms_per_step=dt / args.steps * 1e3,
                   h2d_bytes_per_step=int(hprob.h2d_bytes), d2h_bytes_per_step=int(hprob.d2h_bytes))
        del hprob
        torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic",
                config=dict(workload=w.name, n_nodes=w.n_nodes, n_edges=w.n_edges, d0=w.d0, K=w.K, R=R,
                            hidden=w.hidden, n_classes=w.n_classes, n_train=len(w.train_idx),
                            aggregation_dtype="fp32 in, fp32 accumulate", mlp_dtype="bf16 operands, fp32 accumulate",
                            l2="inputs larger than L2, no flush" if w.n_nodes * w.d0 * 4 > 126e6 else
                               "working set fits L2: reported warm",
                            parallelism="replicas only" if world > 1 else "single GPU",
                            generation_s=round(gen_s, 1)),
                clocks=clocks, e2e=e2e, gpu_launches=launches_per_step(w, R) * args.steps,
                end_to_end_train_time_ms=ms_per_step,
                accuracy=dict(test=res["test_acc"], test_last_iterate=res["test_acc_last"]),
                counts=dict(cross_edges=res["counts"]["cross_edges"], boundary_pairs=res["counts"]["boundary_pairs"],
                            bytes_total=res["counts"]["bytes_total"]))

    if not args.no_breakdown:
        phases, l2_peak = phase_breakdown(w, ws, R, peaks)
        for p in phases:
            p["share_of_step"] = p["ms"] * p["calls_per_step"] / ms_per_step
        dom = max(phases, key=lambda p: p["share_of_step"])
        line["roofline"] = dict(kernel="%s round %d" % (dom["kernel"], dom["round"]), bound=dom["bound"],
                                achieved=dom["achieved"], peak=dom["peak"], unit=dom["unit"], frac=dom["frac"],
                                traffic=dom.get("traffic"), peak_source=peaks["source"],
                                share_of_step=dom["share_of_step"],
                                algorithmic_bytes=dom.get("algorithmic_bytes"), flops=dom.get("flops"),
                                tflops=dom.get("tflops"), ms=dom["ms"], min_ms=dom.get("min_ms"),
                                chain_bytes=dom.get("chain_bytes"), chain_min_ms=dom.get("chain_min_ms"),
                                tensor_min_ms=dom.get("tensor_min_ms"),
                                note="one training iteration (forward product, fused class product / loss / gated "
                                     "back-propagation, two weight-gradient products, reduce + update); min-time roofline "
                                     "counted per product: bytes / HBM peak exceeds flops / tensor peak, so HBM is the "
                                     "bound; chain_* counts the bytes of the launch sequence as built"
                                if dom["kernel"] == "mlp_train_step" and dom["bound"] == "hbm" else
                                "one training iteration: tensor-bound"
                                if dom["kernel"] == "mlp_train_step" else "CSR gather-reduce (aggregation kernels)")
        # the memory-bound side of the path, each round against the ceiling that binds it; with the default
        # workload the rounds of the other large graph follow
        agg = [p for p in phases if p["kernel"] == "aggregate"]
        if args.config == 4 and args.scale == 1.0 and world == 1 and not args.no_second_graph:
            torch.cuda.empty_cache()
            agg += second_large_graph_aggregation(peaks, l2_peak)
        line["roofline_aggregation"] = [
            dict(workload=p.get("workload", w.name), round=p["round"], bound=p["bound"], achieved=p["achieved"],
                 peak=p["peak"], unit="GB/s", frac=p["frac"], traffic=p.get("traffic"), ms=p["ms"],
                 edges_per_s=p["edges_per_s"], algorithmic_gbs=p["algorithmic_gbs"], dram_gbs=p["dram_gbs"],
                 dram_frac=p["dram_frac"], hbm_peak=peaks["hbm_gbs"], ceiling=p["ceiling"])
            for p in agg]
        line["l2"] = dict(peak_gbs=L2_PEAK_GBS, peak_source="ncu lts__throughput, profiles/agg_kernels_cfg4.txt",
                          plain_gather_on_l2_resident_matrix_gbs=l2_peak)
        line["phases"] = [dict(kernel=p["kernel"], round=p["round"], ms=round(p["ms"], 4), calls=p["calls_per_step"],
                               share=round(p["share_of_step"], 4), bound=p["bound"], achieved=round(p["achieved"], 2),
                               unit=p["unit"], frac=round(p["frac"], 4),
                               **({"edges_per_s": p["edges_per_s"]} if "edges_per_s" in p else {}))
                          for p in phases]
    if not args.no_standard and world == 1 and w.aggr in (B.GCN, B.SAGE_MEAN):
        torch.cuda.empty_cache()
        line["standard_training"] = standard_training(w, ws, R, ms_per_step, res["counts"])
    if not args.no_cpu_baseline:
        import oracle
        t, detail, sample, kind = oracle_sample(w, ws, R)
        line["cpu_baseline"] = dict(value=edges_per_step / t, unit=UNIT, cores=oracle.n_threads(), kind=kind,
                                    sample=sample, est_step_s=t, detail=detail)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
