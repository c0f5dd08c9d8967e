#!/usr/bin/env python
"""Benchmark of full-graph GCN training epochs on seeded synthetic graphs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C1..C5] [--impl ours|reference]

One step = one training epoch (all layers forward, loss, all layers backward, Adam) over the
whole graph.  Prints ONE JSON line.  `value` is epochs/s with every input resident in HBM;
`e2e` is the same iteration through the host-buffer entry point (host->device copies of the
features, labels, mask, parameters and moments and device->host copies of the results inside
the timed region); `roofline` covers the aggregation kernels (the dominant kernel), with the
per-call durations measured by CUDA events on the launching stream during the timed steps;
`cpu_baseline` is the CPU oracle timed on a bounded sample of the same workload.  After the headline
(workload C5) short legs run the other four workloads (`workloads`), the wide dense products of C4
alone (`gemm_c4`) and the measured denominators that are not in MEASURED_PEAKS.json (`denominators`:
TF32 matmul throughput, row-gather rate from an L2-resident and from an HBM-resident table).

With N > 1 (launched by torch.distributed.run) every rank trains an independent replica of the
same workload -- the path does not shard -- and `value` is the sum over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2501_01951_b200 import synth

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one aggregation call comes from ncu, which
# may only capture a small case here; the figures below are that capture (profiles/spmm_call_rmat4M_w128.md).
TRAFFIC_NOTE = ("DRAM traffic of a call does not grow in proportion to its size on these graphs (the L2 hit rate of the gathers "
                "falls as the input outgrows the L2: 113 B per stored entry beyond the compulsory rows on the 4M-node case, 180 B "
                "on the 30M-node workload in the one single-pass full-size capture taken, 131.2 GB per call), so the small-case "
                "capture is not scaled to this workload and `traffic` is null here; small_case_capture holds the measured figure "
                "of the same kernels on the case that may be captured, ideal_static_cache a model of this workload's traffic")
SMALL_CASE_CAPTURE = dict(case="R-MAT 4,000,000 nodes, 70,522,690 stored entries, width 128 (profiles/spmm_call_rmat4M_w128.md)",
                          dram_bytes_per_call=12_054_734_848, alg_bytes_per_call=4_692_181_528, ratio=2.57)


METRIC = "full-graph GCN train epochs/s"
UNIT = "epochs/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------ clocks

class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.path = f"/tmp/mixgcn_clocks_{os.getpid()}.csv"
        self.proc = None
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(index), "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------------------------ workload

def spmm_plan(wl, orders, sparse_levels=0, rows_only=False):
    """Widths of the DENSE-input aggregation calls of one epoch: (width, count) per layer, from the
    ordering; the backward aggregations of the top `sparse_levels` layers run row-sparse and are not counted,
    nor is the last layer's forward aggregation when it is restricted to train rows (`rows_only`)."""
    from paper_2501_01951_b200 import binding as mg
    calls = []
    L = len(wl.dims) - 1
    for l in range(L):
        agg = orders[l] == mg.ORDER_AGG_FIRST
        w = wl.dims[l] if agg else wl.dims[l + 1]
        k = 1 + (0 if (l == 0 and agg) else 1)          # forward, plus backward unless first layer agg-first
        if l >= L - sparse_levels and k == 2:
            k = 1                                        # this layer's backward aggregation takes the row-sparse path
        if rows_only and l == L - 1:
            k -= 1                                       # forward aggregation on train rows only
        calls.append((w, k))
    return calls


def spmm_alg_bytes(n, nnz, w):
    """Compulsory bytes of one aggregation of width w: row pointers, column ids, values, one read
    of the input rows, one write of the output rows."""
    return 8 * (n + 1) + 4 * nnz + 4 * nnz + 4 * n * w + 4 * n * w


def gemm_flops(n, dims, orders, bwd_rows=None, fwd_rows_last=None):
    """2*M*N*K over the dense products of one epoch (forward, dW, and dX where it exists).
    bwd_rows[l] (default n) is the number of rows layer l's backward products run on (the compacted
    rows of a row-sparse backward); fwd_rows_last likewise for the last layer's forward product."""
    f = 0
    L = len(dims) - 1
    for l in range(L):
        rb = n if bwd_rows is None or bwd_rows[l] is None else bwd_rows[l]
        rf = fwd_rows_last if (l == L - 1 and fwd_rows_last is not None) else n
        nb = 1 if l == 0 else 2
        f += 2 * dims[l] * dims[l + 1] * (rf + nb * rb)
    return f


def gemm_min_bytes(n, dims, bwd_rows=None, fwd_rows_last=None):
    """Minimum HBM bytes of the dense products of one epoch: forward reads rows x d_in, writes rows x d_out;
    dW reads both; dX reads rows x d_out, writes rows x d_in (weights are negligible)."""
    bts = 0
    L = len(dims) - 1
    for l in range(L):
        rb = n if bwd_rows is None or bwd_rows[l] is None else bwd_rows[l]
        rf = fwd_rows_last if (l == L - 1 and fwd_rows_last is not None) else n
        nb = 1 if l == 0 else 2
        bts += 4 * (dims[l] + dims[l + 1]) * (rf + nb * rb)
    return bts


def build_problem(wl, device):
    src, dst = synth.rmat_graph(wl.n, wl.undirected_edges, wl.seed("graph"), device=device)
    torch.cuda.synchronize()
    return src, dst


def replicas_throughput(ms_local, steps, world, device):
    """Whole-job throughput of `world` independent replicas: the slowest rank's time (max over ranks)
    bounds the job, and every rank completed `steps` epochs in it.  Returns (max ms, epochs/s)."""
    ms = float(ms_local)
    if world > 1:
        tt = torch.tensor([ms], dtype=torch.float64, device=device)
        torch.distributed.all_reduce(tt, op=torch.distributed.ReduceOp.MAX)
        ms = float(tt.item())
    return ms, world * steps / (ms / 1e3)


L2_BYTES = 126e6          # B200 L2 capacity (nominal)


def ideal_cache_floor(deg, n, nnz, w):
    """DRAM bytes of one aggregation if an ideal STATIC cache of the L2's size held the most-gathered rows of
    the input: every cached row is read once, every gather of another row goes to DRAM, index / values /
    output move once.  `deg[v]` = number of rows that gather row v (the in-degree; the entry count on a
    symmetric graph).  Not a bound for schedules that order work to share gathers (the column-ordered
    long-row segments do), but the yardstick for gathers that arrive in an order unrelated to their targets."""
    row_bytes = 4 * w
    k = int(L2_BYTES // row_bytes)
    d = torch.sort(deg.to(torch.int64), descending=True).values
    cached_refs = int(d[:k].sum().item())
    cached_rows = int((d[:k] > 0).sum().item())
    gathers_to_dram = (nnz - cached_refs) + cached_rows
    return int(8 * (n + 1) + 8 * nnz + 4 * n * w + row_bytes * gathers_to_dram), k, cached_refs / max(nnz, 1)


def measure_denominators(mg, ctx, dev):
    """Peaks that MEASURED_PEAKS.json does not hold, measured the same way in this run: fp32 matmul with TF32
    allowed (8192^3, best of 5, CUDA events) and the row-gather rate of an L2-resident (64 MB) and an
    HBM-resident (4 GB) table of 512-byte rows."""
    out = {}
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        a = torch.randn(8192, 8192, device=dev); b = torch.randn(8192, 8192, device=dev)
        best = float("inf")
        for i in range(8):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); c = a @ b; e1.record(); torch.cuda.synchronize()
            if i >= 3:
                best = min(best, e0.elapsed_time(e1))
        out["tf32_tflops_measured"] = round(2 * 8192 ** 3 / best / 1e9, 1)
        del a, b, c
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old
    sink = torch.zeros(1, device=dev)
    for name, rows in (("l2_gather_gbs", (64 << 20) // 512), ("hbm_gather_gbs", (4 << 30) // 512)):
        table = torch.ones(rows, 128, device=dev)
        best = float("inf")
        for i in range(6):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); total = mg.probe_gather(ctx, table, 4096, sink, seed=i + 1); e1.record(); torch.cuda.synchronize()
            if i >= 2:
                best = min(best, e0.elapsed_time(e1))
        out[name] = round(total * 512 / best / 1e6, 1)
        del table
    torch.cuda.empty_cache()
    out["how"] = ("torch.matmul fp32 with TF32 allowed, 8192^3, best of 5; mixgcn_probe_gather on a 64 MB / 4 GB table of "
                  "512-byte rows, best of 4")
    return out


def gemm_peak_for(prec_name, peaks, denoms):
    """(TFLOP/s, label) of the tensor-core peak for the operand type the products ran in."""
    if prec_name == "bf16":
        return peaks["bf16_tflops"], f"bf16 matmul burst ({peaks['source']})"
    if prec_name == "tf32":
        if denoms and denoms.get("tf32_tflops_measured"):
            return denoms["tf32_tflops_measured"], "tf32 matmul burst (measured in this run)"
        return peaks["bf16_tflops"] * 1.1 / 2.25, "bf16 burst x nominal tf32/bf16 ratio"
    return None, "fp32 FMA (no tensor-core peak)"


def timed_epochs(tr, mg, ctx, steps, warmup, t0, barrier):
    """`warmup` untimed epochs, then `steps` epochs between CUDA events with per-launch phase timing on."""
    t = t0
    for _ in range(warmup):
        t += 1
        tr.epoch(t)
    barrier()
    _, _, launches_before = mg.ctx_profile_read(ctx)
    paths_before = mg.ctx_gemm_paths(ctx)
    mg.ctx_profile_enable(ctx, True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(steps):
        t += 1
        tr.epoch(t)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    phase_ms, phase_launches, launches_after = mg.ctx_profile_read(ctx)
    mg.ctx_profile_enable(ctx, False)
    paths_after = mg.ctx_gemm_paths(ctx)
    paths = {k: paths_after[k] - paths_before[k] for k in paths_after}
    return t, ms_total, phase_ms, int(launches_after - launches_before), paths


def backward_rows(tr, mg, n):
    """Rows the dense products of each layer's backward ran on (compacted rows where layer_bwd took that path)."""
    rows = []
    for l, d in enumerate(tr.descs):
        cnt = int(d.gout_row_count)
        rows_flag = bool(d.flags & mg.LAYER_OUT_ROWS_ONLY)
        compacted = bool(d.gout_row_mask) and cnt > 0 and tr.orders[l] == mg.ORDER_AGG_FIRST and (4 * cnt < n or rows_flag or bool(d.gout_plan))
        rows.append(cnt if compacted else None)
    return rows


def phase_figures(mg, wl, tr, n, nnz, steps, phase_ms, peaks, denoms, prec_name, train_rows_only=False, cached_first=False):
    """Aggregation and dense-product figures of `steps` timed epochs from the per-launch phase times."""
    plan = spmm_plan(wl, tr.orders, tr.row_sparse_levels, train_rows_only)
    if cached_first and tr.orders[0] == mg.ORDER_AGG_FIRST:
        plan[0] = (plan[0][0], plan[0][1] - 1)
    calls = sum(k for _, k in plan) * steps
    alg_bytes = sum(spmm_alg_bytes(n, nnz, w) * k for w, k in plan) * steps
    gather = sum(4 * nnz * w * k for w, k in plan) * steps
    spmm_ms = phase_ms["spmm"]
    agg = dict(calls=calls, avg_call_ms=round(spmm_ms / max(calls, 1), 4), alg_bytes_per_call=int(alg_bytes / max(calls, 1)),
               alg_gbs=round(alg_bytes / (spmm_ms / 1e3) / 1e9, 1) if spmm_ms > 0 else 0.0,
               gather_gbs=round(gather / (spmm_ms / 1e3) / 1e9, 1) if spmm_ms > 0 else 0.0)
    agg["frac_of_hbm_peak"] = round(agg["alg_gbs"] / peaks["hbm_gbs"], 4)
    if denoms and denoms.get("l2_gather_gbs"):
        agg["gather_frac_of_l2_gather_rate"] = round(agg["gather_gbs"] / denoms["l2_gather_gbs"], 4)
    bwd_rows = backward_rows(tr, mg, n)
    n_train = int(tr.train_mask.sum().item())
    fwd_rows_last = n_train if (train_rows_only and tr.orders[-1] == mg.ORDER_AGG_FIRST) else None
    flops = gemm_flops(n, wl.dims, tr.orders, bwd_rows, fwd_rows_last) * steps
    gbytes = gemm_min_bytes(n, wl.dims, bwd_rows, fwd_rows_last) * steps
    gemm_ms = phase_ms["gemm"]
    tfl = flops / (gemm_ms / 1e3) / 1e12 if gemm_ms > 0 else 0.0
    peak, peak_label = gemm_peak_for(prec_name, peaks, denoms)
    gemm = dict(tflops=round(tfl, 2), dtype=prec_name, peak_tflops=round(peak, 1) if peak else None, peak_is=peak_label,
                frac_of_peak=round(tfl / peak, 4) if peak else None,
                min_hbm_gbs=round(gbytes / (gemm_ms / 1e3) / 1e9, 1) if gemm_ms > 0 else 0.0,
                frac_of_hbm_peak=round(gbytes / (gemm_ms / 1e3) / 1e9 / peaks["hbm_gbs"], 4) if gemm_ms > 0 else 0.0,
                ms_per_epoch=round(gemm_ms / steps, 3))
    if prec_name == "bf16":
        gemm["frac_of_sustained_peak"] = round(tfl / peaks["bf16_tflops_sustained"], 4)
    return agg, gemm, bwd_rows, plan


def make_trainer(mg, ctx, wl, dev, prec, args=None):
    from paper_2501_01951_b200.train import GcnTrainer, round4
    src, dst = build_problem(wl, dev)
    g = mg.graph_create(ctx, wl.n, src, dst)
    del src, dst
    torch.cuda.empty_cache()
    kw = {}
    if args is not None:
        kw = dict(n_chunks=args.chunks, row_sparse=args.row_sparse if args.row_sparse == "auto" else int(args.row_sparse),
                  train_rows_only=args.train_rows_only, row_plans=not args.no_row_plans,
                  cache_first_aggregation=args.cache_first_aggregation)
    tr = GcnTrainer(ctx, g, wl.dims, prec, **kw)
    X0 = synth.normal_features(g.n, wl.dims[0], wl.seed("features"), device=dev, ld=round4(wl.dims[0]))
    y = synth.uniform_labels(g.n, wl.classes, wl.seed("labels"), device=dev)
    m = synth.bernoulli_mask(g.n, wl.mask_p, wl.seed("mask"), device=dev)
    Ws, bs = synth.make_weights(wl, device=dev)
    tr.set_params(Ws, bs)
    tr.set_inputs(X0, y, m)
    mg.ctx_reserve(ctx, 64 << 20)
    torch.cuda.synchronize()
    return g, tr, X0, y, m, Ws, bs


def workload_leg(mg, key, dev, local_rank, peaks, denoms, steps=5, warmup=3):
    """One of the other workloads: `steps` timed epochs in its own precision; epochs/s, aggregation and product figures."""
    wl = synth.CONFIGS[key]
    prec = mg.PRECISIONS[wl.precision]
    ctx = mg.ctx_create(local_rank)
    try:
        g, tr, X0, y, m, Ws, bs = make_trainer(mg, ctx, wl, dev, prec)
        sync = lambda: torch.cuda.synchronize()
        _, ms_total, phase_ms, launches, paths = timed_epochs(tr, mg, ctx, steps, warmup, 0, sync)
        agg, gemm, _, plan = phase_figures(mg, wl, tr, g.n, g.nnz, steps, phase_ms, peaks, denoms, wl.precision)
        out = dict(workload=wl.name, n=g.n, nnz=g.nnz, dims=list(wl.dims), dtype={"fp32": "f32"}.get(wl.precision, wl.precision),
                   steps=steps, warmup=warmup, ms_per_step=round(ms_total / steps, 3), value=round(steps / (ms_total / 1e3), 4), unit=UNIT,
                   orders=["agg-first" if o == mg.ORDER_AGG_FIRST else "upd-first" for o in tr.orders],
                   aggregation=agg, gemm=gemm, gemm_paths=paths, gpu_launches=launches,
                   phase_ms_per_epoch={k: round(v / steps, 3) for k, v in phase_ms.items()}, loss=round(tr.loss.item(), 6),
                   l2="inputs larger than L2" if 4 * g.n * wl.dims[0] > L2_BYTES else "inputs fit L2 (no flush)",
                   device_status=mg.ctx_poll_status(ctx, raise_on_error=False))
        g.close()
        return out
    except Exception as e:   # report, do not hide
        return dict(workload=wl.name, error=str(e)[:200])
    finally:
        ctx.close()
        torch.cuda.empty_cache()


def gemm_c4_leg(mg, dev, local_rank, peaks, iters=5):
    """The wide dense products of workload C4 alone (1M x 1024 x 1024, bf16 operands, fp32 accumulate and
    results): forward Z W, input gradient dP W^T, weight gradient Z^T dP.  Kernel time = the product's own
    launches (per-launch events), apart from the on-the-fly bf16 conversion of the fp32 operands that a layer
    avoids by having its producers write bf16 copies."""
    ctx = mg.ctx_create(local_rank)
    out = {}
    try:
        M, N, K = 1_000_000, 1024, 1024
        A = synth.uniform_tensor((M, K), 1, device=dev)
        W = synth.uniform_tensor((K, N), 2, device=dev)
        G = synth.uniform_tensor((M, N), 3, device=dev)
        Cm = torch.zeros((M, N), device=dev)
        dW = torch.zeros((K, N), device=dev)
        forms = (("forward_ZW", lambda: mg.gemm(ctx, mg.PREC_BF16, False, False, M, N, K, A, W, Cm)),
                 ("input_grad_dPWt", lambda: mg.gemm(ctx, mg.PREC_BF16, False, True, M, K, N, G, W, Cm)),
                 ("weight_grad_ZtdP", lambda: mg.gemm(ctx, mg.PREC_BF16, True, False, K, N, M, A, G, dW)))
        for name, fn in forms:
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            mg.ctx_profile_read(ctx)
            mg.ctx_profile_enable(ctx, True)
            for _ in range(iters):
                fn()
            phase_ms, _, _ = mg.ctx_profile_read(ctx)
            mg.ctx_profile_enable(ctx, False)
            kern = phase_ms["gemm"] / iters
            tfl = 2 * M * N * K / kern / 1e9
            out[name] = dict(kernel_ms=round(kern, 4), tflops=round(tfl, 1), frac_of_bf16_burst=round(tfl / peaks["bf16_tflops"], 4),
                             frac_of_bf16_sustained=round(tfl / peaks["bf16_tflops_sustained"], 4),
                             convert_ms=round(phase_ms["elementwise"] / iters, 4))
        out["paths"] = mg.ctx_gemm_paths(ctx)
        out["shape"] = "1,000,000 x 1024 x 1024, bf16 operands, fp32 accumulate"
        out["device_status"] = mg.ctx_poll_status(ctx, raise_on_error=False)
    except Exception as e:
        out["error"] = str(e)[:200]
    finally:
        ctx.close()
        torch.cuda.empty_cache()
    return out


def run_ours(args, rank, world, local_rank):
    from paper_2501_01951_b200 import binding as mg
    wl = synth.CONFIGS[args.workload]
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    prec_name = args.precision or wl.precision
    prec = mg.PRECISIONS[prec_name]

    t0 = time.time()
    ctx = mg.ctx_create(local_rank)
    denoms = measure_denominators(mg, ctx, dev) if (rank == 0 and not args.no_extras) else None
    g, tr, X0, y, m, Ws, bs = make_trainer(mg, ctx, wl, dev, prec, args)
    n, nnz = g.n, g.nnz
    setup_s = time.time() - t0

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    clocks = ClockSampler(local_rank)
    t, ms_total, phase_ms, launches, paths = timed_epochs(tr, mg, ctx, args.steps, args.warmup, 0, barrier)
    clk = clocks.stop()
    status = mg.ctx_poll_status(ctx, raise_on_error=False)
    loss_val = tr.loss.item()
    n_train = int(m.sum().item())

    ms_total, value = replicas_throughput(ms_total, args.steps, world, dev)
    ms_per_step = ms_total / args.steps

    # Opt-in variants, reported beside the headline (never instead of it).  Same loss and gradients;
    # train_rows_only gives up the logits of the non-train nodes, cache_first_aggregation keeps
    # A_hat X^(0) across epochs (the paper recomputes it every iteration).
    opt_in = {}
    can_rows = tr.row_sparse_levels >= 1 and n_train > 0 and not args.train_rows_only
    can_cache = tr.orders[0] == mg.ORDER_AGG_FIRST and not args.cache_first_aggregation
    variants = []
    if can_rows:
        variants.append(("train_rows_only", True, False))
    if can_cache:
        variants.append(("cache_first_aggregation", False, True))
    if can_rows and can_cache:
        variants.append(("both", True, True))
    if args.no_extras:
        variants = []
    for name, rows_only, cache in variants:
        tr.configure(train_rows_only=rows_only or args.train_rows_only, cache_first_aggregation=cache or args.cache_first_aggregation)
        for _ in range(2):
            t += 1
            tr.epoch(t)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            t += 1
            tr.epoch(t)
        e1.record()
        barrier()
        ms_s, value_s = replicas_throughput(e0.elapsed_time(e1), args.steps, world, dev)
        opt_in[name] = dict(value=round(value_s, 4), unit=UNIT, ms_per_step=round(ms_s / args.steps, 3), loss=round(tr.loss.item(), 6))
    if variants:
        tr.configure(train_rows_only=args.train_rows_only, cache_first_aggregation=args.cache_first_aggregation)

    # roofline of the aggregation kernels over the timed steps
    agg, gemm, bwd_rows, plan = phase_figures(mg, wl, tr, n, nnz, args.steps, phase_ms, peaks, denoms, prec_name,
                                              args.train_rows_only, args.cache_first_aggregation)
    w_head = plan[0][0]
    roofline = dict(bound="hbm", kernel="spmm (aggregation)", achieved=agg["alg_gbs"], peak=peaks["hbm_gbs"],
                    unit="GB/s", frac=agg["frac_of_hbm_peak"], peak_source=peaks["source"],
                    traffic=None, calls=agg["calls"], avg_call_ms=agg["avg_call_ms"],
                    alg_bytes_per_call=agg["alg_bytes_per_call"], gather_gbs=agg["gather_gbs"])
    roofline["traffic_note"] = TRAFFIC_NOTE
    roofline["small_case_capture"] = SMALL_CASE_CAPTURE
    if rank == 0 and not args.no_extras and g.symmetric:
        floor, k_rows, hit = ideal_cache_floor(mg.graph_degrees(g).to(dev), n, nnz, w_head)
        t_floor = floor / (peaks["hbm_gbs"] * 1e9) * 1e3
        roofline["ideal_static_cache"] = dict(bytes_per_call=floor, cached_rows=k_rows, gathers_served_from_cache=round(hit, 4),
                                              ms_at_hbm_peak=round(t_floor, 3), ratio_to_algorithmic=round(floor / agg["alg_bytes_per_call"], 3),
                                              frac_bound=round(agg["alg_bytes_per_call"] / floor, 4),
                                              note="DRAM bytes if the L2 held the most-gathered input rows and every other gather missed; "
                                                   "frac_bound = algorithmic bytes / these bytes = the roofline fraction a kernel moving them at the full HBM rate would show")
    breakdown = {k: round(v / args.steps, 3) for k, v in phase_ms.items()}

    out = dict(metric=METRIC, value=round(value, 4), unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
               ms_per_step=round(ms_per_step, 3), higher_is_better=True, scaling="weak", vs_baseline=None,
               dtype={"fp32": "f32"}.get(prec_name, prec_name), data="synthetic",
               config=dict(workload=wl.name, n=n, nnz=nnz, dims=list(wl.dims), train_nodes=n_train,
                           orders=["agg-first" if o == mg.ORDER_AGG_FIRST else "upd-first" for o in tr.orders],
                           chunks=args.chunks, row_sparse_levels=tr.row_sparse_levels, backward_rows=[r if r is not None else n for r in bwd_rows], train_rows_only=bool(args.train_rows_only), cache_first_aggregation=bool(args.cache_first_aggregation), row_plans=not args.no_row_plans, l2="inputs larger than L2" if 4 * n * wl.dims[0] > L2_BYTES else "inputs fit L2 (no flush)",
                           parallelism=f"replicas x{world}" if world > 1 else "single GPU", setup_s=round(setup_s, 1)),
               clocks=clk, gpu_launches=launches, gemm_paths=paths,
               roofline=roofline, gemm=gemm, phase_ms_per_epoch=breakdown, loss=round(loss_val, 6), device_status=status)
    if denoms:
        out["denominators"] = denoms
    if opt_in:
        opt_in["note"] = ("opt-in variants, not the headline: train_rows_only = last layer forward, loss and gradient on train rows only; "
                          "cache_first_aggregation = A_hat X^(0) kept across epochs")
        out["opt_in"] = opt_in

    if rank == 0:
        # free the trainer and the device copy of the features before the host-buffer run allocates its arena
        Xh = torch.empty((n, wl.dims[0]), dtype=torch.float32, pin_memory=True)
        Xh.copy_(X0[:, : wl.dims[0]])
        tr.X[0] = None
        del tr, X0
        torch.cuda.empty_cache()
        out["e2e"] = run_e2e(args, mg, ctx, g, wl, prec, Xh, y, m, Ws, bs)
        del Xh
        g.close()
        ctx.close()
        del y, m, Ws, bs
        torch.cuda.empty_cache()
        if world == 1 and not args.no_extras:
            out["workloads"] = {k: workload_leg(mg, k, dev, local_rank, peaks, denoms) for k in synth.CONFIGS if k != args.workload}
            out["gemm_c4"] = gemm_c4_leg(mg, dev, local_rank, peaks)
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(wl, args.cpu_seconds)
        print(json.dumps(out), flush=True)


def run_e2e(args, mg, ctx, g, wl, prec, Xh, y, m, Ws, bs):
    """The same iteration through mixgcn_train_step_host: pinned host inputs, copies inside the timed region.
    The headline variant returns predictions for every node (so the last layer and the loss cover every node,
    as the device-resident headline does) and announces each step's features to the step before it, which
    overlaps their copy with its own backward pass; `plain` is the same without the announcement and
    `train_rows_only` the call without predictions (last layer and loss on the train rows only)."""
    n, d0 = g.n, wl.dims[0]
    try:
        yh, mh = y.cpu().pin_memory(), m.cpu().pin_memory()
        pin = lambda lst: [x.detach().cpu().clone().pin_memory() for x in lst]
        params = sum(x.numel() for x in Ws + bs)
        steps = max(1, min(args.steps, args.e2e_steps))
        predh = torch.empty(n, dtype=torch.int32).pin_memory()

        def run(with_pred, announce):
            W, b = pin(Ws), pin(bs)
            mW, vW = [torch.zeros_like(x).pin_memory() for x in W], [torch.zeros_like(x).pin_memory() for x in W]
            mb, vb = [torch.zeros_like(x).pin_memory() for x in b], [torch.zeros_like(x).pin_memory() for x in b]
            pr = predh if with_pred else None
            if announce:
                mg.train_step_host_prefetch(ctx, Xh)
            mg.train_step_host(ctx, g, wl.dims, prec, Xh, yh, mh, W, b, mW, vW, mb, vb, 1, pred=pr)       # warm-up, allocates the arena
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for i in range(steps):
                if announce:
                    mg.train_step_host_prefetch(ctx, Xh)      # the next step's features (the same pinned buffer here)
                loss = mg.train_step_host(ctx, g, wl.dims, prec, Xh, yh, mh, W, b, mW, vW, mb, vb, 2 + i, pred=pr)
            dt = time.perf_counter() - t0
            torch.cuda.synchronize()        # the copy announced by the last step is outside the timed steps' results
            return dt, loss

        dt, loss = run(True, True)
        dt_plain, _ = run(True, False)
        dt_rows, loss_rows = run(False, False)
        h2d = 4 * n * d0 + 4 * n + n + 3 * 4 * params
        d2h = 4 + 3 * 4 * params + 4 * n
        return dict(value=round(steps / dt, 4), unit=UNIT, steps=steps, ms_per_step=round(dt / steps * 1e3, 3),
                    h2d_bytes_per_step=int(h2d), d2h_bytes_per_step=int(d2h), loss=round(loss, 6),
                    api="mixgcn_train_step_host with pred (predictions for every node returned) + mixgcn_train_step_host_prefetch; pinned host buffers",
                    pred_returned=True, feature_copy_overlapped=True,
                    plain=dict(value=round(steps / dt_plain, 4), ms_per_step=round(dt_plain / steps * 1e3, 3),
                               note="same call without announcing the next step's features: copy, then compute"),
                    train_rows_only=dict(value=round(steps / dt_rows, 4), ms_per_step=round(dt_rows / steps * 1e3, 3), loss=round(loss_rows, 6),
                                         d2h_bytes_per_step=int(d2h - 4 * n),
                                         note="called without pred: last layer and loss on the train rows only (not the headline's work)"))
    except Exception as e:  # report, do not hide
        return dict(value=None, unit=UNIT, error=str(e)[:200], h2d_bytes_per_step=None, d2h_bytes_per_step=None)


# ------------------------------------------------------------------------------------ CPU oracle

def oracle_sample_problem(wl, target_seconds):
    """A smaller R-MAT graph with the workload's mean degree, widths, classes and mask rate, sized so
    that one oracle epoch takes roughly `target_seconds` on this host."""
    from oracle import gcn_oracle as orc
    flops_per_node = 0
    mean_deg = 2 * wl.undirected_edges / wl.n + 1
    for l in range(len(wl.dims) - 1):
        flops_per_node += 2 * mean_deg * wl.dims[l] * (1 if l == 0 else 2) + 2 * wl.dims[l] * wl.dims[l + 1] * (2 if l == 0 else 3)
    rate = 0.6e9 * orc.n_threads()                     # naive fp64 loops: ~0.6 GFLOP/s per thread
    n_s = int(min(wl.n, max(1024, target_seconds * rate / flops_per_node)))
    return n_s, max(1, int(wl.undirected_edges * (n_s / wl.n)))


def oracle_epoch_seconds(wl, n_s, e_s, repeats=1):
    from oracle import gcn_oracle as orc
    s, d = synth.rmat_graph(n_s, e_s, wl.seed("graph"))
    X = synth.normal_features(n_s, wl.dims[0], wl.seed("features")).numpy()
    y = synth.uniform_labels(n_s, wl.classes, wl.seed("labels")).numpy()
    m = synth.bernoulli_mask(n_s, max(wl.mask_p, 4.0 / n_s), wl.seed("mask")).numpy()
    m[0] = 1
    Ws, bs = synth.make_weights(wl)
    Ws, bs = [w.numpy() for w in Ws], [b.numpy() for b in bs]
    go = orc.graph_build(n_s, s.numpy(), d.numpy())
    best = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.train_epoch(go, X, Ws, bs, y, m, None, 1)
        best = min(best, time.perf_counter() - t0)
    return best, go.nnz


def cpu_baseline(wl, target_seconds):
    from oracle import gcn_oracle as orc
    orc.build()
    n_s, e_s = oracle_sample_problem(wl, target_seconds)
    sec, nnz_s = oracle_epoch_seconds(wl, n_s, e_s)
    frac = n_s / wl.n
    return dict(value=round(frac / sec, 6), unit=UNIT, cores=orc.n_threads(), kind="oracle",
                sample=f"one oracle epoch on an R-MAT sample with {n_s} of {wl.n} nodes ({nnz_s} stored entries, same mean "
                       f"degree, widths {list(wl.dims)}) took {sec:.2f} s; epochs/s scaled by the node fraction {frac:.3g}",
                sample_seconds=round(sec, 3))


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle as it stands, each step one epoch on a bounded sample."""
    if rank != 0:
        return
    from oracle import gcn_oracle as orc
    orc.build()
    wl = synth.CONFIGS[args.workload]
    n_s, e_s = oracle_sample_problem(wl, args.cpu_seconds / max(1, args.steps + args.warmup) * 2)
    for _ in range(args.warmup):
        oracle_epoch_seconds(wl, n_s, e_s)
    t0 = time.perf_counter()
    secs = [oracle_epoch_seconds(wl, n_s, e_s)[0] for _ in range(args.steps)]
    wall = time.perf_counter() - t0
    sec = sum(secs) / len(secs)
    frac = n_s / wl.n
    value = frac / sec
    sample = (f"each step = one oracle epoch on an R-MAT sample with {n_s} of {wl.n} nodes (same mean degree and widths); "
              f"epochs/s scaled by the node fraction {frac:.3g}")
    out = dict(impl="reference", metric=METRIC, value=round(value, 6), unit=UNIT, n_gpus=world, steps=args.steps,
               warmup=args.warmup, ms_per_step=round(sec / frac * 1e3, 1), higher_is_better=True, scaling="weak",
               vs_baseline=None, dtype="f64", data="synthetic",
               config=dict(workload=wl.name, n=wl.n, dims=list(wl.dims), sample_nodes=n_s, wall_s=round(wall, 1)),
               cpu_baseline=dict(value=round(value, 6), unit=UNIT, cores=orc.n_threads(), kind="oracle", sample=sample),
               e2e=dict(value=round(value, 6), unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
               gpu_launches=0)
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=os.environ.get("MIXGCN_WORKLOAD", "C5"), choices=list(synth.CONFIGS))
    ap.add_argument("--precision", default=None, choices=["fp32", "tf32", "bf16"])
    ap.add_argument("--chunks", type=int, default=0)
    ap.add_argument("--train-rows-only", action="store_true",
                    help="opt-in shortcut: the last layer's output, the loss and its gradient on train rows only "
                         "(same loss and gradients; no predictions for the other nodes)")
    ap.add_argument("--cache-first-aggregation", action="store_true",
                    help="opt-in: keep A_hat X^(0) of the first layer across epochs instead of recomputing it")
    ap.add_argument("--no-row-plans", action="store_true",
                    help="row-sparse backward by testing the row masks inside the aggregation kernel every iteration "
                         "instead of on restricted matrices built once")
    ap.add_argument("--row-sparse", default="auto", help="layers (from the top) whose backward gets a row mask: auto, 0, 1, 2, ...")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=20.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="headline only: no opt-in variants, no other workloads, no denominators (for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, rank, world, local_rank)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
