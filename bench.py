#!/usr/bin/env python
"""Benchmark of full-graph GCN training epochs on seeded synthetic graphs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C1..C5] [--impl ours|reference]

One step = one training epoch (all layers forward, loss, all layers backward, Adam) over the
whole graph.  Prints ONE JSON line.  `value` is epochs/s with every input resident in HBM;
`e2e` is the same iteration through the host-buffer entry point (host->device copies of the
features, labels, mask, parameters and moments and device->host copies of the results inside
the timed region); `roofline` covers the aggregation kernels (the dominant kernel), with the
per-call durations measured by CUDA events on the launching stream during the timed steps;
`cpu_baseline` is the CPU oracle timed on a bounded sample of the same workload.

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

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of ONE aggregation call at the workload's
# size and width, from a single-pass ncu capture of one call at full size, summarised under profiles/
# (every aggregation of C5 has width 128 and the same graph, so the figure holds for each of its calls).
NCU_SPMM_CALL_DRAM_BYTES = {"C5": 131232026368}

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


def run_ours(args, rank, world, local_rank):
    from paper_2501_01951_b200 import binding as mg
    from paper_2501_01951_b200.train import GcnTrainer, round4
    wl = synth.CONFIGS[args.workload]
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    prec = mg.PRECISIONS[args.precision or wl.precision]

    t0 = time.time()
    ctx = mg.ctx_create(local_rank)
    src, dst = build_problem(wl, dev)
    g = mg.graph_create(ctx, wl.n, src, dst)
    del src, dst
    torch.cuda.empty_cache()
    n, nnz = g.n, g.nnz
    tr = GcnTrainer(ctx, g, wl.dims, prec, n_chunks=args.chunks,
                    row_sparse=args.row_sparse if args.row_sparse == "auto" else int(args.row_sparse),
                    train_rows_only=args.train_rows_only, row_plans=not args.no_row_plans,
                    cache_first_aggregation=args.cache_first_aggregation)
    X0 = synth.normal_features(n, wl.dims[0], wl.seed("features"), device=dev, ld=round4(wl.dims[0]))
    y = synth.uniform_labels(n, wl.classes, wl.seed("labels"), device=dev)
    m = synth.bernoulli_mask(n, wl.mask_p, wl.seed("mask"), device=dev)
    Ws, bs = synth.make_weights(wl, device=dev)
    tr.set_params(Ws, bs)
    tr.set_inputs(X0, y, m)
    mg.ctx_reserve(ctx, 64 << 20)
    torch.cuda.synchronize()
    setup_s = time.time() - t0

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    t = 0
    for _ in range(args.warmup):
        t += 1
        tr.epoch(t)
    barrier()
    _, _, launches_before = mg.ctx_profile_read(ctx)
    mg.ctx_profile_enable(ctx, True)
    clocks = ClockSampler(local_rank)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        t += 1
        tr.epoch(t)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    clk = clocks.stop()
    phase_ms, phase_launches, launches_after = mg.ctx_profile_read(ctx)
    mg.ctx_profile_enable(ctx, False)
    status = mg.ctx_poll_status(ctx, raise_on_error=False)
    loss_val = tr.loss.item()
    n_train = int(m.sum().item())

    ms_total, value = replicas_throughput(ms_total, args.steps, world, dev)
    ms_per_step = ms_total / args.steps

    # rows the dense products of each layer's backward ran on (compacted rows where layer_bwd took that path)
    bwd_rows = []
    for l, d in enumerate(tr.descs):
        cnt = int(d.gout_row_count)
        rows_flag = bool(d.flags & mg.LAYER_OUT_ROWS_ONLY)
        compacted = bool(d.gout_row_mask) and cnt > 0 and tr.orders[l] == mg.ORDER_AGG_FIRST and (4 * cnt < n or rows_flag or bool(d.gout_plan))
        bwd_rows.append(cnt if compacted else None)

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
    plan = spmm_plan(wl, tr.orders, tr.row_sparse_levels, args.train_rows_only)
    if args.cache_first_aggregation and tr.orders[0] == mg.ORDER_AGG_FIRST:
        plan[0] = (plan[0][0], plan[0][1] - 1)
    spmm_calls = sum(k for _, k in plan) * args.steps
    alg_bytes = sum(spmm_alg_bytes(n, nnz, w) * k for w, k in plan) * args.steps
    spmm_ms = phase_ms["spmm"]
    achieved = alg_bytes / (spmm_ms / 1e3) / 1e9 if spmm_ms > 0 else 0.0
    roofline = dict(bound="hbm", kernel="spmm (aggregation)", achieved=round(achieved, 1), peak=peaks["hbm_gbs"],
                    unit="GB/s", frac=round(achieved / peaks["hbm_gbs"], 4), peak_source=peaks["source"],
                    traffic=NCU_SPMM_CALL_DRAM_BYTES.get(args.workload), calls=spmm_calls, avg_call_ms=round(spmm_ms / max(spmm_calls, 1), 4),
                    alg_bytes_per_call=int(alg_bytes / max(spmm_calls, 1)),
                    gather_gbs=round(sum(4 * nnz * w * k for w, k in plan) * args.steps / (spmm_ms / 1e3) / 1e9, 1) if spmm_ms > 0 else 0.0)
    if roofline["traffic"] and spmm_ms > 0:
        # real DRAM throughput of the call: captured bytes over the call's measured duration
        dram_gbs = roofline["traffic"] / (spmm_ms / max(spmm_calls, 1) / 1e3) / 1e9
        roofline.update(dram_gbs=round(dram_gbs, 1), dram_frac=round(dram_gbs / peaks["hbm_gbs"], 4))
    fwd_rows_last = n_train if (args.train_rows_only and tr.orders[-1] == mg.ORDER_AGG_FIRST) else None
    flops = gemm_flops(n, wl.dims, tr.orders, bwd_rows, fwd_rows_last) * args.steps
    gemm_ms = phase_ms["gemm"]
    # The dense products run TF32 on the tensor cores: their peak is the measured bf16 peak times the
    # nominal tf32/bf16 ratio (1.1 / 2.25).  Their minimum HBM bytes: every n x d operand and result once.
    tf32_peak = peaks["bf16_tflops"] * 1.1 / 2.25
    gbytes = gemm_min_bytes(n, wl.dims, bwd_rows, fwd_rows_last) * args.steps
    tfl = flops / (gemm_ms / 1e3) / 1e12 if gemm_ms > 0 else 0.0
    gemm = dict(tflops=round(tfl, 2), tf32_peak_tflops=round(tf32_peak, 1), frac_of_tf32_peak=round(tfl / tf32_peak, 4),
                min_hbm_gbs=round(gbytes / (gemm_ms / 1e3) / 1e9, 1) if gemm_ms > 0 else 0.0,
                frac_of_hbm_peak=round(gbytes / (gemm_ms / 1e3) / 1e9 / peaks["hbm_gbs"], 4) if gemm_ms > 0 else 0.0,
                ms_per_epoch=round(gemm_ms / args.steps, 3))
    breakdown = {k: round(v / args.steps, 3) for k, v in phase_ms.items()}

    out = dict(metric=METRIC, value=round(value, 4), unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
               ms_per_step=round(ms_per_step, 3), higher_is_better=True, scaling="weak", vs_baseline=None,
               dtype={mg.PREC_FP32: "f32", mg.PREC_TF32: "tf32", mg.PREC_BF16: "bf16"}[prec], data="synthetic",
               config=dict(workload=wl.name, n=n, nnz=nnz, dims=list(wl.dims), train_nodes=n_train,
                           orders=["agg-first" if o == mg.ORDER_AGG_FIRST else "upd-first" for o in tr.orders],
                           chunks=args.chunks, row_sparse_levels=tr.row_sparse_levels, backward_rows=[r if r is not None else n for r in bwd_rows], train_rows_only=bool(args.train_rows_only), cache_first_aggregation=bool(args.cache_first_aggregation), row_plans=not args.no_row_plans, l2="inputs larger than L2" if 4 * n * wl.dims[0] > 126e6 else "inputs fit L2 (no flush)",
                           parallelism=f"replicas x{world}" if world > 1 else "single GPU", setup_s=round(setup_s, 1)),
               clocks=clk, gpu_launches=int(launches_after - launches_before),
               roofline=roofline, gemm=gemm, phase_ms_per_epoch=breakdown, loss=round(loss_val, 6), device_status=status)
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
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(wl, args.cpu_seconds)
        print(json.dumps(out), flush=True)


def run_e2e(args, mg, ctx, g, wl, prec, Xh, y, m, Ws, bs):
    """The same iteration through mixgcn_train_step_host: pinned host inputs, copies inside the timed region."""
    n, d0 = g.n, wl.dims[0]
    try:
        yh, mh = y.cpu().pin_memory(), m.cpu().pin_memory()
        pin = lambda lst: [x.detach().cpu().clone().pin_memory() for x in lst]
        W, b = pin(Ws), pin(bs)
        mW, vW = [torch.zeros_like(x).pin_memory() for x in W], [torch.zeros_like(x).pin_memory() for x in W]
        mb, vb = [torch.zeros_like(x).pin_memory() for x in b], [torch.zeros_like(x).pin_memory() for x in b]
        steps = max(1, min(args.steps, args.e2e_steps))
        mg.train_step_host(ctx, g, wl.dims, prec, Xh, yh, mh, W, b, mW, vW, mb, vb, 1)       # warm-up, allocates the arena
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(steps):
            loss = mg.train_step_host(ctx, g, wl.dims, prec, Xh, yh, mh, W, b, mW, vW, mb, vb, 2 + i)
        dt = time.perf_counter() - t0
        params = sum(x.numel() for x in W + b)
        h2d = 4 * n * d0 + 4 * n + n + 3 * 4 * params
        d2h = 4 + 3 * 4 * params
        return dict(value=round(steps / dt, 4), unit=UNIT, steps=steps, ms_per_step=round(dt / steps * 1e3, 3),
                    h2d_bytes_per_step=int(h2d), d2h_bytes_per_step=int(d2h), loss=round(loss, 6),
                    api="mixgcn_train_step_host (pinned host buffers)")
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
