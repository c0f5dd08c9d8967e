"""Single-kernel runs through the C-ABI, sized by flags: for CUDA-event timing of one operation
and as a small, self-ending target for profiler captures.

    python -m paper_2501_01951_b200.microbench --op spmm --n 4000000 --edges 32000000 --w 128
    python -m paper_2501_01951_b200.microbench --op gemm --M 1000000 --N 1024 --K 1024 --precision tf32
    python -m paper_2501_01951_b200.microbench --op loss --n 4000000 --w 172 --mask-p 0.01 --loss-rows 0
    python -m paper_2501_01951_b200.microbench --op model --model sage --n 2449029 --edges 61859140 --dims 100,128,128,47 --precision tf32

Prints one JSON line with the median time and the derived algorithmic GB/s or TFLOP/s.
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import binding as mg
from . import synth


def _time(fn, iters, warmup):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    return statistics.median(ts), min(ts)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", required=True, choices=["spmm", "gemm", "loss", "model"])
    ap.add_argument("--n", type=int, default=1 << 20)
    ap.add_argument("--edges", type=int, default=8 << 20, help="distinct undirected edges of the R-MAT graph")
    ap.add_argument("--w", type=int, default=128)
    ap.add_argument("--M", type=int, default=1 << 20)
    ap.add_argument("--N", type=int, default=256)
    ap.add_argument("--K", type=int, default=256)
    ap.add_argument("--ta", type=int, default=0)
    ap.add_argument("--tb", type=int, default=0)
    ap.add_argument("--precision", default="fp32", choices=list(mg.PRECISIONS))
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=2)
    ap.add_argument("--seed", type=int, default=1005)
    ap.add_argument("--model", default="sage", choices=["gcn", "sage", "gin"], help="model: architecture of the timed training epochs")
    ap.add_argument("--dims", default="128,128,128,64", help="model: layer widths d_0,...,d_L")
    ap.add_argument("--hidden", type=int, default=128, help="model: width of GIN's inner perceptron layer")
    ap.add_argument("--mask-p", type=float, default=0.01, help="loss / model: fraction of train rows")
    ap.add_argument("--loss-rows", type=int, default=0, choices=[0, 1, 2], help="loss: MIXGCN_OPT_LOSS_TRAIN_ROWS_ONLY value")
    ap.add_argument("--slice", type=int, default=0, help="feature-column slice width of the aggregation (0 = default)")
    ap.add_argument("--sampled", type=float, default=0.0, help="spmm: also time the sampled aggregation (Eq. 4) with this fraction of outputs kept")
    args = ap.parse_args()

    dev = torch.device("cuda", 0)
    ctx = mg.ctx_create(0)
    if args.slice:
        mg.ctx_set_option(ctx, mg.OPT_SPMM_SLICE_COLS, args.slice)
    out = dict(op=args.op)
    if args.op == "spmm":
        s, d = synth.rmat_graph(args.n, args.edges, args.seed, device=dev)
        g = mg.graph_create(ctx, args.n, s, d)
        del s, d
        ld = (args.w + 3) // 4 * 4
        Y = synth.normal_features(args.n, args.w, 7, device=dev, ld=ld)
        Z = torch.zeros_like(Y)
        med, best = _time(lambda: mg.spmm(ctx, g, Y, Z, args.w), args.iters, args.warmup)
        alg = 8 * (g.n + 1) + 8 * g.nnz + 8 * g.n * args.w
        out.update(n=g.n, nnz=g.nnz, w=args.w, max_deg=g.max_deg, ms_median=round(med, 4), ms_best=round(best, 4),
                   alg_bytes=alg, alg_gbs=round(alg / med / 1e6, 1), gather_gbs=round(4 * g.nnz * args.w / med / 1e6, 1))
        if args.sampled:
            # the sampled aggregation of Eq. 4 on the same graph: a random element mask, and a mask that
            # drops the same fraction as whole 16-byte groups
            bits = torch.zeros((g.n, (args.w + 31) // 32), dtype=torch.int32, device=dev)
            for name, group in (("element_mask", 1), ("group_mask", 4)):
                cols = (args.w + group - 1) // group
                m8 = torch.empty((g.n, args.w), dtype=torch.uint8, device=dev)
                gen = torch.Generator(device=dev).manual_seed(11)
                for r0 in range(0, g.n, 1 << 21):                       # a seeded mask, drawn in row blocks
                    r1 = min(g.n, r0 + (1 << 21))
                    keep = (torch.rand((r1 - r0, cols), generator=gen, device=dev) < args.sampled).to(torch.uint8)
                    m8[r0:r1] = keep.repeat_interleave(group, dim=1)[:, : args.w]
                mg.mask_pack(ctx, args.w, bits, bytes_mask=m8)
                del keep, m8
                med_s, best_s = _time(lambda: mg.spmm_sampled(ctx, g, Y, Z, args.w, bits), args.iters, args.warmup)
                out["sampled_" + name] = dict(keep_fraction=args.sampled, ms_median=round(med_s, 4), ms_best=round(best_s, 4))
    elif args.op == "model":
        from .sage_gin import GinTrainer, SageTrainer
        from .train import GcnTrainer
        dims = tuple(int(x) for x in args.dims.split(","))
        L = len(dims) - 1
        s, d = synth.rmat_graph(args.n, args.edges, args.seed, device=dev)
        norm = {"gcn": mg.GRAPH_ADD_SELF_LOOPS, "sage": mg.GRAPH_NORM_ROW, "gin": mg.GRAPH_NORM_NONE}[args.model]
        g = mg.graph_create(ctx, args.n, s, d, mg.GRAPH_SYMMETRISE | norm)
        del s, d
        torch.cuda.empty_cache()
        prec = mg.PRECISIONS[args.precision]
        X0 = synth.normal_features(args.n, dims[0], 7, device=dev, ld=(dims[0] + 3) // 4 * 4)
        y = synth.uniform_labels(args.n, dims[-1], 8, device=dev)
        m = synth.bernoulli_mask(args.n, args.mask_p, 9, device=dev)
        W = lambda a, b, k, scale=1.0: synth.glorot_uniform(a, b, k, device=dev) * scale
        zb = lambda k: torch.zeros(k, device=dev)
        if args.model == "gcn":
            tr = GcnTrainer(ctx, g, dims, prec)
            tr.set_params([W(dims[i], dims[i + 1], 20 + i) for i in range(L)], [zb(dims[i + 1]) for i in range(L)])
            tr.set_inputs(X0, y, m)
        elif args.model == "sage":
            tr = SageTrainer(ctx, g, dims, prec)
            tr.set_params([W(dims[i], dims[i + 1], 20 + i) for i in range(L)], [W(dims[i], dims[i + 1], 40 + i) for i in range(L)],
                          [zb(dims[i + 1]) for i in range(L)])
            tr.set_inputs(X0, y, m)
        else:
            tr = GinTrainer(ctx, g, dims, args.hidden, prec)
            tr.set_params([W(dims[i], args.hidden, 20 + i, 0.05) for i in range(L)], [zb(args.hidden) for i in range(L)],
                          [W(args.hidden, dims[i + 1], 40 + i) for i in range(L)], [zb(dims[i + 1]) for i in range(L)])
            tr.set_inputs(X0, y, m)
        step = [0]

        def one():
            step[0] += 1
            tr.epoch(step[0])
        med, best = _time(one, args.iters, args.warmup)
        mg.ctx_profile_read(ctx)
        mg.ctx_profile_enable(ctx, True)
        for _ in range(args.iters):
            one()
        phase_ms, _, _ = mg.ctx_profile_read(ctx)
        mg.ctx_profile_enable(ctx, False)
        out.update(phase_ms_per_epoch={k: round(v / args.iters, 3) for k, v in phase_ms.items()}, paths=mg.ctx_gemm_paths(ctx))
        out.update(model=args.model, n=g.n, nnz=g.nnz, dims=list(dims), precision=args.precision, loss=round(tr.loss.item(), 6),
                   ms_median=round(med, 4), ms_best=round(best, 4), epochs_per_s=round(1e3 / med, 3),
                   device_status=mg.ctx_poll_status(ctx, raise_on_error=False))
    elif args.op == "loss":
        n, C = args.n, args.w
        ld = (C + 3) // 4 * 4
        P = synth.normal_features(n, C, 7, device=dev, ld=ld)
        G = torch.empty_like(P)
        y = synth.uniform_labels(n, C, 8, device=dev)
        m = synth.bernoulli_mask(n, args.mask_p, 9, device=dev)
        loss = torch.zeros(1, device=dev)
        pred = torch.zeros(n, dtype=torch.int32, device=dev)
        nc = torch.zeros(1, dtype=torch.int64, device=dev)
        mg.ctx_set_option(ctx, mg.OPT_LOSS_TRAIN_ROWS_ONLY, args.loss_rows)
        med, best = _time(lambda: mg.loss_softmax_xent(ctx, P, y, m, loss, dlogits=G, pred=pred, n_correct=nc, C_=C),
                          args.iters, args.warmup)
        n_train = int(m.sum().item())
        rows_read = n_train if args.loss_rows == 1 else n
        rows_written = n if args.loss_rows == 0 else n_train
        alg = 4 * C * (rows_read + rows_written) + 9 * n
        out.update(n=n, C=C, train_rows=n_train, loss_rows_option=args.loss_rows, loss=round(loss.item(), 6),
                   ms_median=round(med, 4), ms_best=round(best, 4), alg_bytes=alg, alg_gbs=round(alg / med / 1e6, 1))
    else:
        M, N, K = args.M, args.N, args.K
        r4 = lambda x: (x + 3) // 4 * 4
        A = synth.uniform_tensor((K, r4(M)) if args.ta else (M, r4(K)), 1, device=dev)
        B = synth.uniform_tensor((N, r4(K)) if args.tb else (K, r4(N)), 2, device=dev)
        Cm = torch.zeros((M, r4(N)), device=dev)
        prec = mg.PRECISIONS[args.precision]
        med, best = _time(lambda: mg.gemm(ctx, prec, bool(args.ta), bool(args.tb), M, N, K, A, B, Cm), args.iters, args.warmup)
        # the product's own kernels (phase "gemm"), apart from the on-the-fly bf16 conversion of fp32
        # operands (phase "elementwise") that a layer avoids by having its producers write bf16 copies
        mg.ctx_profile_read(ctx)
        mg.ctx_profile_enable(ctx, True)
        for _ in range(args.iters):
            mg.gemm(ctx, prec, bool(args.ta), bool(args.tb), M, N, K, A, B, Cm)
        phase_ms, _, _ = mg.ctx_profile_read(ctx)
        mg.ctx_profile_enable(ctx, False)
        kern = phase_ms["gemm"] / args.iters
        out.update(M=M, N=N, K=K, ta=args.ta, tb=args.tb, precision=args.precision, ms_median=round(med, 4),
                   ms_best=round(best, 4), tflops=round(2 * M * N * K / med / 1e9, 2),
                   min_gbs=round(4 * (M * K + K * N + M * N) / med / 1e6, 1),
                   kernel_ms=round(kern, 4), kernel_tflops=round(2 * M * N * K / kern / 1e9, 2) if kern > 0 else None,
                   convert_ms=round(phase_ms["elementwise"] / args.iters, 4), paths=mg.ctx_gemm_paths(ctx),
                   device_status=mg.ctx_poll_status(ctx, raise_on_error=False))
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
