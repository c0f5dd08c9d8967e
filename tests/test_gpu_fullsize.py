"""Parity at the workloads' full sizes, in the launch configuration bench.py times.

The oracle cannot run a whole epoch at these sizes in test time, so every operation is checked
teacher-forced on sampled outputs the oracle computes one by one (the GPU's own input to that
operation is copied to the host for the sampled rows), plus properties that hold at any size
(A_hat sqrt(deg~) = sqrt(deg~)); every layer's weight and bias gradient is compared in full with the
fp64 product of the operands that layer's backward call received.  Expected values
come from the oracle or from the definition evaluated with numpy on the generator's edge list."""
import numpy as np
import pytest
import torch

from helpers import TOL_FP32, TOL_LOWP, round4
from oracle import gcn_oracle as orc
from paper_2501_01951_b200 import synth

pytestmark = pytest.mark.gpu

N_SAMPLE = 192


@pytest.fixture(scope="module")
def mg():
    from paper_2501_01951_b200 import build
    build.build()
    from paper_2501_01951_b200 import binding
    return binding


def _sample_rows(n, deg, seed):
    """Random rows plus the longest rows and a few rows with a single entry."""
    rng = np.random.default_rng(seed)
    rows = set(rng.integers(0, n, N_SAMPLE).tolist())
    order = np.argsort(deg)
    rows.update(order[-4:].tolist())
    rows.update(order[:4].tolist())
    return np.array(sorted(rows), dtype=np.int64)


def _sub_oracle_graph(n, src, dst, rows):
    """Oracle rows of A_hat for `rows`, from the definition on the generator's unique undirected
    edge list: neighbours of u are the endpoints of its edges plus u; deg~ = 1 + incident edges.
    Returns a compact oracle Graph over the nodes involved and the map compact id -> node id."""
    deg = (np.bincount(src, minlength=n) + np.bincount(dst, minlength=n) + 1).astype(np.int64)
    sel = np.isin(src, rows) | np.isin(dst, rows)
    s, d = src[sel], dst[sel]
    nodes = np.unique(np.concatenate([rows, s, d]))
    look = lambda x: np.searchsorted(nodes, x).astype(np.int64)       # nodes is sorted and contains every id looked up
    g = orc.graph_build(len(nodes), look(s), look(d))
    # the compact graph knows only the sampled rows' edges; overwrite its values with the full-graph degrees
    r_of = np.repeat(np.arange(g.n), np.diff(g.rowptr))
    g.val = 1.0 / np.sqrt(deg[nodes[r_of]].astype(np.float64) * deg[nodes[g.col]].astype(np.float64))
    return g, nodes, look(rows), deg


def _run_workload(mg, key, precision):
    from paper_2501_01951_b200.train import GcnTrainer
    wl = synth.CONFIGS[key]
    dev = torch.device("cuda", 0)
    ctx = mg.ctx_create(0)
    src, dst = synth.rmat_graph(wl.n, wl.undirected_edges, wl.seed("graph"), device=dev)
    g = mg.graph_create(ctx, wl.n, src, dst)
    src_h, dst_h = src.cpu().numpy(), dst.cpu().numpy()
    del src, dst
    torch.cuda.empty_cache()
    tr = GcnTrainer(ctx, g, wl.dims, precision)
    X0 = synth.normal_features(wl.n, wl.dims[0], wl.seed("features"), device=dev, ld=round4(wl.dims[0]))
    y = synth.uniform_labels(wl.n, wl.classes, wl.seed("labels"), device=dev)
    m = synth.bernoulli_mask(wl.n, wl.mask_p, wl.seed("mask"), device=dev)
    Ws, bs = synth.make_weights(wl, device=dev)
    bs = [synth.uniform_tensor((b.numel(),), 77 + i, -0.1, 0.1, device=dev) for i, b in enumerate(bs)]   # exercise the bias path
    tr.set_params(Ws, bs)
    tr.set_inputs(X0, y, m)
    return wl, ctx, g, tr, src_h, dst_h


def _rel(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


@pytest.mark.parametrize("key", ["C2", "C3", "C4", "C5"])
def test_full_size_workload(mg, key):
    wl = synth.CONFIGS[key]
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    dims = [round4(d) for d in wl.dims]
    cols = sum(dims) + sum(max(dims[l], dims[l + 1]) for l in range(len(dims) - 1)) + max(dims[1:-1])
    need = 4 * wl.n * cols + 36 * wl.undirected_edges
    if free < need * 1.03:
        pytest.skip(f"needs ~{need / 2**30:.0f} GiB of device memory")
    prec = mg.PRECISIONS[wl.precision]
    tol = TOL_FP32 if prec == mg.PREC_FP32 else TOL_LOWP
    wl, ctx, g, tr, src_h, dst_h = _run_workload(mg, key, prec)
    n, L = wl.n, tr.L
    assert g.symmetric and g.n == n and g.nnz == 2 * len(src_h) + n

    # ---- S0: sampled rows of the CSR, bit-exact, against the definition on the edge list
    ex = mg.graph_export(g)
    deg_gpu = ex["deg"].numpy()
    rows = _sample_rows(n, deg_gpu, 1)
    sub, nodes, crow, deg = _sub_oracle_graph(n, src_h, dst_h, rows)
    assert np.array_equal(deg_gpu, deg.astype(np.int32)) and g.max_deg == int(deg.max())
    dinv = (np.float32(1.0) / np.sqrt(deg.astype(np.float32))).astype(np.float32)
    assert ex["dinv"].numpy().tobytes() == dinv.tobytes()
    rp, col, val = ex["rowptr"].numpy(), ex["col"].numpy(), ex["val"].numpy()
    for u, cu in zip(rows, crow):
        want_cols = nodes[sub.col[sub.rowptr[cu]:sub.rowptr[cu + 1]]]
        got = col[rp[u]:rp[u + 1]]
        assert np.array_equal(got, want_cols)
        assert np.array_equal(val[rp[u]:rp[u + 1]], (dinv[u] * dinv[got]).astype(np.float32))
    del ex, rp, col, val

    def rows_of(t, idx, d):
        return t[torch.as_tensor(idx, device=t.device)][:, :d].double().cpu().numpy()

    def check_spmm(Y, Z, w, what, bound=TOL_FP32):
        Ysub = rows_of(Y, nodes, w)                                  # the operation's own input, sampled
        want = orc.aggregate_rows(sub, Ysub, crow)
        assert _rel(rows_of(Z, rows, w), want) <= bound, what

    # ---- forward, layer by layer, teacher-forced on sampled rows
    tr.forward()
    torch.cuda.synchronize()
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    for l in range(L):
        d_in, d_out = wl.dims[l], wl.dims[l + 1]
        W, b = tr.W[l].cpu().numpy(), tr.b[l].cpu().numpy()
        last = l == L - 1
        if tr.orders[l] == mg.ORDER_AGG_FIRST:
            Zl = tr.aggregation_of(l)                  # fp32, or the bf16 copy where only that is written
            check_spmm(tr.X[l], Zl, d_in, f"layer {l} aggregation", TOL_FP32 if Zl.dtype == torch.float32 else tol)
            P = orc.update(rows_of(Zl, rows, d_in), W, b)
            want = P if last else orc.activation(P)
            assert _rel(rows_of(tr.X[l + 1], rows, d_out), want) <= tol, f"layer {l} update"
        else:
            Q = orc.update(rows_of(tr.X[l], rows, d_in), W)
            assert _rel(rows_of(tr.saved[l], rows, d_out), Q) <= tol, f"layer {l} update (first)"
            P = orc.aggregate_rows(sub, rows_of(tr.saved[l], nodes, d_out), crow) + b
            want = P if last else orc.activation(P)
            assert _rel(rows_of(tr.X[l + 1], rows, d_out), want) <= TOL_FP32, f"layer {l} aggregation (second)"

    # ---- property at full scale: sqrt(deg~) is a fixed point of the aggregation (symmetric graph)
    R = torch.zeros(n, 4, device="cuda")
    R[:, 0] = torch.sqrt(torch.as_tensor(deg, device="cuda", dtype=torch.float32))
    Zr = torch.zeros_like(R)
    mg.spmm(ctx, g, R, Zr, 1)
    assert float(torch.linalg.norm(Zr[:, 0] - R[:, 0]) / torch.linalg.norm(R[:, 0])) <= TOL_FP32
    del R, Zr

    # ---- loss on all train rows (they are few enough to copy), gradient on sampled rows
    C = wl.classes
    train_idx = torch.nonzero(tr.train_mask).flatten()
    logits_train = tr.X[L][train_idx][:, :C].cpu().numpy().astype(np.float64)
    labels_train = tr.labels[train_idx].cpu().numpy()
    lo, Gt, pred_t, nc, T = orc.loss(logits_train, labels_train, np.ones(len(labels_train), np.uint8))
    logits_rows = rows_of(tr.X[L], rows, C)
    untrained = torch.nonzero(tr.train_mask == 0).flatten()[:1000]
    logits_untrained = tr.X[L][untrained].clone()
    tr.compute_loss()
    torch.cuda.synchronize()
    assert abs(tr.loss.item() - lo) <= 2e-6 * abs(lo)
    assert int(tr.n_correct.item()) == nc
    assert np.array_equal(tr.pred[train_idx].cpu().numpy(), pred_t)                       # arg-max: bit-exact
    assert np.array_equal(tr.pred[torch.as_tensor(rows, device="cuda")].cpu().numpy(), logits_rows.argmax(axis=1))
    pick = np.random.default_rng(2).integers(0, len(train_idx), 64)
    got = tr.X[L][train_idx[torch.as_tensor(pick, device="cuda")]][:, :C].cpu().numpy()
    assert _rel(got, Gt[pick]) <= TOL_FP32
    if tr.row_plans[L - 1] is None:
        assert float(tr.X[L][untrained][:, :C].abs().max()) == 0.0      # zero gradient outside the train mask
    else:
        assert torch.equal(tr.X[L][untrained], logits_untrained)          # rows the row-plan backward never reads are left alone

    # ---- backward: every layer's dW and db in full (teacher-forced); the last layer's input gradient on sampled rows
    l = L - 1
    d_in, d_out = wl.dims[l], wl.dims[l + 1]
    agg_first = tr.orders[l] == mg.ORDER_AGG_FIRST
    # The gradient w.r.t. the logits is defined as zero outside the train mask; with a row plan the
    # library leaves those rows of the buffer alone (they are never read), and one layer down the same
    # holds for the rows outside the plan's row mask: the reference products apply the same row masks.
    def full_product(lhs, w_l, rhs, w_r, row_mask):
        """lhs^T rhs (w_l x w_r) and 1^T rhs in fp64 over row chunks -- the definition, evaluated by
        torch on the operands the library's call receives (teacher-forced), not by this library."""
        acc = torch.zeros(w_l, w_r, dtype=torch.float64, device="cuda")
        col = torch.zeros(w_r, dtype=torch.float64, device="cuda")
        step = 1 << 17
        for r0 in range(0, n, step):
            gb = rhs[r0:r0 + step, :w_r].double()
            if row_mask is not None:
                keep = row_mask[r0:r0 + step] != 0
                gb = torch.where(keep[:, None], gb, torch.zeros((), dtype=torch.float64, device="cuda"))
            acc += lhs[r0:r0 + step, :w_l].double().T @ gb
            col += gb.sum(dim=0)
        return acc, col

    ref_dW, ref_db = [None] * L, [None] * L

    def around_layer(k, when):
        # every layer's dW and db in full against the fp64 product of that call's own operands
        dk_in, dk_out = wl.dims[k], wl.dims[k + 1]
        rmask = tr.row_masks[k + 1] if tr.row_masks[k + 1] is not None else (tr.train_mask if k == L - 1 else None)
        if when == "before":
            if tr.orders[k] == mg.ORDER_AGG_FIRST:
                ref_dW[k], ref_db[k] = full_product(tr.aggregation_of(k), dk_in, tr.G[k + 1], dk_out, rmask)
            else:
                _, ref_db[k] = full_product(tr.X[k], dk_in, tr.G[k + 1], dk_out, rmask)
        elif tr.orders[k] == mg.ORDER_UPD_FIRST:
            ref_dW[k], _ = full_product(tr.X[k], dk_in, tr.saved[k], dk_out, None)     # dQ = A_hat^T dZ is left in `saved`

    dP_nodes = rows_of(tr.G[L], nodes, d_out)                      # gradient w.r.t. the logits, rows the sample needs
    dP_nodes = dP_nodes * tr.train_mask[torch.as_tensor(nodes, device="cuda")].cpu().numpy()[:, None]
    tr.backward(on_layer=around_layer)
    torch.cuda.synchronize()
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    Wt = tr.W[l].cpu().numpy().T.copy()
    gate = rows_of(tr.X[l], rows, d_in) > 0
    if agg_first:
        # G_in = gate(A_hat^T (dP W^T)); symmetric graph: A_hat^T = A_hat
        want_gin = orc.aggregate_rows(sub, orc.update(dP_nodes, Wt), crow)
        assert _rel(rows_of(tr.G[l], rows, d_in), want_gin * gate) <= tol
    else:
        # dQ = A_hat^T dP is left in `saved`; dW = X_in^T dQ; G_in = gate(dQ W^T)
        want_dq = orc.aggregate_rows(sub, dP_nodes, crow)
        assert _rel(rows_of(tr.saved[l], rows, d_out), want_dq) <= TOL_FP32
        assert _rel(rows_of(tr.G[l], rows, d_in), orc.update(rows_of(tr.saved[l], rows, d_out), Wt) * gate) <= tol
    for k in range(L):
        e_w = _rel(tr.dW[k].double().cpu().numpy(), ref_dW[k].cpu().numpy())
        e_b = _rel(tr.db[k].double().cpu().numpy(), ref_db[k].cpu().numpy())
        print(f"{key} ({wl.precision}): layer {k} weight gradient, relative Frobenius error vs the fp64 product of the same "
              f"operands: dW {e_w:.2e}  db {e_b:.2e}")
        assert e_w <= tol, f"dW[{k}]"
        assert e_b <= TOL_FP32 * 10, f"db[{k}]"          # a column sum in fp32 partials and an fp64 final pass
    for t in tr.dW + tr.db:
        assert bool(torch.isfinite(t).all())

    # ---- the iteration as the benchmark runs it: the loss taken inside the last layer's aggregation (no logits
    # written).  Its logits are the same fp32 numbers, so the predictions must be the separate calls' bit for bit.
    if tr.last_layer_takes_the_loss():
        ref_pred, ref_nc = tr.pred.clone(), int(tr.n_correct.item())
        grad_rows = train_idx[torch.as_tensor(pick, device="cuda")]
        tr.pred.fill_(-7); tr.X[L].fill_(float("nan"))
        tr.forward_and_loss()
        torch.cuda.synchronize()
        assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
        assert abs(tr.loss.item() - lo) <= 2e-6 * abs(lo)
        assert torch.equal(tr.pred, ref_pred) and int(tr.n_correct.item()) == ref_nc
        assert _rel(tr.X[L][grad_rows][:, :C].cpu().numpy(), Gt[pick]) <= TOL_FP32
        if tr.row_plans[L - 1] is None:
            assert float(tr.X[L][untrained][:, :C].abs().max()) == 0.0
        tr.backward()
        torch.cuda.synchronize()
        for k in range(L):
            assert _rel(tr.dW[k].double().cpu().numpy(), ref_dW[k].cpu().numpy()) <= tol, f"dW[{k}] with the loss inside the aggregation"
            assert _rel(tr.db[k].double().cpu().numpy(), ref_db[k].cpu().numpy()) <= TOL_FP32 * 10, f"db[{k}] with the loss inside the aggregation"

    # ---- the train-rows-only shortcut at full size: same loss and gradients as the full computation
    # above; rows outside the train mask hold NaN beforehand, so reading one of them would show
    ref_loss, ref_dW, ref_db = tr.loss.item(), [t.clone() for t in tr.dW], [t.clone() for t in tr.db]
    tr.configure(train_rows_only=True)
    assert tr.row_sparse_levels >= 1
    tr.X[L].fill_(float("nan"))
    if agg_first:
        tr.saved[l].fill_(float("nan"))
    tr.forward(); tr.compute_loss(); tr.backward()
    torch.cuda.synchronize()
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    assert abs(tr.loss.item() - ref_loss) <= 1e-5 * abs(ref_loss)
    for k in range(L):
        assert _rel(tr.dW[k].double().cpu().numpy(), ref_dW[k].double().cpu().numpy()) <= 4 * tol, f"dW[{k}] with the shortcut"
        assert _rel(tr.db[k].double().cpu().numpy(), ref_db[k].double().cpu().numpy()) <= 4 * tol, f"db[{k}] with the shortcut"
    g.close()
    ctx.close()
