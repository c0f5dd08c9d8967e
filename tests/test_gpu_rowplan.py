"""Row plans: the row-sparse aggregation on a matrix restricted ahead of time to the kept input rows.
Structure (kept rows, reachable output rows, kept entries) is checked bit-exactly against the
definition on the oracle's CSR; values against the oracle's full aggregation of the zero-padded input."""
import numpy as np
import pytest
import torch

from helpers import ADAM, TOL_FP32, host, padded, rel_fro, round4
from oracle import gcn_oracle as orc
from paper_2501_01951_b200 import synth
from test_gpu_parity import _tiny_problem, build_both

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2501_01951_b200 import build
    build.build()
    from paper_2501_01951_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(mg):
    c = mg.ctx_create(0)
    yield c
    assert mg.ctx_poll_status(c, raise_on_error=False) == 0
    c.close()


def _rmat_both(mg, ctx):
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    return orc.graph_build(wl.n, s.numpy(), d.numpy()), mg.graph_create(ctx, wl.n, s, d)


@pytest.mark.parametrize("name", ["messy-directed", "hub", "hub-directed", "rmat"])
@pytest.mark.parametrize("p", [0.0, 0.02, 0.5, 1.0])
@pytest.mark.parametrize("transposed", [True, False])
def test_rowplan_structure_and_aggregation(mg, ctx, name, p, transposed):
    go, gg = _rmat_both(mg, ctx) if name == "rmat" else build_both(mg, ctx, name)
    n, w = go.n, 44
    mask = synth.bernoulli_mask(n, p, 931) if 0.0 < p < 1.0 else torch.full((n,), int(p), dtype=torch.uint8)
    if 0.0 < p < 1.0:
        mask[0] = 1                                                   # the hub's column is kept
    plan = mg.rowplan_create(ctx, gg, mask.cuda(), transposed=transposed)
    keep = mask.numpy().astype(bool)
    rowptr, col = (go.rowptr_t, go.col_t) if transposed else (go.rowptr, go.col)
    kept_entry = keep[col]
    per_row = np.add.reduceat(np.concatenate([kept_entry.astype(np.int64), [0]]), rowptr[:-1]) * (np.diff(rowptr) > 0)
    assert plan.in_count == int(keep.sum()) and plan.nnz == int(kept_entry.sum())
    assert np.array_equal(plan.in_rows().cpu().numpy(), np.nonzero(keep)[0].astype(np.int32))
    out_mask = plan.out_row_mask().cpu().numpy()
    assert np.array_equal(out_mask.astype(bool), per_row > 0) and plan.out_count == int((per_row > 0).sum())
    # aggregation of the compacted input = the oracle's aggregation of the input with the other rows zero
    Y = synth.uniform_tensor((n, w), 932, -1, 1)
    Yz = Y.numpy() * keep[:, None]
    want = orc.aggregate(go, Yz, transposed=transposed)
    Yc = padded(Y[torch.as_tensor(np.nonzero(keep)[0])]) if keep.any() else torch.zeros(0, round4(w), device="cuda")
    Z = torch.full((n, round4(w)), 9.0, device="cuda")
    mg.spmm_rowplan(ctx, plan, Yc, Z, w)
    assert rel_fro(host(Z, w), want) <= TOL_FP32
    assert np.all(host(Z, w)[out_mask == 0] == 0.0)                  # rows without a kept entry are exactly zero
    Z2 = torch.full((n, round4(w)), 9.0, device="cuda")
    mg.spmm_rowplan(ctx, plan, Yc, Z2, w, rows_only=True)
    assert torch.equal(Z2[torch.as_tensor(out_mask.astype(bool))], Z[torch.as_tensor(out_mask.astype(bool))])
    assert np.all(host(Z2)[out_mask == 0] == 9.0)                    # left alone
    plan.close()
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("name", ["messy-directed", "hub"])
@pytest.mark.parametrize("order", ["agg", "upd"])
@pytest.mark.parametrize("gin_rows_only", [False, True])
def test_layer_bwd_with_row_plan_matches_dense_definition(mg, ctx, name, order, gin_rows_only):
    go, gg = build_both(mg, ctx, name)
    n, d_in, d_out = go.n, 40, 24
    o = mg.ORDER_AGG_FIRST if order == "agg" else mg.ORDER_UPD_FIRST
    X = synth.uniform_tensor((n, d_in), 301, -1, 1)
    W = synth.glorot_uniform(d_in, d_out, 302)
    b = synth.uniform_tensor((d_out,), 303, -0.2, 0.2)
    rows = synth.bernoulli_mask(n, 0.05, 304)
    rows[0] = 1
    Gout = synth.uniform_tensor((n, d_out), 305, -1, 1) * rows[:, None].float()
    flags = mg.LAYER_RELU | mg.LAYER_GATE_GIN | (mg.LAYER_GIN_ROWS_ONLY if gin_rows_only else 0)
    desc = mg.layer_desc(d_in, d_out, round4(d_in), round4(d_out), round4(max(d_in, d_out)), o, mg.PREC_FP32, flags)
    Xd, Wd, bd = padded(X), W.cuda(), b.cuda()
    saved = torch.zeros(n, round4(max(d_in, d_out)), device="cuda")
    Xout = torch.zeros(n, round4(d_out), device="cuda")
    mg.layer_fwd(ctx, gg, desc, Xd, Wd, bd, None, saved, Xout)
    plan = mg.rowplan_create(ctx, gg, rows.cuda())
    desc.gout_plan = plan.h
    Gd = padded(Gout)
    Gd[~rows.cuda().bool()] = float("nan")                           # only the plan's rows of G_out may be read
    Gin = torch.full((n, round4(d_in)), 5.0, device="cuda")
    dW = torch.zeros(d_in, d_out, device="cuda"); db = torch.zeros(d_out, device="cuda")
    mg.layer_bwd(ctx, gg, desc, Xd, saved, Xout, None, Wd, Gd, Gin, dW, db)
    Z = orc.aggregate(go, X.numpy())
    Pp = orc.update(Z, W.numpy(), b.numpy())
    _, dWo, dbo, dZo = orc.update_bwd(Z, Pp, W.numpy(), Gout.numpy(), True)
    want_gin = orc.aggregate(go, dZo, transposed=True) * (X.numpy() > 0)
    assert rel_fro(host(dW), dWo) <= TOL_FP32 and rel_fro(db.cpu().numpy(), dbo) <= TOL_FP32
    got = host(Gin, d_in)
    if gin_rows_only and order == "agg":
        om = plan.out_row_mask().cpu().numpy().astype(bool)
        assert rel_fro(got[om], want_gin[om]) <= TOL_FP32
        assert np.all(host(Gin)[~om] == 5.0) and np.all(want_gin[~om] == 0.0)
    else:
        assert rel_fro(got, want_gin) <= TOL_FP32
    plan.close()
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_row_plan_argument_checks(mg, ctx):
    go, gg = build_both(mg, ctx, "messy-sym")
    n = go.n
    with pytest.raises(ValueError):
        mg.rowplan_create(ctx, gg, torch.ones(n + 1, dtype=torch.uint8, device="cuda"))
    fwd_plan = mg.rowplan_create(ctx, gg, torch.ones(n, dtype=torch.uint8, device="cuda"), transposed=False)
    desc = mg.layer_desc(8, 8, 8, 8, 8, mg.ORDER_AGG_FIRST, mg.PREC_FP32, mg.LAYER_FIRST)
    desc.gout_plan = fwd_plan.h                                        # backward needs the transposed orientation
    X = torch.zeros(n, 8, device="cuda"); W = torch.zeros(8, 8, device="cuda"); dW = torch.zeros(8, 8, device="cuda")
    with pytest.raises(mg.MixgcnError):
        mg.layer_bwd(ctx, gg, desc, X, X.clone(), X.clone(), None, W, X.clone(), None, dW, None)
    with pytest.raises(ValueError):
        mg.spmm_rowplan(ctx, fwd_plan, torch.zeros(3, 8, device="cuda"), torch.zeros(n, 8, device="cuda"), 8)
    fwd_plan.close()
