"""The train-rows-only shortcut of the last layer: aggregation, update, loss and gradient computed on
the train rows alone (MIXGCN_LAYER_OUT_ROWS_ONLY, MIXGCN_OPT_LOSS_TRAIN_ROWS_ONLY).  The paper's
Algorithm 2 computes every row of H^(L); the loss reads train rows only, so loss and gradients must
be those of the full computation -- checked against the CPU oracle through the C-ABI."""
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


@pytest.mark.parametrize("name", ["messy-directed", "hub"])
@pytest.mark.parametrize("order", ["agg", "upd"])
@pytest.mark.parametrize("d_in,d_out", [(40, 24), (172, 9)])
def test_layer_fwd_out_rows_only(mg, ctx, name, order, d_in, d_out):
    """Kept rows carry the layer's output (the oracle's, and bitwise the unrestricted call's
    aggregation); every other row of X_out and of `saved` keeps what it held."""
    go, gg = build_both(mg, ctx, name)
    n = go.n
    o = mg.ORDER_AGG_FIRST if order == "agg" else mg.ORDER_UPD_FIRST
    X = synth.uniform_tensor((n, d_in), 901, -1, 1)
    W = synth.glorot_uniform(d_in, d_out, 902)
    b = synth.uniform_tensor((d_out,), 903, -0.2, 0.2)
    rows = synth.bernoulli_mask(n, 0.07, 904)
    rows[0] = 1                                                      # the hub row (cut into segments) is kept
    rows[n - 1] = 1
    ld_s = round4(max(d_in, d_out))
    desc = mg.layer_desc(d_in, d_out, round4(d_in), round4(d_out), ld_s, o, mg.PREC_FP32, mg.LAYER_RELU)
    Xd, Wd, bd = padded(X), W.cuda(), b.cuda()
    saved_full = torch.zeros(n, ld_s, device="cuda"); out_full = torch.zeros(n, round4(d_out), device="cuda")
    mg.layer_fwd(ctx, gg, desc, Xd, Wd, bd, None, saved_full, out_full)
    rows_d = rows.cuda()
    desc.flags |= mg.LAYER_OUT_ROWS_ONLY
    desc.gout_row_mask = rows_d.data_ptr(); desc.gout_row_count = int(rows.sum())
    saved = torch.full((n, ld_s), 5.0, device="cuda"); out = torch.full((n, round4(d_out)), 7.0, device="cuda")
    mg.layer_fwd(ctx, gg, desc, Xd, Wd, bd, None, saved, out)
    keep = rows.numpy().astype(bool)
    want = np.maximum(orc.update(orc.aggregate(go, X.numpy()), W.numpy(), b.numpy()), 0.0)
    got = host(out, d_out)
    assert rel_fro(got[keep], want[keep]) <= TOL_FP32
    assert np.all(out.cpu().numpy()[~keep] == 7.0)                   # untouched
    if order == "agg":
        assert torch.equal(saved[rows_d.bool(), :d_in], saved_full[rows_d.bool(), :d_in])   # same sums, same order
        assert np.all(saved.cpu().numpy()[~keep] == 5.0)
    else:
        assert torch.equal(out[rows_d.bool(), :d_out], out_full[rows_d.bool(), :d_out])
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_spmm_row_filter_on_skewed_graph_with_several_long_rows(mg, ctx):
    """R-MAT graph whose hubs are cut into segments: some long rows are kept and some are not."""
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s, d)
    n, d_in, d_out = wl.n, 64, 12
    lens = np.diff(go.rowptr)
    assert (lens > 512).sum() >= 2                                    # the case this test is about
    rows = synth.bernoulli_mask(n, 0.5, 921)
    longs = np.nonzero(lens > 512)[0]
    rows[int(longs[0])] = 1; rows[int(longs[1])] = 0                  # one long row in, one out
    W = synth.glorot_uniform(d_in, d_out, 922)
    desc = mg.layer_desc(d_in, d_out, d_in, round4(d_out), d_in, mg.ORDER_AGG_FIRST, mg.PREC_FP32, mg.LAYER_OUT_ROWS_ONLY)
    rows_d = rows.cuda()
    desc.gout_row_mask = rows_d.data_ptr(); desc.gout_row_count = int(rows.sum())
    saved = torch.full((n, d_in), 5.0, device="cuda"); out = torch.full((n, round4(d_out)), 7.0, device="cuda")
    mg.layer_fwd(ctx, gg, desc, padded(X), W.cuda(), None, None, saved, out)
    keep = rows.numpy().astype(bool)
    Z = orc.aggregate(go, X.numpy())
    assert rel_fro(host(saved)[keep], Z[keep]) <= TOL_FP32
    assert rel_fro(host(out, d_out)[keep], orc.update(Z, W.numpy(), None)[keep]) <= TOL_FP32
    assert np.all(host(saved)[~keep] == 5.0) and np.all(host(out)[~keep] == 7.0)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_out_rows_only_argument_checks(mg, ctx):
    go, gg = build_both(mg, ctx, "messy-sym")
    n, d = go.n, 8
    desc = mg.layer_desc(d, d, 8, 8, 8, mg.ORDER_AGG_FIRST, mg.PREC_FP32, mg.LAYER_OUT_ROWS_ONLY)
    X = torch.zeros(n, 8, device="cuda"); sv = torch.zeros(n, 8, device="cuda"); W = torch.zeros(d, d, device="cuda")
    out = torch.zeros(n, 8, device="cuda")
    with pytest.raises(mg.MixgcnError):                               # no row mask
        mg.layer_fwd(ctx, gg, desc, X, W, None, None, sv, out)
    rows = torch.ones(n, dtype=torch.uint8, device="cuda")
    desc.gout_row_mask = rows.data_ptr(); desc.gout_row_count = n
    drop = torch.ones(n, d, dtype=torch.uint8, device="cuda")
    with pytest.raises(mg.MixgcnError):                               # dropout mask not supported here
        mg.layer_fwd(ctx, gg, desc, X, W, None, drop, sv, out)
    mg.layer_fwd(ctx, gg, desc, X, W, None, None, sv, out)            # every row kept: fine
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("C", [7, 172, 300])
def test_loss_train_rows_only_option(mg, C):
    c2 = mg.ctx_create(0)
    n, ld = 3001, round4(C)
    logits = synth.uniform_tensor((n, C), 911, -4, 4)
    y = synth.uniform_labels(n, C, 912)
    m = synth.bernoulli_mask(n, 0.1, 913)
    P = padded(logits)
    loss0 = torch.zeros(1, device="cuda"); d0 = torch.zeros(n, ld, device="cuda")
    pred0 = torch.zeros(n, dtype=torch.int32, device="cuda"); nc0 = torch.zeros(1, dtype=torch.int64, device="cuda")
    mg.loss_softmax_xent(c2, P, y.cuda(), m.cuda(), loss0, dlogits=d0, pred=pred0, n_correct=nc0, C_=C)
    mg.ctx_set_option(c2, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 1)
    loss1 = torch.zeros(1, device="cuda"); d1 = torch.full((n, ld), 3.0, device="cuda")
    pred1 = torch.zeros(n, dtype=torch.int32, device="cuda"); nc1 = torch.zeros(1, dtype=torch.int64, device="cuda")
    mg.loss_softmax_xent(c2, P, y.cuda(), m.cuda(), loss1, dlogits=d1, pred=pred1, n_correct=nc1, C_=C)
    mg.ctx_set_option(c2, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 0)
    keep = m.numpy().astype(bool)
    ref = orc.loss(logits.numpy(), y.numpy(), m.numpy())
    assert abs(loss1.item() - ref[0]) <= 1e-5 * abs(ref[0])
    assert abs(loss1.item() - loss0.item()) <= 1e-6 * abs(loss0.item())
    assert rel_fro(host(d1, C)[keep], ref[1][keep]) <= TOL_FP32
    assert np.all(d1.cpu().numpy()[~keep] == 3.0)                    # rows outside the mask are left alone
    p1 = pred1.cpu().numpy()
    assert np.array_equal(p1[keep], pred0.cpu().numpy()[keep]) and np.all(p1[~keep] == -1)
    assert nc1.item() == nc0.item()
    # aliasing the logits (what the trainer does) gives the same train rows
    Pa = P.clone()
    mg.ctx_set_option(c2, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 1)
    mg.loss_softmax_xent(c2, Pa, y.cuda(), m.cuda(), loss1, dlogits=Pa, C_=C)
    mg.ctx_set_option(c2, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 0)
    assert torch.equal(Pa[m.cuda().bool(), :C], d1[m.cuda().bool(), :C])
    assert torch.equal(Pa[~m.cuda().bool()], P[~m.cuda().bool()])
    # value 2: logits of every row are read (pred everywhere), gradient rows outside the mask left alone
    mg.ctx_set_option(c2, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 2)
    loss2 = torch.zeros(1, device="cuda"); d2 = torch.full((n, ld), 3.0, device="cuda")
    pred2 = torch.zeros(n, dtype=torch.int32, device="cuda"); nc2 = torch.zeros(1, dtype=torch.int64, device="cuda")
    mg.loss_softmax_xent(c2, P, y.cuda(), m.cuda(), loss2, dlogits=d2, pred=pred2, n_correct=nc2, C_=C)
    mg.ctx_set_option(c2, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 0)
    assert loss2.item() == loss0.item() and nc2.item() == nc0.item() and torch.equal(pred2, pred0)
    assert torch.equal(d2[m.cuda().bool()], d0[m.cuda().bool()]) and np.all(d2.cpu().numpy()[~keep] == 3.0)
    with pytest.raises(mg.MixgcnError):
        mg.ctx_set_option(c2, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 3)
    assert mg.ctx_poll_status(c2, raise_on_error=False) == 0
    c2.close()


@pytest.mark.parametrize("levels", [1, 2])
@pytest.mark.parametrize("last_order", ["agg", "upd"])
def test_training_epochs_train_rows_only_match_oracle(mg, ctx, levels, last_order):
    """Two epochs with the shortcut: loss, train accuracy count, every gradient and the weight update
    are those of the oracle's full computation."""
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    m = synth.bernoulli_mask(wl.n, 0.03, 77)
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s, d)
    dims = (64, 32, 16, 8)
    Ws = [synth.glorot_uniform(dims[i], dims[i + 1], 400 + i) for i in range(3)]
    bs = [synth.uniform_tensor((dims[i + 1],), 410 + i, -0.1, 0.1) for i in range(3)]
    orders = [mg.ORDER_AGG_FIRST, mg.ORDER_AGG_FIRST, mg.ORDER_AGG_FIRST if last_order == "agg" else mg.ORDER_UPD_FIRST]
    tr = GcnTrainer(ctx, gg, dims, mg.PREC_FP32, order=orders, row_sparse=levels, train_rows_only=True)
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    tr.X[3].fill_(float("nan")); tr.saved[2].fill_(float("nan"))      # rows outside the mask must never be read
    Wo, bo, state = [w.numpy() for w in Ws], [b.numpy() for b in bs], None
    keep = m.numpy().astype(bool)
    for t in (1, 2):
        tr.forward(); tr.compute_loss(); tr.backward(); tr.step(t, **ADAM)
        ref = orc.train_epoch(go, X.numpy(), Wo, bo, y.numpy(), m.numpy(), state, t, **ADAM)
        assert abs(tr.loss.item() - ref["loss"]) <= 1e-5 * abs(ref["loss"])
        assert tr.n_correct.item() == ref["n_correct"]
        for l in range(3):
            assert rel_fro(tr.dW[l].cpu().numpy(), ref["dW"][l]) <= TOL_FP32
            assert rel_fro(tr.db[l].cpu().numpy(), ref["db"][l]) <= TOL_FP32
            big = np.abs(ref["dW"][l]) > 1e-4 * np.abs(ref["dW"][l]).max()
            dgpu = tr.W[l].cpu().numpy().astype(np.float64) - Wo[l]
            assert rel_fro(dgpu[big], (ref["W"][l] - Wo[l])[big]) <= 1e-3
        Wo, bo, state = ref["W"], ref["b"], ref["state"]
        tr.W = [torch.tensor(w, dtype=torch.float32, device="cuda") for w in Wo]
        tr.b = [torch.tensor(b, dtype=torch.float32, device="cuda") for b in bo]
        for l in range(3):
            tr.mW[l].copy_(torch.tensor(state["mW"][l])); tr.vW[l].copy_(torch.tensor(state["vW"][l]))
            tr.mb[l].copy_(torch.tensor(state["mb"][l])); tr.vb[l].copy_(torch.tensor(state["vb"][l]))
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_train_rows_only_needs_row_sparse_backward(mg, ctx):
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    gg = mg.graph_create(ctx, wl.n, s, d)
    tr = GcnTrainer(ctx, gg, wl.dims, mg.PREC_FP32, row_sparse=0, train_rows_only=True)
    tr.set_params(Ws, bs)
    with pytest.raises(ValueError):
        tr.set_inputs(padded(X), y.cuda(), m.cuda())


def test_cached_first_aggregation_matches_oracle_and_skips_the_call(mg):
    """Opt-in: A_hat X^(0) of the first layer is kept across iterations (features and graph do not
    change); every epoch still matches the oracle, which recomputes it."""
    from paper_2501_01951_b200.train import GcnTrainer
    c2 = mg.ctx_create(0)
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(c2, wl.n, s, d)
    tr = GcnTrainer(c2, gg, wl.dims, mg.PREC_FP32, order=mg.ORDER_AGG_FIRST, cache_first_aggregation=True)
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    Wo, bo, state = [w.numpy() for w in Ws], [b.numpy() for b in bs], None
    mg.ctx_profile_enable(c2, True)
    spmm_launches = []
    for t in (1, 2, 3):
        mg.ctx_profile_read(c2)
        tr.forward()
        _, launches, _ = mg.ctx_profile_read(c2)
        spmm_launches.append(launches["spmm"])
        tr.compute_loss(); tr.backward(); tr.step(t, **ADAM)
        ref = orc.train_epoch(go, X.numpy(), Wo, bo, y.numpy(), m.numpy(), state, t, **ADAM)
        assert abs(tr.loss.item() - ref["loss"]) <= 1e-5 * abs(ref["loss"])
        for l in range(tr.L):
            assert rel_fro(tr.dW[l].cpu().numpy(), ref["dW"][l]) <= TOL_FP32
            assert rel_fro(tr.db[l].cpu().numpy(), ref["db"][l]) <= TOL_FP32
        Wo, bo, state = ref["W"], ref["b"], ref["state"]
        tr.W = [torch.tensor(w, dtype=torch.float32, device="cuda") for w in Wo]
        tr.b = [torch.tensor(b, dtype=torch.float32, device="cuda") for b in bo]
        for l in range(tr.L):
            tr.mW[l].copy_(torch.tensor(state["mW"][l])); tr.vW[l].copy_(torch.tensor(state["vW"][l]))
            tr.mb[l].copy_(torch.tensor(state["mb"][l])); tr.vb[l].copy_(torch.tensor(state["vb"][l]))
    mg.ctx_profile_enable(c2, False)
    assert spmm_launches[1] == spmm_launches[2] < spmm_launches[0]   # one aggregation fewer from the second epoch on
    # new inputs invalidate the cached product
    X2 = synth.normal_features(wl.n, wl.dims[0], 4242)
    tr.set_inputs(padded(X2), y.cuda(), m.cuda())
    tr.forward()
    want = orc.aggregate(go, X2.numpy())
    assert rel_fro(host(tr.saved[0], wl.dims[0]), want) <= TOL_FP32
    # the flag is refused where `saved` would not survive the backward pass
    desc = mg.layer_desc(8, 8, 8, 8, 8, mg.ORDER_AGG_FIRST, mg.PREC_FP32, mg.LAYER_SAVED_IS_VALID)
    Z = torch.zeros(wl.n, 8, device="cuda"); W = torch.zeros(8, 8, device="cuda")
    with pytest.raises(mg.MixgcnError):
        mg.layer_fwd(c2, gg, desc, Z, W, None, None, Z.clone(), Z.clone())
    assert mg.ctx_poll_status(c2, raise_on_error=False) == 0
    gg.close(); c2.close()


@pytest.mark.parametrize("prec", ["tf32", "bf16"])
@pytest.mark.parametrize("row_plans", [True, False])
@pytest.mark.parametrize("rows_only", [False, True])
def test_low_precision_products_on_the_row_sparse_paths(mg, ctx, prec, row_plans, rows_only):
    """TF32 / BF16 products through the compacted-row backward (row plans or in-kernel row masks) and the
    train-rows-only last layer: the compact operands have no bf16 copy from a producer, so the library
    converts them on the fly.  Loss and the last layer's gradient (no ReLU mask below the loss) within the
    low-precision bound of the oracle; every other gradient within the inner-product bound."""
    from helpers import TOL_LOWP
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, _, _, _, _, _ = _tiny_problem()
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s, d)
    dims = (40, 32, 24, 10)
    n = go.n
    X = synth.normal_features(n, dims[0], 71)
    y = synth.uniform_labels(n, dims[-1], 72)
    m = synth.bernoulli_mask(n, 0.02, 73); m[5] = 1
    Ws = [synth.glorot_uniform(dims[l], dims[l + 1], 74 + l) for l in range(3)]
    bs = [synth.uniform_tensor((dims[l + 1],), 84 + l, -0.1, 0.1) for l in range(3)]
    ref = orc.train_epoch(go, X.numpy(), [w.numpy() for w in Ws], [b.numpy() for b in bs], y.numpy(), m.numpy(), None, 1, **ADAM)
    tr = GcnTrainer(ctx, gg, dims, mg.PRECISIONS[prec], order=mg.ORDER_AGG_FIRST, row_sparse=2, row_plans=row_plans,
                    train_rows_only=rows_only)
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    before = mg.ctx_gemm_paths(ctx)
    tr.forward(); tr.compute_loss(); tr.backward()
    torch.cuda.synchronize()
    after = mg.ctx_gemm_paths(ctx)
    key = "tc_tf32" if prec == "tf32" else "tc_bf16"
    assert after[key] - before[key] == 8 and after["simt"] == before["simt"]          # every product on the requested kernels
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    assert abs(tr.loss.item() - ref["loss"]) <= TOL_LOWP * abs(ref["loss"])
    assert rel_fro(tr.dW[2].cpu().numpy(), ref["dW"][2]) <= TOL_LOWP
    Gout = ref["G"]
    for l in range(2, -1, -1):
        dP, dW, db, dZ = orc.update_bwd(ref["Zs"][l], ref["Ps"][l], Ws[l].numpy(), Gout, relu=l < 2, need_dZ=l > 0)
        scale_w = np.linalg.norm(np.abs(ref["Zs"][l]).T @ np.abs(dP))
        assert np.linalg.norm(tr.dW[l].cpu().numpy() - ref["dW"][l]) <= TOL_LOWP * scale_w
        if l > 0:
            Gout = orc.aggregate(go, dZ, transposed=True)
    gg.close()
