"""Parity of the CUDA path (through the C-ABI) with the CPU oracle, element by element, on the
same seeded inputs.  Integer / index work must be bit-exact; fp32 results must agree with the
fp64 oracle within TOL_FP32 relative Frobenius error."""
import math

import numpy as np
import pytest
import torch

from helpers import ADAM, TOL_FP32, host, padded, rel_fro, round4
from oracle import gcn_oracle as orc
from paper_2501_01951_b200 import synth

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


def i32(a):
    return torch.tensor(np.asarray(a), dtype=torch.int32)


def messy_edges(n, m, seed):
    """Edge list with duplicates, both orientations, self-loops and isolated nodes."""
    rng = np.random.default_rng(seed)
    hi = max(1, (3 * n) // 4)                  # leave the top quarter of ids isolated
    src, dst = rng.integers(0, hi, m), rng.integers(0, hi, m)
    src[: m // 10] = dst[: m // 10]            # self-loops
    src = np.concatenate([src, src[: m // 5]])
    dst = np.concatenate([dst, dst[: m // 5]])  # duplicates
    return src.astype(np.int32), dst.astype(np.int32)


def star_plus(n, hub_deg, seed):
    """A hub of degree hub_deg (forces the CTA-per-row path) plus random edges."""
    rng = np.random.default_rng(seed)
    s = np.concatenate([np.zeros(hub_deg, np.int64), rng.integers(0, n, 3 * n)])
    d = np.concatenate([np.arange(1, hub_deg + 1), rng.integers(0, n, 3 * n)])
    return s.astype(np.int32), d.astype(np.int32)


GRAPHS = {
    "messy-sym": lambda: (300, *messy_edges(300, 2000, 1), True),
    "messy-directed": lambda: (257, *messy_edges(257, 1500, 2), False),
    "single-node": lambda: (1, np.zeros(0, np.int32), np.zeros(0, np.int32), True),
    "edgeless": lambda: (40, np.zeros(0, np.int32), np.zeros(0, np.int32), True),
    "hub": lambda: (9000, *star_plus(9000, 6000, 3), True),
    "hub-directed": lambda: (9000, *star_plus(9000, 6000, 4), False),
}


def build_both(mg, ctx, name):
    n, s, d, sym = GRAPHS[name]()
    flags_o = orc.ADD_SELF_LOOPS | (orc.SYMMETRISE if sym else 0)
    flags_g = mg.GRAPH_ADD_SELF_LOOPS | (mg.GRAPH_SYMMETRISE if sym else 0)
    go = orc.graph_build(n, s, d, flags_o)
    gg = mg.graph_create(ctx, n, i32(s), i32(d), flags_g)
    return go, gg


# --------------------------------------------------------------------------- S0 graph build

@pytest.mark.parametrize("name", list(GRAPHS))
@pytest.mark.parametrize("on_device", [False, True])
def test_graph_build_bit_exact(mg, ctx, name, on_device):
    n, s, d, sym = GRAPHS[name]()
    go = orc.graph_build(n, s, d, orc.ADD_SELF_LOOPS | (orc.SYMMETRISE if sym else 0))
    ts, td = i32(s), i32(d)
    if on_device:
        ts, td = ts.cuda(), td.cuda()
    gg = mg.graph_create(ctx, n, ts, td, mg.GRAPH_ADD_SELF_LOOPS | (mg.GRAPH_SYMMETRISE if sym else 0))
    assert (gg.n, gg.nnz) == (go.n, go.nnz)
    assert gg.max_deg == int(go.deg.max())
    e = mg.graph_export(gg)
    assert np.array_equal(e["rowptr"].numpy(), go.rowptr)
    assert np.array_equal(e["col"].numpy(), go.col)
    assert np.array_equal(e["deg"].numpy(), go.deg)
    assert e["dinv"].numpy().tobytes() == go.dinv32.tobytes()
    assert e["val"].numpy().tobytes() == go.val32.tobytes()
    et = mg.graph_export(gg, transposed=True)
    assert np.array_equal(et["rowptr"].numpy(), go.rowptr_t)
    assert np.array_equal(et["col"].numpy(), go.col_t)
    assert et["val"].numpy().tobytes() == go.val32[go.src_index_t].tobytes()
    is_sym = np.array_equal(go.rowptr, go.rowptr_t) and np.array_equal(go.col, go.col_t)
    assert gg.symmetric == is_sym
    # schedule: a permutation, by descending entry count, ties by ascending id
    perm = mg.graph_export_schedule(gg).numpy().astype(np.int64)
    assert np.array_equal(np.sort(perm), np.arange(n))
    key = (-go.deg[perm].astype(np.int64)) * (n + 1) + perm
    assert np.all(np.diff(key) > 0)


def test_graph_closed_forms(mg, ctx):
    n = 33
    s, d = np.triu_indices(n, 1)
    e = mg.graph_export(mg.graph_create(ctx, n, i32(s), i32(d)))
    assert int(e["rowptr"][-1]) == n * n
    np.testing.assert_allclose(e["val"].numpy(), 1.0 / n, rtol=2e-7)          # complete graph: J/n
    r = np.arange(n)
    e = mg.graph_export(mg.graph_create(ctx, n, i32(r), i32((r + 1) % n)))
    assert int(e["rowptr"][-1]) == 3 * n
    np.testing.assert_allclose(e["val"].numpy(), 1.0 / 3.0, rtol=2e-7)        # 2-regular
    e = mg.graph_export(mg.graph_create(ctx, n, i32([]), i32([])))
    assert np.array_equal(e["col"].numpy(), r) and np.all(e["val"].numpy() == 1.0)   # A_hat = I


def test_graph_tiny_workload_matches_oracle(mg, ctx):
    wl = synth.CONFIGS["C1"]
    s, d = synth.rmat_graph(wl.n, wl.undirected_edges, wl.seed("graph"))
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s.cuda(), d.cuda())
    e = mg.graph_export(gg)
    assert np.array_equal(e["rowptr"].numpy(), go.rowptr) and np.array_equal(e["col"].numpy(), go.col)
    assert e["val"].numpy().tobytes() == go.val32.tobytes()
    assert gg.symmetric


def test_graph_from_csr_and_validation(mg, ctx):
    go, _ = build_both(mg, ctx, "messy-directed")
    for dev in ("cpu", "cuda"):
        gg = mg.graph_create_from_csr(ctx, go.n, torch.tensor(go.rowptr).to(dev), torch.tensor(go.col).to(dev))
        e = mg.graph_export(gg)
        assert e["val"].numpy().tobytes() == go.val32.tobytes()
        et = mg.graph_export(gg, transposed=True)
        assert np.array_equal(et["col"].numpy(), go.col_t)
    rp = torch.tensor([0, 2, 3], dtype=torch.int64)
    for col in ([1, 0, 1], [0, 0, 1], [0, 5, 1]):                     # unsorted, duplicate, out of range
        with pytest.raises(mg.MixgcnError) as ex:
            mg.graph_create_from_csr(ctx, 2, rp, i32(col))
        assert ex.value.status == mg.EBADGRAPH
    with pytest.raises(mg.MixgcnError) as ex:
        mg.graph_create_from_csr(ctx, 2, torch.tensor([0, 3, 2], dtype=torch.int64), i32([0, 1, 1]))
    assert ex.value.status == mg.EBADGRAPH
    with pytest.raises(mg.MixgcnError) as ex:
        mg.graph_create(ctx, 4, i32([0, 7]), i32([1, 2]))
    assert ex.value.status == mg.EBADGRAPH
    with pytest.raises(mg.MixgcnError) as ex:
        mg.graph_create(ctx, 0, i32([]), i32([]))
    assert ex.value.status == mg.EINVAL


# --------------------------------------------------------------------------- S1 / S5 aggregation

WIDTHS = [1, 3, 4, 8, 41, 47, 64, 100, 128, 172, 256, 602, 1024, 1100]


@pytest.mark.parametrize("name", ["messy-sym", "messy-directed", "hub", "hub-directed", "edgeless"])
@pytest.mark.parametrize("w", WIDTHS)
def test_spmm_matches_oracle(mg, ctx, name, w):
    if name.startswith("hub") and w in (3, 47, 100, 602, 1100):
        pytest.skip("hub graphs cover a subset of widths")
    go, gg = build_both(mg, ctx, name)
    X = synth.uniform_tensor((go.n, w), seed=w + 11, lo=-2, hi=2)
    Y = padded(X, fill=float("nan"))                       # pad columns must never reach the result
    for transposed in (False, True):
        Z = torch.full((go.n, round4(w) + 4), 7.0, device="cuda")[:, : round4(w) + 4]
        mg.spmm(ctx, gg, Y, Z, w, transposed=transposed)
        want = orc.aggregate(go, X.numpy(), transposed=transposed)
        assert rel_fro(host(Z, w), want) <= TOL_FP32
        assert torch.all(Z[:, w:round4(w)] == 0) and torch.all(Z[:, round4(w):] == 7.0)


def test_spmm_closed_forms_and_determinism(mg, ctx):
    n = 64
    s, d = np.triu_indices(n, 1)
    gg = mg.graph_create(ctx, n, i32(s), i32(d))
    X = synth.normal_features(n, 20, 5)
    Y, Z = padded(X), torch.zeros(n, 20, device="cuda")
    mg.spmm(ctx, gg, Y, Z, 20)
    np.testing.assert_allclose(host(Z), np.tile(X.numpy().astype(np.float64).mean(0), (n, 1)), rtol=1e-5, atol=1e-6)
    # symmetric graph: sqrt(deg~) is a fixed point of the aggregation
    wl = synth.CONFIGS["C1"]
    s, d = synth.rmat_graph(wl.n, wl.undirected_edges, wl.seed("graph"))
    gg = mg.graph_create(ctx, wl.n, s, d)
    deg = mg.graph_export(gg)["deg"].float()
    R = padded(torch.sqrt(deg)[:, None].repeat(1, 4))
    Z = torch.zeros_like(R)
    mg.spmm(ctx, gg, R, Z, 4)
    assert rel_fro(host(Z), host(R)) <= TOL_FP32
    X = padded(synth.normal_features(wl.n, 64, 6))
    Z1, Z2 = torch.zeros_like(X), torch.zeros_like(X)
    mg.spmm(ctx, gg, X, Z1, 64)
    mg.spmm(ctx, gg, X, Z2, 64)
    assert torch.equal(Z1, Z2)                                     # bitwise reproducible


def test_spmm_epilogue(mg, ctx):
    go, gg = build_both(mg, ctx, "messy-directed")
    n, w = go.n, 41
    X = synth.uniform_tensor((n, w), 21, -1, 1)
    bias = synth.uniform_tensor((w,), 22, -0.5, 0.5)
    drop = (synth.uniform_tensor((n, w), 23, 0, 1) < 0.7).to(torch.uint8)
    gate = synth.uniform_tensor((n, w), 24, -1, 1)
    Z = torch.zeros(n, round4(w), device="cuda")
    epi = mg.make_epilogue(bias=bias.cuda(), relu=True, drop_mask=drop.cuda(), keep_scale=1 / 0.7,
                           gate=padded(gate), gate_scale=1.5)
    mg.spmm(ctx, gg, padded(X), Z, w, epi=epi)
    P = orc.aggregate(go, X.numpy()) + bias.numpy().astype(np.float64)
    want = orc.activation(P, True, drop.numpy(), 1 / 0.7) * np.where(gate.numpy() > 0, 1.5, 0.0)
    assert rel_fro(host(Z, w), want) <= TOL_FP32


# --------------------------------------------------------------------------- S2 / S4 dense update

GEMM_SHAPES = [  # M, N, K
    (1, 1, 1), (5, 3, 2), (130, 70, 33), (257, 41, 602), (300, 256, 100), (1000, 172, 128), (129, 129, 129),
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("ta,tb", [(False, False), (False, True), (True, False), (True, True)])
def test_gemm_fp32_matches_oracle(mg, ctx, M, N, K, ta, tb):
    A = synth.uniform_tensor((K, M) if ta else (M, K), 31 + M, -1, 1)
    B = synth.uniform_tensor((N, K) if tb else (K, N), 32 + N, -1, 1)
    Cd = torch.full((M, round4(N) + 4), 3.0, device="cuda")
    mg.gemm(ctx, mg.PREC_FP32, ta, tb, M, N, K, padded(A, fill=float("nan")), padded(B, fill=float("nan")), Cd)
    Ao = A.numpy().astype(np.float64).T if ta else A.numpy().astype(np.float64)
    Bo = B.numpy().astype(np.float64).T if tb else B.numpy().astype(np.float64)
    want = orc.update(Ao, Bo)
    assert rel_fro(host(Cd, N), want) <= TOL_FP32
    assert torch.all(Cd[:, round4(N):] == 3.0)


def test_gemm_unaligned_weight_matrix(mg, ctx):
    """W is dense d_in x d_out with d_out % 4 != 0: its rows are not 16-byte aligned."""
    M, N, K = 200, 41, 100
    A, W = synth.uniform_tensor((M, K), 1, -1, 1), synth.uniform_tensor((K, N), 2, -1, 1)
    Cd = torch.zeros(M, round4(N), device="cuda")
    mg.gemm(ctx, mg.PREC_FP32, False, False, M, N, K, padded(A), W.cuda(), Cd)
    assert rel_fro(host(Cd, N), orc.update(A.numpy(), W.numpy())) <= TOL_FP32
    dW = torch.zeros(K, N, device="cuda")
    G = synth.uniform_tensor((M, N), 3, -1, 1)
    mg.gemm(ctx, mg.PREC_FP32, True, False, K, N, M, padded(A), padded(G), dW)
    assert rel_fro(host(dW), A.numpy().astype(np.float64).T @ G.numpy().astype(np.float64)) <= TOL_FP32


def test_gemm_long_reduction_split_k(mg, ctx):
    """Weight-gradient shape: K = number of nodes, split over CTAs, fixed-order reduction."""
    M, N, K = 100, 47, 70001
    A, B = synth.normal_features(K, M, 41), synth.normal_features(K, N, 42)
    Cd1, Cd2 = torch.zeros(M, round4(N), device="cuda"), torch.zeros(M, round4(N), device="cuda")
    mg.gemm(ctx, mg.PREC_FP32, True, False, M, N, K, padded(A), padded(B), Cd1)
    mg.gemm(ctx, mg.PREC_FP32, True, False, M, N, K, padded(A), padded(B), Cd2)
    want = A.numpy().astype(np.float64).T @ B.numpy().astype(np.float64)
    assert rel_fro(host(Cd1, N), want) <= TOL_FP32
    assert torch.equal(Cd1, Cd2)


def test_gemm_epilogue(mg, ctx):
    M, N, K = 150, 70, 50
    A, B = synth.uniform_tensor((M, K), 51, -1, 1), synth.uniform_tensor((K, N), 52, -1, 1)
    bias = synth.uniform_tensor((N,), 53, -1, 1)
    drop = (synth.uniform_tensor((M, N), 54, 0, 1) < 0.5).to(torch.uint8)
    Cd = torch.zeros(M, round4(N), device="cuda")
    epi = mg.make_epilogue(bias=bias.cuda(), relu=True, drop_mask=drop.cuda(), keep_scale=2.0)
    mg.gemm(ctx, mg.PREC_FP32, False, False, M, N, K, padded(A), padded(B), Cd, epi=epi)
    want = orc.activation(orc.update(A.numpy(), B.numpy(), bias.numpy()), True, drop.numpy(), 2.0)
    assert rel_fro(host(Cd, N), want) <= TOL_FP32


# --------------------------------------------------------------------------- S3 loss

@pytest.mark.parametrize("Cc", [1, 8, 41, 47, 64, 172, 1000])
def test_loss_matches_oracle(mg, ctx, Cc):
    n = 777
    P = synth.uniform_tensor((n, Cc), 60 + Cc, -6, 6)
    labels = synth.uniform_labels(n, Cc, 61)
    mask = synth.bernoulli_mask(n, 0.4, 62)
    lo, G, pred, nc, T = orc.loss(P.numpy(), labels.numpy(), mask.numpy())
    Pd = padded(P)
    loss = torch.zeros(1, device="cuda"); Gd = torch.full_like(Pd, 9.0)
    predd = torch.zeros(n, dtype=torch.int32, device="cuda"); ncd = torch.zeros(1, dtype=torch.int64, device="cuda")
    mg.loss_softmax_xent(ctx, Pd, labels.cuda(), mask.cuda(), loss, Gd, predd, ncd, C_=Cc)
    assert abs(loss.item() - lo) <= 1e-6 * max(1.0, abs(lo))
    assert rel_fro(host(Gd, Cc), G) <= TOL_FP32
    assert np.array_equal(predd.cpu().numpy(), pred) and ncd.item() == nc         # arg-max: bit-exact
    assert torch.all(Gd[mask.cuda() == 0, :Cc] == 0)
    # in place over the logits
    P2 = Pd.clone()
    mg.loss_softmax_xent(ctx, P2, labels.cuda(), mask.cuda(), loss, P2, None, None, C_=Cc)
    assert torch.equal(P2[:, :Cc], Gd[:, :Cc])


@pytest.mark.parametrize("Cc,ld", [(41, 256), (172, 176), (47, 64)])
def test_loss_on_a_column_slice_leaves_the_other_columns_alone(mg, ctx, Cc, ld):
    """logits / dlogits are n x C views of a wider buffer (ld > round4(C)): columns beyond the pad to a
    multiple of 4 belong to the caller and must survive, and the result must be the dense layout's."""
    n = 1500
    P = synth.uniform_tensor((n, Cc), 160 + Cc, -6, 6)
    labels = synth.uniform_labels(n, Cc, 161)
    mask = synth.bernoulli_mask(n, 0.3, 162)
    lo, G, pred, nc, T = orc.loss(P.numpy(), labels.numpy(), mask.numpy())
    wide = torch.full((n, ld), 123.0, device="cuda")
    wide[:, :Cc] = P.cuda()
    Gw = torch.full((n, ld), -77.0, device="cuda")
    loss = torch.zeros(1, device="cuda")
    predd = torch.zeros(n, dtype=torch.int32, device="cuda"); ncd = torch.zeros(1, dtype=torch.int64, device="cuda")
    mg.loss_softmax_xent(ctx, wide, labels.cuda(), mask.cuda(), loss, Gw, predd, ncd, C_=Cc)
    assert abs(loss.item() - lo) <= 1e-6 * max(1.0, abs(lo))
    assert rel_fro(host(Gw, Cc), G) <= TOL_FP32
    assert np.array_equal(predd.cpu().numpy(), pred) and ncd.item() == nc
    assert torch.all(Gw[:, round4(Cc):] == -77.0) and torch.all(wide[:, Cc:] == 123.0)
    # in place over the slice
    mg.loss_softmax_xent(ctx, wide, labels.cuda(), mask.cuda(), loss, wide, None, None, C_=Cc)
    assert rel_fro(host(wide, Cc), G) <= TOL_FP32 and torch.all(wide[:, round4(Cc):] == 123.0)


def test_loss_closed_form_and_ties(mg, ctx):
    n, Cc = 50, 41
    labels = synth.uniform_labels(n, Cc, 1).cuda()
    mask = torch.ones(n, dtype=torch.uint8, device="cuda")
    loss = torch.zeros(1, device="cuda"); pred = torch.ones(n, dtype=torch.int32, device="cuda")
    mg.loss_softmax_xent(ctx, torch.zeros(n, round4(Cc), device="cuda"), labels, mask, loss, None, pred, None, C_=Cc)
    assert abs(loss.item() - math.log(Cc)) < 1e-6 and torch.all(pred == 0)


def test_loss_device_side_errors_set_the_status_word(mg, ctx):
    n, Cc = 20, 5
    P = torch.zeros(n, 8, device="cuda"); loss = torch.ones(1, device="cuda"); G = torch.ones(n, 8, device="cuda")
    labels = torch.zeros(n, dtype=torch.int32, device="cuda")
    mg.loss_softmax_xent(ctx, P, labels, torch.zeros(n, dtype=torch.uint8, device="cuda"), loss, G, None, None, C_=Cc)
    with pytest.raises(mg.MixgcnError) as e:
        mg.ctx_poll_status(ctx)
    assert e.value.status == mg.EDEVICE and loss.item() == 0 and torch.all(G[:, :Cc] == 0)
    labels[3] = 9
    mg.loss_softmax_xent(ctx, P, labels, torch.ones(n, dtype=torch.uint8, device="cuda"), loss, G, None, None, C_=Cc)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 2
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0      # cleared by the read


# --------------------------------------------------------------------------- S6 Adam

def test_adam_matches_oracle(mg, ctx):
    shapes = [(64, 32), (32,), (1024, 100), (7,)] + [(3, 5)] * 20        # > one batch of tensors
    P = [synth.uniform_tensor(s, 70 + i, -1, 1) for i, s in enumerate(shapes)]
    pd = [p.cuda() for p in P]
    md = [torch.zeros_like(p) for p in pd]; vd = [torch.zeros_like(p) for p in pd]
    po = [p.numpy().astype(np.float64) for p in P]
    mo = [np.zeros_like(p) for p in po]; vo = [np.zeros_like(p) for p in po]
    for t in range(1, 5):
        Gs = [synth.uniform_tensor(s, 100 * t + i, -1e-2, 1e-2) for i, s in enumerate(shapes)]
        mg.adam_step(ctx, pd, [g.cuda() for g in Gs], md, vd, t, **ADAM)
        for i in range(len(shapes)):
            po[i], mo[i], vo[i] = orc.adam(po[i], Gs[i].numpy(), mo[i], vo[i], t, **ADAM)
    for i in range(len(shapes)):
        assert rel_fro(pd[i].cpu().numpy(), po[i]) <= 1e-6
        assert rel_fro(md[i].cpu().numpy(), mo[i]) <= 1e-6 and rel_fro(vd[i].cpu().numpy(), vo[i]) <= 1e-6


# --------------------------------------------------------------------------- layers and whole epochs

def _run_layer(mg, ctx, go, gg, d_in, d_out, order, relu, first, use_drop, n_chunks, seed):
    n = go.n
    X = synth.uniform_tensor((n, d_in), seed, -1, 1)
    W = synth.glorot_uniform(d_in, d_out, seed + 1)
    b = synth.uniform_tensor((d_out,), seed + 2, -0.2, 0.2)
    Gout = synth.uniform_tensor((n, d_out), seed + 3, -1, 1)
    drop = (synth.uniform_tensor((n, d_out), seed + 4, 0, 1) < 0.6).to(torch.uint8) if use_drop else None
    ks = 1 / 0.6 if use_drop else 1.0
    flags = (mg.LAYER_RELU if relu else 0) | (mg.LAYER_FIRST if first else 0)
    desc = mg.layer_desc(d_in, d_out, round4(d_in), round4(d_out), round4(max(d_in, d_out)), order, mg.PREC_FP32,
                         flags, ks, 1.0, n_chunks)
    Xd, Wd, bd = padded(X), W.cuda(), b.cuda()
    dropd = None if drop is None else drop.cuda()
    saved = torch.zeros(n, round4(max(d_in, d_out)), device="cuda")
    Xout = torch.zeros(n, round4(d_out), device="cuda")
    mg.layer_fwd(ctx, gg, desc, Xd, Wd, bd, dropd, saved, Xout)
    Z = orc.aggregate(go, X.numpy())
    Pp = orc.update(Z, W.numpy(), b.numpy())
    want = orc.activation(Pp, relu, None if drop is None else drop.numpy(), ks)
    assert rel_fro(host(Xout, d_out), want) <= TOL_FP32
    Gd = padded(Gout)
    Gin = None if first else torch.zeros(n, round4(d_in), device="cuda")
    dW = torch.zeros(d_in, d_out, device="cuda"); db = torch.zeros(d_out, device="cuda")
    mg.layer_bwd(ctx, gg, desc, Xd, saved, Xout, dropd, Wd, Gd, Gin, dW, db)
    _, dWo, dbo, dZo = orc.update_bwd(Z, Pp, W.numpy(), Gout.numpy(), relu, None if drop is None else drop.numpy(),
                                      ks, need_dZ=not first)
    assert rel_fro(host(dW), dWo) <= TOL_FP32 and rel_fro(db.cpu().numpy(), dbo) <= TOL_FP32
    if not first:
        assert rel_fro(host(Gin, d_in), orc.aggregate(go, dZo, transposed=True)) <= TOL_FP32


@pytest.mark.parametrize("name", ["messy-sym", "messy-directed"])
@pytest.mark.parametrize("order", ["agg", "upd"])
@pytest.mark.parametrize("d_in,d_out", [(64, 32), (33, 41), (8, 100)])
def test_layer_fwd_bwd_both_orders(mg, ctx, name, order, d_in, d_out):
    go, gg = build_both(mg, ctx, name)
    o = mg.ORDER_AGG_FIRST if order == "agg" else mg.ORDER_UPD_FIRST
    _run_layer(mg, ctx, go, gg, d_in, d_out, o, relu=True, first=False, use_drop=True, n_chunks=0, seed=80)
    _run_layer(mg, ctx, go, gg, d_in, d_out, o, relu=False, first=True, use_drop=False, n_chunks=0, seed=90)


@pytest.mark.parametrize("n_chunks", [2, 3, 7])
def test_layer_chunked_pipeline_matches_unchunked(mg, ctx, n_chunks):
    go, gg = build_both(mg, ctx, "hub")
    _run_layer(mg, ctx, go, gg, 64, 48, mg.ORDER_AGG_FIRST, relu=True, first=False, use_drop=True,
               n_chunks=n_chunks, seed=95)


@pytest.mark.parametrize("name", ["messy-sym", "messy-directed", "hub"])
@pytest.mark.parametrize("w", [8, 41, 128, 300])
@pytest.mark.parametrize("transposed", [False, True])
def test_sampled_spmm_matches_eq4(mg, ctx, name, w, transposed):
    """Z = (A_hat Y) (.) M (Eq. 4) with M as a bitmap: against the oracle, bitwise equal to the unmasked
    aggregation where the mask keeps an output, exactly zero where it does not -- for a random half mask, a
    mask with whole 16-byte groups and whole rows dropped (the loads that can be skipped), and the ReLU form."""
    go, gg = build_both(mg, ctx, name)
    n = go.n
    Y = synth.uniform_tensor((n, w), 511 + w, -1, 1)
    ld_bits = (w + 31) // 32 + 1                                     # one spare word per row: must stay untouched
    Yd = padded(Y, fill=float("nan"))
    plain = torch.zeros(n, round4(w), device="cuda")
    mg.spmm(ctx, gg, Yd, plain, w, transposed=transposed)
    rng = np.random.default_rng(w)
    M1 = rng.integers(0, 2, (n, w)).astype(np.uint8)
    M2 = np.repeat(rng.integers(0, 2, (n, (w + 3) // 4)), 4, axis=1)[:, :w].astype(np.uint8)
    M2[rng.integers(0, 2, n) == 0] = 0
    for M in (M1, M2):
        bits = torch.full((n, ld_bits), -1, dtype=torch.int32, device="cuda")
        mg.mask_pack(ctx, w, bits, bytes_mask=torch.tensor(M).cuda().contiguous())
        assert torch.all(bits[:, -1] == -1)
        Z = torch.full((n, round4(w)), 7.0, device="cuda")
        mg.spmm_sampled(ctx, gg, Yd, Z, w, bits, transposed=transposed)
        want = orc.sampled_aggregate(go, Y.numpy(), M, transposed=transposed)
        assert rel_fro(host(Z, w), want) <= TOL_FP32
        Mt = torch.tensor(M).cuda().bool()
        assert torch.equal(Z[:, :w][Mt], plain[:, :w][Mt]) and torch.all(Z[:, :w][~Mt] == 0)
    # backward form: the mask is the ReLU mask of another activation
    A = synth.uniform_tensor((n, w), 512 + w, -1, 1)
    bits = torch.zeros((n, ld_bits), dtype=torch.int32, device="cuda")
    mg.mask_pack(ctx, w, bits, X=padded(A))
    Z = torch.zeros(n, round4(w), device="cuda")
    mg.spmm_sampled(ctx, gg, Yd, Z, w, bits, transposed=transposed)
    assert rel_fro(host(Z, w), orc.sampled_aggregate(go, Y.numpy(), A.numpy() > 0, transposed=transposed)) <= TOL_FP32
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("d_in,d_out", [(64, 41), (128, 172), (40, 300), (130, 260)])
@pytest.mark.parametrize("prec", ["tf32", "bf16", "fp32"])
def test_bias_gradient_beside_the_weight_gradient(mg, ctx, d_in, d_out, prec):
    """db = 1^T dP comes out of the weight-gradient product's kernel where that kernel reads dP as fp32 words
    (TF32), from the column-sum kernels otherwise: either way it must be the column sum of the gradient the
    call was given, to fp32 accuracy, whatever the width (tiles of 32-column chunks, ragged last chunk)."""
    from helpers import TOL_LOWP
    go, gg = build_both(mg, ctx, "hub")
    n = go.n
    X = synth.uniform_tensor((n, d_in), 611, -1, 1); W = synth.glorot_uniform(d_in, d_out, 612)
    G = synth.uniform_tensor((n, d_out), 613, -1, 1) + 0.25           # column sums well away from zero
    desc = mg.layer_desc(d_in, d_out, round4(d_in), round4(d_out), round4(d_in), mg.ORDER_AGG_FIRST, mg.PRECISIONS[prec], 0)
    Xd, Wd = padded(X), W.cuda()
    saved = torch.zeros(n, round4(d_in), device="cuda"); Xout = torch.zeros(n, round4(d_out), device="cuda")
    mg.layer_fwd(ctx, gg, desc, Xd, Wd, None, None, saved, Xout)
    Gd = padded(G, fill=float("nan")); Gin = torch.zeros(n, round4(d_in), device="cuda")
    dW = torch.zeros(d_in, d_out, device="cuda"); db = torch.full((d_out,), 9.0, device="cuda")
    mg.layer_bwd(ctx, gg, desc, Xd, saved, Xout, None, Wd, Gd, Gin, dW, db)
    want_db = G.numpy().astype(np.float64).sum(axis=0)
    assert rel_fro(db.cpu().numpy(), want_db) <= 1e-6
    Z = orc.aggregate(go, X.numpy())
    assert rel_fro(host(dW), Z.T @ G.numpy().astype(np.float64)) <= (TOL_FP32 if prec == "fp32" else TOL_LOWP)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def _tiny_problem():
    wl = synth.CONFIGS["C1"]
    s, d = synth.rmat_graph(wl.n, wl.undirected_edges, wl.seed("graph"))
    X = synth.normal_features(wl.n, wl.dims[0], wl.seed("features"))
    y = synth.uniform_labels(wl.n, wl.classes, wl.seed("labels"))
    m = synth.bernoulli_mask(wl.n, wl.mask_p, wl.seed("mask"))
    Ws, bs = synth.make_weights(wl)
    return wl, s, d, X, y, m, Ws, bs


@pytest.mark.parametrize("order", ["auto", "agg", "upd"])
@pytest.mark.parametrize("fuse_gate", [True, False])
def test_training_epochs_match_oracle_on_tiny(mg, ctx, order, fuse_gate):
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s, d)
    o = {"auto": mg.ORDER_AUTO, "agg": mg.ORDER_AGG_FIRST, "upd": mg.ORDER_UPD_FIRST}[order]
    tr = GcnTrainer(ctx, gg, wl.dims, mg.PREC_FP32, order=o, fuse_gate=fuse_gate)
    if order == "auto":
        assert tr.orders == [mg.ORDER_AGG_FIRST, mg.ORDER_UPD_FIRST]
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    Wo, bo, state = [w.numpy() for w in Ws], [b.numpy() for b in bs], None
    for t in range(1, 4):
        tr.forward()
        logits = host(tr.X[-1], wl.classes).copy()
        tr.compute_loss(); tr.backward(); tr.step(t, **ADAM)
        ref = orc.train_epoch(go, X.numpy(), Wo, bo, y.numpy(), m.numpy(), state, t, **ADAM)
        assert rel_fro(logits, ref["logits"]) <= TOL_FP32
        assert abs(tr.loss.item() - ref["loss"]) <= 1e-5 * abs(ref["loss"])
        # arg-max must agree wherever the oracle's top-2 gap is not a near-tie
        top2 = np.sort(ref["logits"], axis=1)[:, -2:]
        clear = (top2[:, 1] - top2[:, 0]) > 1e-4 * np.abs(ref["logits"]).max()
        assert np.array_equal(tr.pred.cpu().numpy()[clear], ref["pred"][clear])
        for l in range(tr.L):
            assert rel_fro(tr.dW[l].cpu().numpy(), ref["dW"][l]) <= TOL_FP32
            assert rel_fro(tr.db[l].cpu().numpy(), ref["db"][l]) <= TOL_FP32
            # Adam turns g into ~sign(g) when |g| is tiny: compare the update where g is not negligible
            gmax = np.abs(ref["dW"][l]).max()
            big = np.abs(ref["dW"][l]) > 1e-4 * gmax
            dgpu = tr.W[l].cpu().numpy().astype(np.float64) - Wo[l]
            dref = ref["W"][l] - Wo[l]
            assert rel_fro(dgpu[big], dref[big]) <= 1e-3
        # continue both sides from the oracle's weights so that one side's rounding does not compound
        Wo, bo, state = ref["W"], ref["b"], ref["state"]
        tr.W = [torch.tensor(w, dtype=torch.float32, device="cuda") for w in Wo]
        tr.b = [torch.tensor(b, dtype=torch.float32, device="cuda") for b in bo]
        for l in range(tr.L):
            tr.mW[l].copy_(torch.tensor(state["mW"][l])); tr.vW[l].copy_(torch.tensor(state["vW"][l]))
            tr.mb[l].copy_(torch.tensor(state["mb"][l])); tr.vb[l].copy_(torch.tensor(state["vb"][l]))


def test_epoch_is_bitwise_deterministic(mg, ctx):
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    gg = mg.graph_create(ctx, wl.n, s, d)
    outs = []
    for _ in range(2):
        tr = GcnTrainer(ctx, gg, wl.dims, mg.PREC_FP32)
        tr.set_params(Ws, bs)
        tr.set_inputs(padded(X), y.cuda(), m.cuda())
        for t in range(1, 3):
            tr.epoch(t)
        outs.append([w.clone() for w in tr.W] + [tr.loss.clone()])
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_argument_errors(mg, ctx):
    go, gg = build_both(mg, ctx, "messy-sym")
    n = go.n
    Y, Z = torch.zeros(n, 8, device="cuda"), torch.zeros(n, 8, device="cuda")
    with pytest.raises(mg.MixgcnError) as e:
        mg.spmm(ctx, gg, Y, Z, 0)
    assert e.value.status == mg.EINVAL
    with pytest.raises(mg.MixgcnError):
        mg.spmm(ctx, gg, Y, Y, 8)                                   # overlap
    with pytest.raises(mg.MixgcnError):
        mg.spmm(ctx, gg, Y, Z, 12)                                  # ld < w
    with pytest.raises(mg.MixgcnError):
        mg.spmm(ctx, gg, torch.zeros(n, 9, device="cuda")[:, :6], Z, 6)   # ld % 4 != 0
    with pytest.raises(mg.MixgcnError):
        mg.adam_step(ctx, [Y], [Y], [Y], [Y], 0)                    # t < 1
    assert torch.all(Z == 0)                                         # outputs untouched on host-side errors


def test_train_step_host_matches_oracle_and_device_path(mg, ctx):
    """The host-buffer entry point runs the same kernels as the device-buffer calls."""
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    gg = mg.graph_create(ctx, wl.n, s, d)
    W = [w.clone() for w in Ws]; b = [x.clone() for x in bs]
    mW = [torch.zeros_like(w) for w in W]; vW = [torch.zeros_like(w) for w in W]
    mb = [torch.zeros_like(x) for x in b]; vb = [torch.zeros_like(x) for x in b]
    pred = torch.zeros(wl.n, dtype=torch.int32)
    tr = GcnTrainer(ctx, gg, wl.dims, mg.PREC_FP32)
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    for t in (1, 2):
        loss = mg.train_step_host(ctx, gg, wl.dims, mg.PREC_FP32, X, y, m, W, b, mW, vW, mb, vb, t, pred=pred, **ADAM)
        tr.forward_and_loss(); tr.backward(); tr.step(t, **ADAM)      # the iteration as epoch() runs it
        assert loss == tr.loss.item()
        for l in range(tr.L):
            assert torch.equal(W[l], tr.W[l].cpu()) and torch.equal(b[l], tr.b[l].cpu())
            assert torch.equal(mW[l], tr.mW[l].cpu()) and torch.equal(vb[l], tr.vb[l].cpu())
        assert torch.equal(pred, tr.pred.cpu())
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    ref = orc.train_epoch(go, X.numpy(), [w.numpy() for w in Ws], [x.numpy() for x in bs], y.numpy(), m.numpy(), None, 1, **ADAM)
    W1 = [w.clone() for w in Ws]; b1 = [x.clone() for x in bs]
    z = lambda lst: [torch.zeros_like(x) for x in lst]
    loss = mg.train_step_host(ctx, gg, wl.dims, mg.PREC_FP32, X, y, m, W1, b1, z(W1), z(W1), z(b1), z(b1), 1, **ADAM)
    assert abs(loss - ref["loss"]) <= 1e-5 * abs(ref["loss"])


def test_train_step_host_prefetch_gives_the_same_iterations(mg):
    """Announcing the next call's features lets a call start their copy early; the iterations must be the
    ones without the announcement, bit for bit, also when the features change between calls, when the
    announcement is not honoured by the next call, and with the oracle's loss on the first step."""
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    Xa = X.clone().pin_memory()
    Xb = (X * 0.5 + 0.25).contiguous().pin_memory()
    feats = [Xa, Xb, Xb, Xa, Xa]
    results = []
    for announce in (False, True):
        c = mg.ctx_create(0)
        gg = mg.graph_create(c, wl.n, s, d)
        W = [w.clone() for w in Ws]; b = [x.clone() for x in bs]
        z = lambda lst: [torch.zeros_like(x) for x in lst]
        mW, vW, mb, vb = z(W), z(W), z(b), z(b)
        losses = []
        for t, Xt in enumerate(feats, start=1):
            if announce and t < len(feats):
                # step 3 announces a buffer the next call does not use: the announcement must simply lapse
                mg.train_step_host_prefetch(c, Xb if t == 3 else feats[t])
            losses.append(mg.train_step_host(c, gg, wl.dims, mg.PREC_FP32, Xt, y, m, W, b, mW, vW, mb, vb, t, **ADAM))
        assert mg.ctx_poll_status(c, raise_on_error=False) == 0
        results.append((losses, [w.clone() for w in W], [x.clone() for x in b]))
        gg.close(); c.close()
    assert results[0][0] == results[1][0]
    for a, b_ in zip(results[0][1] + results[0][2], results[1][1] + results[1][2]):
        assert torch.equal(a, b_)
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    ref = orc.train_epoch(go, X.numpy(), [w.numpy() for w in Ws], [x.numpy() for x in bs], y.numpy(), m.numpy(), None, 1, **ADAM)
    assert abs(results[1][0][0] - ref["loss"]) <= 1e-5 * abs(ref["loss"])


# --------------------------------------------------------------------------- tensor-core products

def _tf32_trunc(a):
    """fp32 values with the 13 low mantissa bits cleared (what a TF32 operand read keeps)."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) & np.uint32(0xFFFFE000)
    return b.view(np.float32).astype(np.float64)


TC_SHAPES = [  # M, N, K
    (128, 128, 32), (128, 16, 8), (300, 41, 100), (257, 256, 602), (1000, 172, 128), (640, 1024, 256), (513, 602, 47),
]


@pytest.mark.parametrize("M,N,K", TC_SHAPES)
@pytest.mark.parametrize("tb", [False, True])
def test_gemm_tf32_forward_forms(mg, ctx, M, N, K, tb):
    from helpers import TOL_LOWP
    A = synth.uniform_tensor((M, K), 131 + M, -1, 1)
    B = synth.uniform_tensor((N, K) if tb else (K, N), 132 + N, -1, 1)
    bias = synth.uniform_tensor((N,), 133, -1, 1)
    Cd = torch.full((M, round4(N) + 4), 3.0, device="cuda")
    epi = mg.make_epilogue(bias=bias.cuda(), relu=True)
    mg.gemm(ctx, mg.PREC_TF32, False, tb, M, N, K, padded(A, fill=float("nan")), B.cuda().contiguous(), Cd, epi=epi)
    Bo = B.numpy().T if tb else B.numpy()
    want = orc.activation(orc.update(A.numpy(), Bo, bias.numpy()), True)
    assert rel_fro(host(Cd, N), want) <= TOL_LOWP
    assert torch.all(Cd[:, round4(N):] == 3.0)
    # tighter: against the product of TF32-truncated operands the result is fp32-accurate
    want_t = orc.activation(orc.update(_tf32_trunc(A.numpy()), _tf32_trunc(Bo), bias.numpy()), True)
    assert rel_fro(host(Cd, N), want_t) <= 2e-5
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (64, 32, 4096), (100, 47, 70001), (602, 256, 9000), (1024, 64, 5000), (128, 172, 33333)])
def test_gemm_tf32_weight_gradient_form(mg, ctx, M, N, K):
    from helpers import TOL_LOWP
    A, B = synth.normal_features(K, M, 141), synth.normal_features(K, N, 142)
    Cd = torch.full((M, N), 3.0, device="cuda")
    mg.gemm(ctx, mg.PREC_TF32, True, False, M, N, K, padded(A, fill=float("nan")), padded(B, fill=float("nan")), Cd)
    want = A.numpy().astype(np.float64).T @ B.numpy().astype(np.float64)
    assert rel_fro(host(Cd), want) <= TOL_LOWP
    want_t = _tf32_trunc(A.numpy()).T @ _tf32_trunc(B.numpy())
    assert rel_fro(host(Cd), want_t) <= 2e-5
    Cd2 = torch.zeros_like(Cd)
    mg.gemm(ctx, mg.PREC_TF32, True, False, M, N, K, padded(A, fill=float("nan")), padded(B, fill=float("nan")), Cd2)
    assert torch.equal(Cd, Cd2)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def _gradients_with_given_relu_masks(go, ref, Ws, X_gpu):
    """The oracle's backward pass with the ReLU masks of the GPU's forward pass (X_gpu[l+1] > 0) in place
    of its own.  A reduced-precision forward pass flips the mask where a pre-activation is within its
    rounding error of zero; each flip changes an O(1) entry of the gradient below it, so whole-iteration
    gradients differ from the fp64 ones by about the square root of the operand rounding error, which no
    dense product can repair.  Given the same masks the products' own error is what remains."""
    L = len(Ws)
    Gout, dWs, dbs = ref["G"], [None] * L, [None] * L
    for l in range(L - 1, -1, -1):
        mask_src = X_gpu[l + 1] if l < L - 1 else ref["Ps"][l]
        dP, dWs[l], dbs[l], dZ = orc.update_bwd(ref["Zs"][l], mask_src, Ws[l].numpy(), Gout, relu=l < L - 1, need_dZ=l > 0)
        if l > 0:
            Gout = orc.aggregate(go, dZ, transposed=True)
    return dWs, dbs


def _bf16_round(a):
    """fp32 values rounded to bf16 (nearest, ties to even), as fp64."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


@pytest.mark.parametrize("M,N,K", TC_SHAPES + [(1000, 256, 1024), (333, 1024, 200)])
@pytest.mark.parametrize("tb", [False, True])
def test_gemm_bf16_forward_forms(mg, ctx, M, N, K, tb):
    """bf16 x bf16 -> fp32 on the tensor cores: within the low-precision bound of the fp64 product, and
    fp32-accurate against the product of the bf16-rounded operands (which an fp32 or TF32 kernel would miss)."""
    from helpers import TOL_LOWP
    A = synth.uniform_tensor((M, K), 231 + M, -1, 1)
    B = synth.uniform_tensor((N, K) if tb else (K, N), 232 + N, -1, 1)
    bias = synth.uniform_tensor((N,), 233, -1, 1)
    Cd = torch.full((M, round4(N) + 4), 3.0, device="cuda")
    epi = mg.make_epilogue(bias=bias.cuda(), relu=True)
    before = mg.ctx_gemm_paths(ctx)["tc_bf16"]
    mg.gemm(ctx, mg.PREC_BF16, False, tb, M, N, K, padded(A, fill=float("nan")), B.cuda().contiguous(), Cd, epi=epi)
    assert mg.ctx_gemm_paths(ctx)["tc_bf16"] == before + 1          # the bf16 kernel served it, not a fallback
    Bo = B.numpy().T if tb else B.numpy()
    want = orc.activation(orc.update(A.numpy(), Bo, bias.numpy()), True)
    assert rel_fro(host(Cd, N), want) <= TOL_LOWP
    assert torch.all(Cd[:, round4(N):] == 3.0)
    want_r = orc.activation(orc.update(_bf16_round(A.numpy()), _bf16_round(Bo), bias.numpy()), True)
    assert rel_fro(host(Cd, N), want_r) <= 2e-5
    assert rel_fro(host(Cd, N), want) > 1e-4                         # and it really is a bf16 product
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (64, 32, 4096), (100, 47, 70001), (602, 256, 9000), (1024, 64, 5000),
                                   (128, 172, 33333), (1024, 1024, 20000)])
def test_gemm_bf16_weight_gradient_form(mg, ctx, M, N, K):
    from helpers import TOL_LOWP
    A, B = synth.normal_features(K, M, 241), synth.normal_features(K, N, 242)
    Cd = torch.full((M, N), 3.0, device="cuda")
    before = mg.ctx_gemm_paths(ctx)["tc_bf16"]
    mg.gemm(ctx, mg.PREC_BF16, True, False, M, N, K, padded(A, fill=float("nan")), padded(B, fill=float("nan")), Cd)
    assert mg.ctx_gemm_paths(ctx)["tc_bf16"] == before + 1
    want = A.numpy().astype(np.float64).T @ B.numpy().astype(np.float64)
    assert rel_fro(host(Cd), want) <= TOL_LOWP
    want_r = _bf16_round(A.numpy()).T @ _bf16_round(B.numpy())
    assert rel_fro(host(Cd), want_r) <= 2e-5
    Cd2 = torch.zeros_like(Cd)
    mg.gemm(ctx, mg.PREC_BF16, True, False, M, N, K, padded(A, fill=float("nan")), padded(B, fill=float("nan")), Cd2)
    assert torch.equal(Cd, Cd2)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("orders", ["auto", "agg", "upd"])
@pytest.mark.parametrize("lp_copies", [True, False])
def test_training_epoch_bf16_within_low_precision_bound(mg, ctx, orders, lp_copies):
    """A whole iteration with bf16 operands in every dense product: with the bf16 companions written by
    the producing kernels and with on-the-fly conversion the results are the same bits, and both are
    within the low-precision bound of the oracle."""
    from helpers import TOL_LOWP
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s, d)
    order = {"auto": mg.ORDER_AUTO, "agg": mg.ORDER_AGG_FIRST, "upd": mg.ORDER_UPD_FIRST}[orders]
    outs = []
    for copies in ([True, False] if lp_copies else [False]):
        tr = GcnTrainer(ctx, gg, wl.dims, mg.PREC_BF16, order=order, lp_copies=copies, row_sparse=0)
        tr.set_params(Ws, bs)
        tr.set_inputs(padded(X), y.cuda(), m.cuda())
        before = mg.ctx_gemm_paths(ctx)
        tr.forward()
        logits = host(tr.X[-1], wl.classes).astype(np.float64)
        X_gpu = [None] + [host(tr.X[l], wl.dims[l]).astype(np.float64) for l in range(1, tr.L + 1)]
        tr.compute_loss(); tr.backward()
        after = mg.ctx_gemm_paths(ctx)
        assert after["tc_bf16"] - before["tc_bf16"] == 3 * tr.L - 1 and after["simt"] == before["simt"] and after["tc_tf32"] == before["tc_tf32"]
        outs.append((logits, [w.cpu().numpy().astype(np.float64) for w in tr.dW], [b.cpu().numpy().astype(np.float64) for b in tr.db]))
    if len(outs) == 2:
        assert np.array_equal(outs[0][0], outs[1][0])
        for a, b in zip(outs[0][1] + outs[0][2], outs[1][1] + outs[1][2]):
            assert np.array_equal(a, b)
    logits, dWs, dbs = outs[0]
    ref = orc.train_epoch(go, X.numpy(), [w.numpy() for w in Ws], [b.numpy() for b in bs], y.numpy(), m.numpy(), None, 1, **ADAM)
    assert rel_fro(logits, ref["logits"]) <= TOL_LOWP
    fw, fb = _gradients_with_given_relu_masks(go, ref, Ws, X_gpu)
    for l in range(len(dWs)):
        print(f"bf16 epoch ({orders}): layer {l} rel. Frobenius error dW {rel_fro(dWs[l], ref['dW'][l]):.2e} db {rel_fro(dbs[l], ref['db'][l]):.2e}"
              f"; with the GPU's ReLU masks given to the oracle: dW {rel_fro(dWs[l], fw[l]):.2e} db {rel_fro(dbs[l], fb[l]):.2e}")
        assert rel_fro(dWs[l], fw[l]) <= TOL_LOWP and rel_fro(dbs[l], fb[l]) <= TOL_LOWP
    assert rel_fro(dWs[-1], ref["dW"][-1]) <= TOL_LOWP            # no ReLU mask below the loss: the plain bound holds
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    gg.close()


def test_bf16_layer_keeps_only_the_bf16_copy_of_the_aggregation(mg, ctx):
    """SAVED_LP_ONLY: the forward leaves the fp32 `saved` alone (both products read the bf16 copy), the
    results are the bits of the run that writes both, and the flag is refused where something reads fp32."""
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    gg = mg.graph_create(ctx, wl.n, s, d)
    outs = []
    for only in (True, False):
        tr = GcnTrainer(ctx, gg, wl.dims, mg.PREC_BF16, order=mg.ORDER_AGG_FIRST, row_sparse=0, saved_lp_only=only)
        tr.set_params(Ws, bs)
        tr.set_inputs(padded(X), y.cuda(), m.cuda())
        for sv in tr.saved:
            sv.fill_(7.0)
        tr.forward()
        for l, sv in enumerate(tr.saved):
            assert bool(tr.descs[l].flags & mg.LAYER_SAVED_LP_ONLY) == only
            assert bool(torch.all(sv == 7.0)) == only
        logits = tr.X[-1].clone()
        tr.compute_loss(); tr.backward()
        outs.append([logits] + [w.clone() for w in tr.dW] + [b.clone() for b in tr.db])
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    # refused: fp32 products, and a row-sparse backward (which gathers fp32 rows of `saved`)
    tr = GcnTrainer(ctx, gg, wl.dims, mg.PREC_BF16, order=mg.ORDER_AGG_FIRST, row_sparse=0)
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    dsc = tr.descs[0]
    for change in ("precision", "row_mask"):
        keep = (dsc.precision, dsc.gout_row_mask)
        dsc.flags |= mg.LAYER_SAVED_LP_ONLY
        if change == "precision":
            dsc.precision = mg.PREC_TF32
        else:
            dsc.gout_row_mask = tr.train_mask.data_ptr()
        with pytest.raises(mg.MixgcnError) as e:
            mg.layer_fwd(ctx, gg, dsc, tr.X[0], tr.W[0], tr.b[0], None, tr.saved[0], tr.X[1])
        assert e.value.status == mg.EINVAL
        dsc.precision, dsc.gout_row_mask = keep
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    gg.close()


PAIR_SHAPES = [(4096, 512, 512), (5000, 1024, 520), (4100, 600, 1000), (8191, 777, 513)]   # M, N, K: ragged in every dimension


@pytest.mark.parametrize("M,N,K", PAIR_SHAPES)
@pytest.mark.parametrize("prec", ["tf32", "bf16"])
@pytest.mark.parametrize("tb", [False, True])
def test_gemm_on_cta_pairs(mg, ctx, M, N, K, prec, tb):
    """Wide, deep K-major products run on pairs of CTAs (one 256 x 256 tile per pair): same checks as the
    single-CTA kernels, and the single-CTA kernel must agree with the pair kernel to fp32 accuracy."""
    from helpers import TOL_LOWP
    P = mg.PRECISIONS[prec]
    rnd = _tf32_trunc if prec == "tf32" else _bf16_round
    A = synth.uniform_tensor((M, K), 331 + M, -1, 1)
    B = synth.uniform_tensor((N, K) if tb else (K, N), 332 + N, -1, 1)
    bias = synth.uniform_tensor((N,), 333, -1, 1)
    Cd = torch.full((M, round4(N) + 4), 3.0, device="cuda")
    epi = mg.make_epilogue(bias=bias.cuda(), relu=True)
    before = mg.ctx_gemm_paths(ctx)["cta_pairs"]
    mg.gemm(ctx, P, False, tb, M, N, K, padded(A, fill=float("nan")), B.cuda().contiguous(), Cd, epi=epi)
    assert mg.ctx_gemm_paths(ctx)["cta_pairs"] == before + 1
    Bo = B.numpy().T if tb else B.numpy()
    assert rel_fro(host(Cd, N), orc.activation(orc.update(A.numpy(), Bo, bias.numpy()), True)) <= TOL_LOWP
    assert rel_fro(host(Cd, N), orc.activation(orc.update(rnd(A.numpy()), rnd(Bo), bias.numpy()), True)) <= 2e-5
    assert torch.all(Cd[:, round4(N):] == 3.0)
    mg.ctx_set_option(ctx, mg.OPT_GEMM_CTA_PAIRS, 0)
    try:
        C1 = torch.full_like(Cd, 3.0)
        mg.gemm(ctx, P, False, tb, M, N, K, padded(A, fill=float("nan")), B.cuda().contiguous(), C1, epi=epi)
        assert mg.ctx_gemm_paths(ctx)["cta_pairs"] == before + 1
    finally:
        mg.ctx_set_option(ctx, mg.OPT_GEMM_CTA_PAIRS, 1)
    assert rel_fro(host(Cd, N), host(C1, N)) <= 2e-6
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("M,N,K", [(512, 512, 4096), (1024, 1024, 20000), (600, 777, 9001), (520, 1000, 33333)])
@pytest.mark.parametrize("prec", ["tf32", "bf16"])
def test_weight_gradient_on_cta_pairs(mg, ctx, M, N, K, prec):
    from helpers import TOL_LOWP
    P = mg.PRECISIONS[prec]
    rnd = _tf32_trunc if prec == "tf32" else _bf16_round
    A, B = synth.normal_features(K, M, 351), synth.normal_features(K, N, 352)
    Cd = torch.full((M, round4(N)), 3.0, device="cuda")
    before = mg.ctx_gemm_paths(ctx)["cta_pairs"]
    mg.gemm(ctx, P, True, False, M, N, K, padded(A, fill=float("nan")), padded(B, fill=float("nan")), Cd)
    assert mg.ctx_gemm_paths(ctx)["cta_pairs"] == before + 1
    assert rel_fro(host(Cd, N), A.numpy().astype(np.float64).T @ B.numpy().astype(np.float64)) <= TOL_LOWP
    assert rel_fro(host(Cd, N), rnd(A.numpy()).T @ rnd(B.numpy())) <= 2e-5
    C2 = torch.zeros_like(Cd)
    mg.gemm(ctx, P, True, False, M, N, K, padded(A, fill=float("nan")), padded(B, fill=float("nan")), C2)
    assert torch.equal(Cd[:, :N], C2[:, :N])                               # fixed-order reduction: reproducible bits
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_weight_gradient_on_cta_pairs_without_a_split(mg, ctx):
    """K too short to split: the pair kernel writes the final tile itself and applies the epilogue."""
    M, N, K = 2048, 2048, 4096
    A, B = synth.normal_features(K, M, 361), synth.normal_features(K, N, 362)
    bias = synth.uniform_tensor((N,), 363, -1, 1)
    Cd = torch.zeros(M, N, device="cuda")
    before = mg.ctx_gemm_paths(ctx)["cta_pairs"]
    mg.gemm(ctx, mg.PREC_BF16, True, False, M, N, K, A.cuda(), B.cuda(), Cd, epi=mg.make_epilogue(bias=bias.cuda(), relu=True))
    assert mg.ctx_gemm_paths(ctx)["cta_pairs"] == before + 1
    want = np.maximum(_bf16_round(A.numpy()).T @ _bf16_round(B.numpy()) + bias.numpy().astype(np.float64), 0.0)
    assert rel_fro(host(Cd), want) <= 2e-5
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("with_copies", [True, False])
def test_chunked_pipeline_with_bf16_products(mg, ctx, with_copies):
    """Row chunks on two streams with BF16 products: with the caller's bf16 copy of `saved` each chunk's
    update reads its rows of it; without, the chunks fall back to TF32 (two streams cannot share the
    conversion workspace).  Output within the low-precision bound either way."""
    from helpers import TOL_LOWP
    go, gg = build_both(mg, ctx, "hub")
    n, d_in, d_out = go.n, 64, 48
    X = synth.uniform_tensor((n, d_in), 371, -1, 1); W = synth.glorot_uniform(d_in, d_out, 372)
    b = synth.uniform_tensor((d_out,), 373, -0.2, 0.2)
    desc = mg.layer_desc(d_in, d_out, round4(d_in), round4(d_out), round4(d_in), mg.ORDER_AGG_FIRST, mg.PREC_BF16, mg.LAYER_RELU,
                         1.0, 1.0, 3)
    saved = torch.zeros(n, round4(d_in), device="cuda"); Xout = torch.zeros(n, round4(d_out), device="cuda")
    keep = []
    if with_copies:
        s_lp = torch.zeros(n, 64, dtype=torch.bfloat16, device="cuda"); o_lp = torch.zeros(n, 48, dtype=torch.bfloat16, device="cuda")
        keep = [s_lp, o_lp]
        desc.saved_lp, desc.ld_saved_lp = s_lp.data_ptr(), 64
        desc.x_out_lp, desc.ld_out_lp = o_lp.data_ptr(), 48
        desc.ld_in_lp = 64
    before = mg.ctx_gemm_paths(ctx)
    mg.layer_fwd(ctx, gg, desc, padded(X), W.cuda(), b.cuda(), None, saved, Xout)
    torch.cuda.synchronize()
    after = mg.ctx_gemm_paths(ctx)
    key = "tc_bf16" if with_copies else "tc_tf32"
    assert after[key] - before[key] == 3
    Z = orc.aggregate(go, X.numpy())
    want = orc.activation(orc.update(Z, W.numpy(), b.numpy()), True)
    assert rel_fro(host(Xout, d_out), want) <= TOL_LOWP
    assert rel_fro(host(saved, d_in), Z) <= TOL_FP32
    if with_copies:
        assert rel_fro(keep[0].float().cpu().numpy(), _bf16_round(host(saved, d_in))) == 0.0          # the copy is bf16(saved), bit for bit
        assert rel_fro(keep[1].float().cpu().numpy(), _bf16_round(host(Xout, d_out))) == 0.0
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_gemm_on_cta_pairs_with_gate_and_dropout(mg, ctx):
    """The per-element epilogue terms (gate by another tensor's sign, dropout mask) on the pair kernel."""
    M, N, K = 4200, 520, 512
    A = synth.uniform_tensor((M, K), 341, -1, 1); B = synth.uniform_tensor((K, N), 342, -1, 1)
    gate = synth.uniform_tensor((M, N), 343, -1, 1)
    drop = (synth.uniform_tensor((M, N), 344, 0, 1) < 0.7).to(torch.uint8)
    Cd = torch.zeros(M, round4(N), device="cuda")
    epi = mg.make_epilogue(drop_mask=drop.cuda(), keep_scale=1.25, gate=padded(gate), gate_scale=0.5)
    before = mg.ctx_gemm_paths(ctx)["cta_pairs"]
    mg.gemm(ctx, mg.PREC_BF16, False, False, M, N, K, padded(A), B.cuda(), Cd, epi=epi)
    assert mg.ctx_gemm_paths(ctx)["cta_pairs"] == before + 1
    want = _bf16_round(A.numpy()) @ _bf16_round(B.numpy())
    want = np.where(drop.numpy() != 0, want * 1.25, 0.0)
    want = np.where(gate.numpy() > 0, want * 0.5, 0.0)
    assert rel_fro(host(Cd, N), want) <= 2e-5
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("prec", ["tf32", "bf16"])
def test_bounded_wait_runs_out_and_the_context_stays_usable(mg, ctx, prec):
    """Failure detection without a fault: a test hook makes the TMA producer of the tensor-core kernel
    leave one stage unfilled and shortens the wait limit; the kernel must give up, report through the
    status word (MIXGCN_ETIMEOUT), free its tensor memory and return, and the next product on the same
    context must be right."""
    from helpers import TOL_LOWP
    P = mg.PRECISIONS[prec]
    M, N, K = 128, 128, 64
    A = synth.uniform_tensor((M, K), 801, -1, 1); B = synth.uniform_tensor((K, N), 802, -1, 1)
    Cd = torch.zeros(M, N, device="cuda")
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    mg.ctx_set_option(ctx, mg.OPT_DEBUG_WAIT_LIMIT, 2000)
    mg.ctx_set_option(ctx, mg.OPT_DEBUG_DROP_LOAD, 1)
    try:
        mg.gemm(ctx, P, False, False, M, N, K, A.cuda(), B.cuda(), Cd)
        with pytest.raises(mg.MixgcnError) as e:
            mg.ctx_poll_status(ctx)
        assert e.value.status == mg.ETIMEOUT
    finally:
        mg.ctx_set_option(ctx, mg.OPT_DEBUG_DROP_LOAD, 0)
        mg.ctx_set_option(ctx, mg.OPT_DEBUG_WAIT_LIMIT, 0)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0          # cleared by the read
    for _ in range(3):                                                  # tensor memory was freed: later launches get theirs
        Cd.fill_(7.0)
        mg.gemm(ctx, P, False, False, M, N, K, A.cuda(), B.cuda(), Cd)
        assert rel_fro(host(Cd), A.numpy().astype(np.float64) @ B.numpy().astype(np.float64)) <= TOL_LOWP
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_colsum_rejects_layouts_it_cannot_read(mg, ctx):
    X = torch.zeros(64, 44, device="cuda"); out = torch.zeros(41, device="cuda")
    bad_ld = X[:, :41].contiguous()                 # ld = 41: not a multiple of 4
    rc = mg.lib.mixgcn_colsum(ctx.h, mg.C.c_int64(64), mg.C.c_int32(41), mg.C.c_void_p(bad_ld.data_ptr()), mg.C.c_int64(41),
                              mg.C.c_void_p(out.data_ptr()), None)
    assert rc == mg.EINVAL
    rc = mg.lib.mixgcn_colsum(ctx.h, mg.C.c_int64(63), mg.C.c_int32(40), mg.C.c_void_p(X.data_ptr() + 4), mg.C.c_int64(44),
                              mg.C.c_void_p(out.data_ptr()), None)
    assert rc == mg.EINVAL                          # not 16-byte aligned
    X[:, :41] = 1.0
    mg.colsum(ctx, X, out, 41)
    assert torch.all(out == 64.0)


def test_training_epoch_tf32_within_low_precision_bound(mg, ctx):
    from helpers import TOL_LOWP
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s, d)
    tr = GcnTrainer(ctx, gg, wl.dims, mg.PREC_TF32)
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    tr.forward()
    logits = host(tr.X[-1], wl.classes).copy()
    X_gpu = [None] + [host(tr.X[l], wl.dims[l]).astype(np.float64) for l in range(1, tr.L + 1)]
    tr.compute_loss(); tr.backward()
    ref = orc.train_epoch(go, X.numpy(), [w.numpy() for w in Ws], [b.numpy() for b in bs], y.numpy(), m.numpy(), None, 1, **ADAM)
    assert rel_fro(logits, ref["logits"]) <= TOL_LOWP
    assert abs(tr.loss.item() - ref["loss"]) <= TOL_LOWP * abs(ref["loss"])
    # Below a ReLU the whole-iteration gradient also carries the mask flips of the reduced-precision
    # forward pass (see _gradients_with_given_relu_masks): the stated relative bound is asserted with the
    # masks given, and on the last layer as it stands; against the plain oracle every layer is held to
    # the inner-product bound (the error of sum_i a_i b_i is at most u * sum_i |a_i| |b_i|) and its
    # relative error is printed.
    fw, fb = _gradients_with_given_relu_masks(go, ref, Ws, X_gpu)
    for l in range(tr.L):
        print(f"tf32 epoch: layer {l} with the GPU's ReLU masks given to the oracle: dW {rel_fro(tr.dW[l].cpu().numpy(), fw[l]):.2e} "
              f"db {rel_fro(tr.db[l].cpu().numpy(), fb[l]):.2e}")
        assert rel_fro(tr.dW[l].cpu().numpy(), fw[l]) <= TOL_LOWP and rel_fro(tr.db[l].cpu().numpy(), fb[l]) <= TOL_LOWP
    assert rel_fro(tr.dW[-1].cpu().numpy(), ref["dW"][-1]) <= TOL_LOWP
    Gout = ref["G"]
    for l in range(tr.L - 1, -1, -1):
        dP, dW, db, dZ = orc.update_bwd(ref["Zs"][l], ref["Ps"][l], Ws[l].numpy(), Gout, relu=l < tr.L - 1, need_dZ=l > 0)
        scale_w = np.linalg.norm(np.abs(ref["Zs"][l]).T @ np.abs(dP))
        scale_b = np.linalg.norm(np.abs(dP).sum(axis=0))
        assert np.linalg.norm(tr.dW[l].cpu().numpy() - ref["dW"][l]) <= TOL_LOWP * scale_w
        assert np.linalg.norm(tr.db[l].cpu().numpy() - ref["db"][l]) <= TOL_LOWP * scale_b
        print(f"tf32 epoch: layer {l} rel. Frobenius error dW {rel_fro(tr.dW[l].cpu().numpy(), ref['dW'][l]):.2e} "
              f"db {rel_fro(tr.db[l].cpu().numpy(), ref['db'][l]):.2e}")
        if l > 0:
            Gout = orc.aggregate(go, dZ, transposed=True)


# --------------------------------------------------------------------------- row-sparse backward

@pytest.mark.parametrize("name", ["messy-directed", "hub"])
@pytest.mark.parametrize("order", ["agg", "upd"])
@pytest.mark.parametrize("give_count", [True, False])
def test_layer_bwd_row_sparse_matches_dense_definition(mg, ctx, name, order, give_count):
    """G_out with a few non-zero rows: the row-sparse path (compacted products when the count is
    given, masked aggregation otherwise) must give the dense definition's gradients."""
    go, gg = build_both(mg, ctx, name)
    n, d_in, d_out = go.n, 40, 24
    o = mg.ORDER_AGG_FIRST if order == "agg" else mg.ORDER_UPD_FIRST
    X = synth.uniform_tensor((n, d_in), 301, -1, 1)
    W = synth.glorot_uniform(d_in, d_out, 302)
    b = synth.uniform_tensor((d_out,), 303, -0.2, 0.2)
    rows = synth.bernoulli_mask(n, 0.05, 304)
    rows[0] = 1                                                       # the hub's own row is among them
    Gout = synth.uniform_tensor((n, d_out), 305, -1, 1) * rows[:, None].float()
    desc = mg.layer_desc(d_in, d_out, round4(d_in), round4(d_out), round4(max(d_in, d_out)), o, mg.PREC_FP32,
                         mg.LAYER_RELU | mg.LAYER_GATE_GIN)
    Xd, Wd, bd = padded(X), W.cuda(), b.cuda()
    saved = torch.zeros(n, round4(max(d_in, d_out)), device="cuda")
    Xout = torch.zeros(n, round4(d_out), device="cuda")
    mg.layer_fwd(ctx, gg, desc, Xd, Wd, bd, None, saved, Xout)
    rows_d = rows.cuda()
    gin_mask = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
    desc.gout_row_mask = rows_d.data_ptr()
    desc.gout_row_count = int(rows.sum()) if give_count else 0
    desc.gin_row_mask = gin_mask.data_ptr()
    Gd = padded(Gout)
    Gin = torch.full((n, round4(d_in)), 5.0, device="cuda")
    dW = torch.zeros(d_in, d_out, device="cuda"); db = torch.zeros(d_out, device="cuda")
    mg.layer_bwd(ctx, gg, desc, Xd, saved, Xout, None, Wd, Gd, Gin, dW, db)
    Z = orc.aggregate(go, X.numpy())
    Pp = orc.update(Z, W.numpy(), b.numpy())
    _, dWo, dbo, dZo = orc.update_bwd(Z, Pp, W.numpy(), Gout.numpy(), True)
    want_gin = orc.aggregate(go, dZo, transposed=True) * (X.numpy() > 0)
    assert rel_fro(host(dW), dWo) <= TOL_FP32 and rel_fro(db.cpu().numpy(), dbo) <= TOL_FP32
    assert rel_fro(host(Gin, d_in), want_gin) <= TOL_FP32
    m = gin_mask.cpu().numpy()
    assert set(np.unique(m)) <= {0, 1}
    nonzero_rows = np.abs(orc.aggregate(go, dZo, transposed=True)).sum(axis=1) > 0
    assert np.all(m[nonzero_rows] == 1)                              # the reported mask covers every non-zero row
    assert np.all(host(Gin, d_in)[m == 0] == 0)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_row_sparse_wrong_count_is_reported_not_a_fault(mg, ctx):
    go, gg = build_both(mg, ctx, "messy-sym")
    n, d = go.n, 8
    desc = mg.layer_desc(d, d, 8, 8, 8, mg.ORDER_AGG_FIRST, mg.PREC_FP32, mg.LAYER_FIRST)
    rows = torch.zeros(n, dtype=torch.uint8, device="cuda"); rows[:10] = 1
    desc.gout_row_mask = rows.data_ptr(); desc.gout_row_count = 3      # wrong on purpose (host-side mistake)
    X = torch.zeros(n, 8, device="cuda"); sv = torch.zeros(n, 8, device="cuda"); W = torch.zeros(d, d, device="cuda")
    G = torch.zeros(n, 8, device="cuda"); dW = torch.zeros(d, d, device="cuda")
    mg.layer_bwd(ctx, gg, desc, X, sv, X, None, W, G, None, dW, None)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 4


@pytest.mark.parametrize("levels", [1, 2])
@pytest.mark.parametrize("row_plans", [True, False])
def test_training_epoch_row_sparse_matches_oracle(mg, ctx, levels, row_plans):
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    m = synth.bernoulli_mask(wl.n, 0.03, 77)                           # few train nodes
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s, d)
    dims = (64, 32, 16, 8)                                             # three layers so that two levels exist
    Ws = [synth.glorot_uniform(dims[i], dims[i + 1], 400 + i) for i in range(3)]
    bs = [synth.uniform_tensor((dims[i + 1],), 410 + i, -0.1, 0.1) for i in range(3)]
    tr = GcnTrainer(ctx, gg, dims, mg.PREC_FP32, order=mg.ORDER_AGG_FIRST, row_sparse=levels, row_plans=row_plans)
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    assert tr.row_sparse_levels == levels
    assert all((p is not None) == (row_plans and l >= 3 - levels) for l, p in enumerate(tr.row_plans))
    tr.forward(); tr.compute_loss(); tr.backward()
    ref = orc.train_epoch(go, X.numpy(), [w.numpy() for w in Ws], [b.numpy() for b in bs], y.numpy(), m.numpy(), None, 1, **ADAM)
    assert abs(tr.loss.item() - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    for l in range(3):
        assert rel_fro(tr.dW[l].cpu().numpy(), ref["dW"][l]) <= TOL_FP32
        assert rel_fro(tr.db[l].cpu().numpy(), ref["db"][l]) <= TOL_FP32
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_second_level_row_set_is_counted_and_compacted(mg, ctx):
    """Very few train nodes: the row mask reported by the top layer's backward is small enough for the
    layer below to run its dense products on the compacted rows (count taken by mixgcn_count_rows)."""
    from paper_2501_01951_b200.train import GcnTrainer
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    m = torch.zeros(wl.n, dtype=torch.uint8)
    deg = np.bincount(np.concatenate([s.numpy(), d.numpy()]), minlength=wl.n)
    m[torch.as_tensor(np.nonzero((deg > 0) & (deg <= 3))[0][:6])] = 1        # six low-degree train nodes
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, wl.n, s, d)
    dims = (64, 32, 16, 8)
    Ws = [synth.glorot_uniform(dims[i], dims[i + 1], 400 + i) for i in range(3)]
    bs = [synth.uniform_tensor((dims[i + 1],), 410 + i, -0.1, 0.1) for i in range(3)]
    tr = GcnTrainer(ctx, gg, dims, mg.PREC_FP32, order=mg.ORDER_AGG_FIRST, row_sparse=2, row_plans=False)
    tr.set_params(Ws, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    ref = orc.train_epoch(go, X.numpy(), [w.numpy() for w in Ws], [b.numpy() for b in bs], y.numpy(), m.numpy(), None, 1, **ADAM)
    for _ in range(2):                                                   # second pass reuses the stored count
        tr.forward(); tr.compute_loss(); tr.backward()
        cnt = tr.descs[1].gout_row_count
        assert cnt == int(tr.row_masks[2].sum().item()) == mg.count_rows(ctx, tr.row_masks[2])
        assert 0 < cnt * 4 < wl.n                                        # the compacted path was taken
        nonzero = np.abs(orc.aggregate(go, orc.update_bwd(ref["Zs"][2], ref["Ps"][2], Ws[2].numpy(), ref["G"], relu=False)[3],
                                       transposed=True)).sum(axis=1) > 0
        assert np.all(tr.row_masks[2].cpu().numpy()[nonzero] == 1)
        for l in range(3):
            assert rel_fro(tr.dW[l].cpu().numpy(), ref["dW"][l]) <= TOL_FP32
            assert rel_fro(tr.db[l].cpu().numpy(), ref["db"][l]) <= TOL_FP32
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("name", ["messy-sym", "messy-directed", "hub"])
@pytest.mark.parametrize("norm", ["row", "none"])
def test_graph_aggregator_modes(mg, ctx, name, norm):
    """Row-mean and plain-sum values: stored values bit-exact against the oracle's fp32 recipe in both
    orientations, aggregation in both orientations within the fp32 tolerance."""
    n, s, d, sym = GRAPHS[name]()
    flags_o = orc.ADD_SELF_LOOPS | (orc.SYMMETRISE if sym else 0)
    flags_g = mg.GRAPH_ADD_SELF_LOOPS | (mg.GRAPH_SYMMETRISE if sym else 0) | (mg.GRAPH_NORM_ROW if norm == "row" else mg.GRAPH_NORM_NONE)
    go = orc.graph_build(n, s, d, flags_o, norm=norm)
    gg = mg.graph_create(ctx, n, i32(s), i32(d), flags_g)
    ex, ext = mg.graph_export(gg), mg.graph_export(gg, transposed=True)
    assert np.array_equal(ex["rowptr"].numpy(), go.rowptr) and np.array_equal(ex["col"].numpy(), go.col)
    assert ex["val"].numpy().tobytes() == go.val32.tobytes()
    assert np.array_equal(ext["rowptr"].numpy(), go.rowptr_t) and np.array_equal(ext["col"].numpy(), go.col_t)
    assert ext["val"].numpy().tobytes() == go.val32[go.src_index_t].tobytes()
    w = 36
    Y = synth.uniform_tensor((n, w), 801, -1, 1)
    Z = torch.zeros(n, round4(w), device="cuda")
    for tr_ in (False, True):
        mg.spmm(ctx, gg, padded(Y), Z, w, transposed=tr_)
        assert rel_fro(host(Z, w), orc.aggregate(go, Y.numpy(), transposed=tr_)) <= TOL_FP32
    with pytest.raises(mg.MixgcnError):
        mg.graph_create(ctx, n, i32(s), i32(d), mg.GRAPH_NORM_ROW | mg.GRAPH_NORM_NONE)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("name", ["messy-directed", "hub"])
@pytest.mark.parametrize("transposed", [False, True])
def test_spmm_residual_epilogue(mg, ctx, name, transposed):
    """Z = gate(relu?(s * R + A_hat Y + bias)): the residual term comes first, then bias and gate."""
    go, gg = build_both(mg, ctx, name)
    n, w = go.n, 44
    Y = synth.uniform_tensor((n, w), 701, -1, 1)
    R = synth.uniform_tensor((n, w), 702, -1, 1)
    b = synth.uniform_tensor((w,), 703, -0.5, 0.5)
    gate = synth.uniform_tensor((n, w), 704, -1, 1)
    Yd, Rd, gd = padded(Y), padded(R), padded(gate)
    Z = torch.zeros(n, round4(w), device="cuda")
    mg.spmm(ctx, gg, Yd, Z, w, transposed=transposed, epi=mg.make_epilogue(bias=b.cuda(), residual=Rd, residual_scale=1.25,
                                                                              gate=gd, gate_scale=2.0))
    want = (1.25 * R.numpy() + orc.aggregate(go, Y.numpy(), transposed=transposed) + b.numpy()) * (gate.numpy() > 0) * 2.0
    assert rel_fro(host(Z, w), want) <= TOL_FP32
    # the self term with the input itself as residual: (s I + A_hat) Y
    mg.spmm(ctx, gg, Yd, Z, w, transposed=transposed, epi=mg.make_epilogue(residual=Yd, residual_scale=0.5))
    assert rel_fro(host(Z, w), 0.5 * Y.numpy() + orc.aggregate(go, Y.numpy(), transposed=transposed)) <= TOL_FP32
    with pytest.raises(mg.MixgcnError):
        mg.spmm(ctx, gg, Yd, Z, w, epi=mg.make_epilogue(residual=Z))                     # residual must not be the output
    with pytest.raises(mg.MixgcnError):
        mg.gemm(ctx, mg.PREC_FP32, False, False, 8, 8, 8, torch.zeros(8, 8, device="cuda"), torch.zeros(8, 8, device="cuda"),
                torch.zeros(8, 8, device="cuda"), epi=mg.make_epilogue(residual=torch.zeros(8, 8, device="cuda")))
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_spmm_column_slices_do_not_change_the_result(mg):
    """Feature-column slicing (the p:q-1 ranges of Algorithm 2) is a schedule, not arithmetic."""
    c2 = mg.ctx_create(0)
    n, s, d, sym = GRAPHS["hub"]()
    gg = mg.graph_create(c2, n, i32(s), i32(d))
    X = padded(synth.uniform_tensor((n, 172), 501, -1, 1))
    Z0 = torch.zeros_like(X); Z1 = torch.zeros_like(X); Z2 = torch.zeros_like(X)
    mg.spmm(c2, gg, X, Z0, 172)
    mg.ctx_set_option(c2, mg.OPT_SPMM_SLICE_COLS, 32)
    mg.spmm(c2, gg, X, Z1, 172)
    mg.ctx_set_option(c2, mg.OPT_SPMM_SLICE_COLS, 100)
    mg.spmm(c2, gg, X, Z2, 172)
    assert torch.equal(Z0, Z1) and torch.equal(Z0, Z2)
    with pytest.raises(mg.MixgcnError):
        mg.ctx_set_option(c2, mg.OPT_SPMM_SLICE_COLS, 6)
    with pytest.raises(mg.MixgcnError):
        mg.ctx_set_option(c2, 99, 1)
    gg.close(); c2.close()


# --------------------------------------------------------------------------- more tensor-core paths

def test_gemm_tf32_generic_epilogue_and_wide_bias(mg, ctx):
    """The tensor-core kernel's per-element epilogue (dropout mask, gate) and the bias path for N > 1024."""
    from helpers import TOL_LOWP
    M, N, K = 333, 70, 96
    A, B = synth.uniform_tensor((M, K), 601, -1, 1), synth.uniform_tensor((K, N), 602, -1, 1)
    bias = synth.uniform_tensor((N,), 603, -1, 1)
    drop = (synth.uniform_tensor((M, N), 604, 0, 1) < 0.5).to(torch.uint8)
    gate = synth.uniform_tensor((M, N), 605, -1, 1)
    Cd = torch.zeros(M, round4(N), device="cuda")
    epi = mg.make_epilogue(bias=bias.cuda(), relu=True, drop_mask=drop.cuda(), keep_scale=2.0, gate=padded(gate), gate_scale=0.5)
    mg.gemm(ctx, mg.PREC_TF32, False, False, M, N, K, padded(A), padded(B), Cd, epi=epi)
    want = orc.activation(orc.update(A.numpy(), B.numpy(), bias.numpy()), True, drop.numpy(), 2.0) * np.where(gate.numpy() > 0, 0.5, 0.0)
    assert rel_fro(host(Cd, N), want) <= TOL_LOWP
    M, N, K = 200, 1100, 64
    A, B = synth.uniform_tensor((M, K), 611, -1, 1), synth.uniform_tensor((K, N), 612, -1, 1)
    bias = synth.uniform_tensor((N,), 613, -1, 1)
    Cd = torch.zeros(M, round4(N), device="cuda")
    mg.gemm(ctx, mg.PREC_TF32, False, False, M, N, K, padded(A), padded(B), Cd, epi=mg.make_epilogue(bias=bias.cuda(), relu=True))
    assert rel_fro(host(Cd, N), orc.activation(orc.update(A.numpy(), B.numpy(), bias.numpy()), True)) <= TOL_LOWP
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("order", ["agg", "upd"])
def test_layer_tf32_with_dropout_both_orders(mg, ctx, order):
    from helpers import TOL_LOWP
    go, gg = build_both(mg, ctx, "messy-directed")
    n, d_in, d_out = go.n, 48, 40
    o = mg.ORDER_AGG_FIRST if order == "agg" else mg.ORDER_UPD_FIRST
    X = synth.uniform_tensor((n, d_in), 621, -1, 1)
    W = synth.glorot_uniform(d_in, d_out, 622)
    b = synth.uniform_tensor((d_out,), 623, -0.2, 0.2)
    Gout = synth.uniform_tensor((n, d_out), 624, -1, 1)
    drop = (synth.uniform_tensor((n, d_out), 625, 0, 1) < 0.6).to(torch.uint8)
    ks = 1 / 0.6
    desc = mg.layer_desc(d_in, d_out, round4(d_in), round4(d_out), round4(max(d_in, d_out)), o, mg.PREC_TF32,
                         mg.LAYER_RELU | mg.LAYER_GATE_GIN, ks, 1.0, 0)
    Xd, Wd, bd, dd = padded(X), W.cuda(), b.cuda(), drop.cuda()
    saved = torch.zeros(n, round4(max(d_in, d_out)), device="cuda"); Xout = torch.zeros(n, round4(d_out), device="cuda")
    mg.layer_fwd(ctx, gg, desc, Xd, Wd, bd, dd, saved, Xout)
    Z = orc.aggregate(go, X.numpy()); Pp = orc.update(Z, W.numpy(), b.numpy())
    assert rel_fro(host(Xout, d_out), orc.activation(Pp, True, drop.numpy(), ks)) <= TOL_LOWP
    Gd = padded(Gout); Gin = torch.zeros(n, round4(d_in), device="cuda")
    dW = torch.zeros(d_in, d_out, device="cuda"); db = torch.zeros(d_out, device="cuda")
    mg.layer_bwd(ctx, gg, desc, Xd, saved, Xout, dd, Wd, Gd, Gin, dW, db)
    dP, dWo, dbo, dZo = orc.update_bwd(Z, Pp, W.numpy(), Gout.numpy(), True, drop.numpy(), ks)
    assert np.linalg.norm(host(dW) - dWo) <= TOL_LOWP * np.linalg.norm(np.abs(Z).T @ np.abs(dP))
    assert rel_fro(db.cpu().numpy(), dbo) <= TOL_LOWP
    want_gin = orc.aggregate(go, dZo, transposed=True) * (X.numpy() > 0)
    assert rel_fro(host(Gin, d_in), want_gin) <= TOL_LOWP
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("with_pred", [False, True])
def test_train_step_host_row_sparse_matches_oracle(mg, ctx, with_pred):
    """Few train nodes: the host-buffer step takes the row-sparse backward; without `pred` it also
    restricts the last layer and the loss to the train rows."""
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    m = synth.bernoulli_mask(wl.n, 0.02, 88)
    gg = mg.graph_create(ctx, wl.n, s, d)
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    W = [w.clone() for w in Ws]; b = [x.clone() for x in bs]
    z = lambda lst: [torch.zeros_like(x) for x in lst]
    mW, vW, mb, vb = z(W), z(W), z(b), z(b)
    pred = torch.full((wl.n,), -7, dtype=torch.int32) if with_pred else None
    loss = mg.train_step_host(ctx, gg, wl.dims, mg.PREC_FP32, X, y, m, W, b, mW, vW, mb, vb, 1, **ADAM, pred=pred)
    if with_pred:
        p = pred.numpy()
        assert p.min() >= 0 and p.max() < wl.classes                 # every node has a prediction
    ref = orc.train_epoch(go, X.numpy(), [w.numpy() for w in Ws], [x.numpy() for x in bs], y.numpy(), m.numpy(), None, 1, **ADAM)
    assert abs(loss - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    for l in range(len(W)):
        # first moments are (1 - beta1) * gradient after one step: an exact view of dW, db
        assert rel_fro(mW[l].numpy() / (1 - ADAM["beta1"]), ref["dW"][l]) <= 2e-5
        assert rel_fro(mb[l].numpy() / (1 - ADAM["beta1"]), ref["db"][l]) <= 2e-5
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_train_step_host_reuses_and_rebuilds_its_row_plans(mg):
    """Same graph and mask: the second call reuses the plans of the first.  A changed mask, or another
    graph, must rebuild them -- every call matches the oracle for its own inputs."""
    c2 = mg.ctx_create(0)
    wl, s, d, X, y, m, Ws, bs = _tiny_problem()
    masks = [synth.bernoulli_mask(wl.n, 0.02, 88), synth.bernoulli_mask(wl.n, 0.02, 88), synth.bernoulli_mask(wl.n, 0.03, 89)]
    gg = mg.graph_create(c2, wl.n, s, d)
    go = orc.graph_build(wl.n, s.numpy(), d.numpy())
    s2, d2 = synth.rmat_graph(wl.n, wl.undirected_edges, 999)
    graphs = [(gg, go)] * 3 + [(mg.graph_create(c2, wl.n, s2, d2), orc.graph_build(wl.n, s2.numpy(), d2.numpy()))]
    masks.append(masks[2])
    for (g_gpu, g_orc), mask in zip(graphs, masks):
        W = [w.clone() for w in Ws]; b = [x.clone() for x in bs]
        z = lambda lst: [torch.zeros_like(x) for x in lst]
        mW, vW, mb, vb = z(W), z(W), z(b), z(b)
        loss = mg.train_step_host(c2, g_gpu, wl.dims, mg.PREC_FP32, X, y, mask, W, b, mW, vW, mb, vb, 1, **ADAM)
        ref = orc.train_epoch(g_orc, X.numpy(), [w.numpy() for w in Ws], [x.numpy() for x in bs], y.numpy(), mask.numpy(), None, 1, **ADAM)
        assert abs(loss - ref["loss"]) <= 1e-5 * abs(ref["loss"])
        for l in range(len(W)):
            assert rel_fro(mW[l].numpy() / (1 - ADAM["beta1"]), ref["dW"][l]) <= 2e-5
            assert rel_fro(mb[l].numpy() / (1 - ADAM["beta1"]), ref["db"][l]) <= 2e-5
    assert mg.ctx_poll_status(c2, raise_on_error=False) == 0
    c2.close()


def test_graph_size_limits_are_checked_on_the_host(mg, ctx):
    e = i32([])
    with pytest.raises(mg.MixgcnError) as ex:
        mg.graph_create(ctx, 2**31 - 1, e, e)
    assert ex.value.status == mg.EBADGRAPH
    with pytest.raises(mg.MixgcnError) as ex:
        mg.graph_create(ctx, -5, e, e)
    assert ex.value.status == mg.EINVAL
