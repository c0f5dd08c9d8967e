"""Pins for the CPU oracle: each part is checked against something other than itself --
dense brute force on tiny graphs, closed forms that follow from Section 2.1 / Eq. 3 of the
paper, library routines (numpy, scipy.sparse, torch autograd, torch.optim.Adam), invariants
and finite differences.  No GPU and no CUDA code is involved."""
import math
import os

import numpy as np
import pytest
import scipy.sparse as sp
import torch
from hypothesis import given, settings, strategies as st

from oracle import gcn_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------- brute force helpers

def dense_atilde(n, src, dst, sym=True):
    A = np.zeros((n, n))
    for u, v in zip(src, dst):
        if u == v:
            continue
        A[u, v] = 1.0
        if sym:
            A[v, u] = 1.0
    return A + np.eye(n)


def dense_ahat(n, src, dst, sym=True):
    At = dense_atilde(n, src, dst, sym)
    D = At.sum(axis=1)
    return At / np.sqrt(np.outer(D, D))


def csr_to_dense(g, vals=None, transposed=False):
    M = np.zeros((g.n, g.n))
    rp, cl = (g.rowptr_t, g.col_t) if transposed else (g.rowptr, g.col)
    vl = (g.val_t if transposed else g.val) if vals is None else vals
    for u in range(g.n):
        for i in range(rp[u], rp[u + 1]):
            M[u, cl[i]] = vl[i]
    return M


def ring(n):
    s = np.arange(n)
    return s, (s + 1) % n


def complete(n):
    s, d = np.triu_indices(n, 1)
    return s, d


edge_lists = st.integers(1, 24).flatmap(
    lambda n: st.tuples(st.just(n), st.lists(st.tuples(st.integers(0, n - 1), st.integers(0, n - 1)), max_size=80)))


# ----------------------------------------------------------------------- O1: structure

@settings(max_examples=60, deadline=None)
@given(edge_lists, st.booleans())
def test_csr_matches_dense_bruteforce(ne, sym):
    n, edges = ne
    src = np.array([e[0] for e in edges], dtype=np.int32)
    dst = np.array([e[1] for e in edges], dtype=np.int32)
    g = orc.graph_build(n, src, dst, (orc.SYMMETRISE if sym else 0) | orc.ADD_SELF_LOOPS)
    At = dense_atilde(n, src, dst, sym)
    assert g.nnz == int(At.sum())
    assert g.rowptr[0] == 0 and np.all(np.diff(g.rowptr) >= 1)
    for u in range(n):
        row = g.col[g.rowptr[u]:g.rowptr[u + 1]]
        assert np.all(np.diff(row) > 0)                       # strictly ascending, no duplicates
        assert np.array_equal(row, np.nonzero(At[u])[0])
    assert np.array_equal(g.deg, At.sum(axis=1).astype(np.int32))
    # transposed structure, built on its own
    AtT = At.T
    for u in range(n):
        assert np.array_equal(g.col_t[g.rowptr_t[u]:g.rowptr_t[u + 1]], np.nonzero(AtT[u])[0])
    np.testing.assert_allclose(csr_to_dense(g), dense_ahat(n, src, dst, sym), rtol=1e-15, atol=0)
    np.testing.assert_allclose(csr_to_dense(g, transposed=True), dense_ahat(n, src, dst, sym).T, rtol=1e-15, atol=0)


def test_entry_counts_closed_form():
    n = 17
    assert orc.graph_build(n, *complete(n)).nnz == n * n
    assert orc.graph_build(n, *ring(n)).nnz == 3 * n
    m = 9
    assert orc.graph_build(m + 1, np.zeros(m, np.int32), np.arange(1, m + 1)).nnz == 3 * m + 1
    assert orc.graph_build(n, np.zeros(0, np.int32), np.zeros(0, np.int32)).nnz == n
    # duplicates and both orientations of an edge collapse; input self-loops do not add a second diagonal
    g = orc.graph_build(3, [0, 1, 0, 2, 2], [1, 0, 1, 2, 2])
    assert g.nnz == 3 + 2
    assert np.array_equal(g.col, [0, 1, 0, 1, 2])


def test_symmetric_input_gives_identical_transpose():
    g = orc.graph_build(50, *ring(50))
    assert np.array_equal(g.rowptr, g.rowptr_t) and np.array_equal(g.col, g.col_t)
    assert np.array_equal(g.val, g.val_t)


def test_bad_ids_rejected():
    with pytest.raises(ValueError):
        orc.graph_build(4, [0, 5], [1, 2])


# ----------------------------------------------------------------------- O2: normalisation

def test_complete_graph_is_J_over_n():
    n = 12
    g = orc.graph_build(n, *complete(n))
    np.testing.assert_allclose(csr_to_dense(g), np.full((n, n), 1.0 / n), rtol=1e-15)


def test_regular_graph_entries():
    n = 20
    g = orc.graph_build(n, *ring(n))          # 2-regular
    np.testing.assert_allclose(g.val, 1.0 / 3.0, rtol=1e-15)


def test_path2_and_edgeless():
    g = orc.graph_build(2, [0], [1])
    np.testing.assert_allclose(csr_to_dense(g), [[0.5, 0.5], [0.5, 0.5]], rtol=1e-15)
    g = orc.graph_build(5, [], [])
    np.testing.assert_array_equal(csr_to_dense(g), np.eye(5))


def test_star_golden():
    want = np.loadtxt(os.path.join(GOLD, "star_k14_ahat.txt"))
    g = orc.graph_build(5, [0, 0, 0, 0], [1, 2, 3, 4])
    np.testing.assert_allclose(csr_to_dense(g), want, rtol=1e-15)
    m = 7
    g = orc.graph_build(m + 1, np.zeros(m, np.int32), np.arange(1, m + 1))
    A = csr_to_dense(g)
    assert A[0, 0] == pytest.approx(1 / (m + 1), rel=1e-15)
    assert A[0, 3] == pytest.approx(1 / math.sqrt(2 * (m + 1)), rel=1e-15)
    assert A[3, 3] == pytest.approx(0.5, rel=1e-15)


def test_fp32_storage_recipe():
    """val32 = fl(fl(1/fl(sqrt(deg_u))) * fl(1/fl(sqrt(deg_v)))) with IEEE fp32 operations."""
    rng = np.random.default_rng(0)
    n = 40
    src, dst = rng.integers(0, n, 150), rng.integers(0, n, 150)
    g = orc.graph_build(n, src, dst)
    dinv = (np.float32(1.0) / np.sqrt(g.deg.astype(np.float32))).astype(np.float32)
    assert np.array_equal(g.dinv32, dinv)
    rows = np.repeat(np.arange(n), np.diff(g.rowptr))
    assert np.array_equal(g.val32, (dinv[rows] * dinv[g.col]).astype(np.float32))
    np.testing.assert_allclose(g.val32, g.val, rtol=3e-7)


def test_directed_graph_uses_row_sum_degrees():
    # 0->1, 0->2, 1->2 stored as rows: row sums (incl. diagonal) are 3, 2, 1
    g = orc.graph_build(3, [0, 0, 1], [1, 2, 2], orc.ADD_SELF_LOOPS)
    assert list(g.deg) == [3, 2, 1]
    A = csr_to_dense(g)
    assert A[0, 1] == pytest.approx(1 / math.sqrt(6)) and A[1, 2] == pytest.approx(1 / math.sqrt(2))
    assert A[1, 0] == 0 and A[2, 2] == 1.0


# ----------------------------------------------------------------------- O3: aggregation

@settings(max_examples=25, deadline=None)
@given(edge_lists, st.booleans(), st.integers(1, 9))
def test_aggregate_matches_dense(ne, sym, d):
    n, edges = ne
    src = [e[0] for e in edges]; dst = [e[1] for e in edges]
    g = orc.graph_build(n, src, dst, (orc.SYMMETRISE if sym else 0) | orc.ADD_SELF_LOOPS)
    X = np.random.default_rng(n * 100 + d).standard_normal((n, d))
    Ah = dense_ahat(n, src, dst, sym)
    np.testing.assert_allclose(orc.aggregate(g, X), Ah @ X, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(orc.aggregate(g, X, transposed=True), Ah.T @ X, rtol=1e-12, atol=1e-13)
    rows = np.arange(n)[::2]
    np.testing.assert_allclose(orc.aggregate_rows(g, X, rows), (Ah @ X)[rows], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(orc.aggregate_rows(g, X, rows, transposed=True), (Ah.T @ X)[rows], rtol=1e-12, atol=1e-13)


def test_sampled_aggregate_is_the_masked_dense_product():
    # Eq. 4 on a dense matrix: (A_hat X) (.) M, with a mask that keeps nothing, everything, and a random half
    n, d = 12, 7
    rng = np.random.default_rng(4)
    src, dst = rng.integers(0, n, 30), rng.integers(0, n, 30)
    g = orc.graph_build(n, src, dst)
    Ah = dense_ahat(n, list(src), list(dst), True)
    X = rng.standard_normal((n, d))
    for M in (np.zeros((n, d)), np.ones((n, d)), rng.integers(0, 2, (n, d))):
        np.testing.assert_allclose(orc.sampled_aggregate(g, X, M), (Ah @ X) * M, rtol=1e-12, atol=1e-13)
    M = rng.integers(0, 2, (n, d))
    assert np.all(orc.sampled_aggregate(g, X, M)[M == 0] == 0.0)


def test_aggregate_vs_scipy_at_tiny_size():
    from paper_2501_01951_b200 import synth
    wl = synth.CONFIGS["C1"]
    s, d = synth.rmat_graph(wl.n, wl.undirected_edges, wl.seed("graph"))
    g = orc.graph_build(wl.n, s.numpy(), d.numpy())
    X = synth.normal_features(wl.n, 16, 7).numpy().astype(np.float64)
    M = sp.csr_matrix((g.val, g.col, g.rowptr), shape=(wl.n, wl.n))
    np.testing.assert_allclose(orc.aggregate(g, X), M @ X, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(orc.aggregate(g, X, transposed=True), M.T @ X, rtol=1e-12, atol=1e-13)
    # symmetric graph: sqrt(deg~) is the eigenvector of A_hat with eigenvalue 1
    r = np.sqrt(g.deg.astype(np.float64))[:, None]
    np.testing.assert_allclose(orc.aggregate(g, r), r, rtol=1e-12)


def test_complete_graph_aggregation_is_column_mean():
    n = 9
    g = orc.graph_build(n, *complete(n))
    X = np.random.default_rng(1).standard_normal((n, 5))
    np.testing.assert_allclose(orc.aggregate(g, X), np.tile(X.mean(axis=0), (n, 1)), rtol=1e-13)


def test_regular_graph_row_sums_are_one():
    g = orc.graph_build(30, *ring(30))
    np.testing.assert_allclose(orc.aggregate(g, np.ones((30, 3))), 1.0, rtol=1e-14)


def test_adjoint_identity_on_directed_graph():
    rng = np.random.default_rng(3)
    n = 60
    g = orc.graph_build(n, rng.integers(0, n, 300), rng.integers(0, n, 300), orc.ADD_SELF_LOOPS)
    X, G = rng.standard_normal((n, 4)), rng.standard_normal((n, 4))
    assert np.sum(orc.aggregate(g, X) * G) == pytest.approx(np.sum(X * orc.aggregate(g, G, transposed=True)), rel=1e-12)


# ----------------------------------------------------------------------- O3: update / epilogue

@pytest.mark.parametrize("norm", ["row", "none"])
@pytest.mark.parametrize("sym", [True, False])
def test_other_aggregators_match_their_definitions(norm, sym):
    """Row-mean (GraphSAGE mean aggregator) and plain-sum (GIN) values on the stored structure, against
    the dense matrices written out: A_tilde with rows divided by their entry count, and A_tilde itself."""
    n = 37
    rng = np.random.default_rng(5)
    src, dst = rng.integers(0, 30, 160).astype(np.int32), rng.integers(0, 30, 160).astype(np.int32)   # ids >= 30 stay isolated
    flags = orc.ADD_SELF_LOOPS | (orc.SYMMETRISE if sym else 0)
    g = orc.graph_build(n, src, dst, flags, norm=norm)
    At = np.zeros((n, n))
    At[src, dst] = 1.0
    if sym:
        At[dst, src] = 1.0
    At[np.arange(n), np.arange(n)] = 1.0
    dense = At / At.sum(axis=1, keepdims=True) if norm == "row" else At
    got = np.zeros((n, n)); gotT = np.zeros((n, n))
    for u in range(n):
        got[u, g.col[g.rowptr[u]:g.rowptr[u + 1]]] = g.val[g.rowptr[u]:g.rowptr[u + 1]]
        gotT[u, g.col_t[g.rowptr_t[u]:g.rowptr_t[u + 1]]] = g.val_t[g.rowptr_t[u]:g.rowptr_t[u + 1]]
    assert np.allclose(got, dense, rtol=0, atol=1e-15) and np.allclose(gotT, dense.T, rtol=0, atol=1e-15)
    X = rng.standard_normal((n, 5))
    assert np.allclose(orc.aggregate(g, X), dense @ X, atol=1e-12)
    assert np.allclose(orc.aggregate(g, X, transposed=True), dense.T @ X, atol=1e-12)
    if norm == "row":
        assert np.allclose(orc.aggregate(g, np.ones((n, 1))), 1.0)              # a mean of ones is one
        assert np.array_equal(g.val32, (np.float32(1.0) / np.diff(g.rowptr).astype(np.float32))[np.repeat(np.arange(n), np.diff(g.rowptr))])
    else:
        assert np.array_equal(orc.aggregate(g, np.ones((n, 1)))[:, 0], np.diff(g.rowptr).astype(np.float64))   # row sums = entry counts


def test_update_and_activation_vs_numpy():
    rng = np.random.default_rng(4)
    Z, W, b = rng.standard_normal((37, 11)), rng.standard_normal((11, 6)), rng.standard_normal(6)
    np.testing.assert_allclose(orc.update(Z, W, b), Z @ W + b, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(orc.update(Z, W), Z @ W, rtol=1e-13, atol=1e-14)
    P = Z @ W + b
    mask = (rng.random(P.shape) < 0.5).astype(np.uint8)
    np.testing.assert_array_equal(orc.activation(P), np.maximum(P, 0))
    np.testing.assert_allclose(orc.activation(P, True, mask, 2.0), np.maximum(P, 0) * mask * 2.0, rtol=1e-15)
    np.testing.assert_array_equal(orc.activation(P, False), P)


def test_edgeless_graph_is_an_mlp():
    rng = np.random.default_rng(5)
    n, dims = 13, (6, 5, 4)
    g = orc.graph_build(n, [], [])
    X = rng.standard_normal((n, dims[0]))
    Ws = [rng.standard_normal((dims[i], dims[i + 1])) for i in range(2)]
    bs = [rng.standard_normal(dims[i + 1]) for i in range(2)]
    _, _, Xs = orc.forward(g, X, Ws, bs)
    np.testing.assert_allclose(Xs[-1], np.maximum(X @ Ws[0] + bs[0], 0) @ Ws[1] + bs[1], rtol=1e-13, atol=1e-14)


def test_product_order_does_not_matter():
    rng = np.random.default_rng(6)
    n = 50
    g = orc.graph_build(n, rng.integers(0, n, 200), rng.integers(0, n, 200))
    X, W = rng.standard_normal((n, 7)), rng.standard_normal((7, 3))
    np.testing.assert_allclose(orc.update(orc.aggregate(g, X), W), orc.aggregate(g, orc.update(X, W)), rtol=1e-11, atol=1e-13)


# ----------------------------------------------------------------------- O4: loss

@pytest.mark.parametrize("Cc", [8, 41, 47, 64, 172])
def test_zero_logits_give_ln_C(Cc):
    n = 10
    labels = np.arange(n) % Cc
    mask = np.array([1, 0] * 5, dtype=np.uint8)
    lo, G, pred, nc, T = orc.loss(np.zeros((n, Cc)), labels, mask)
    assert T == 5 and lo == pytest.approx(math.log(Cc), rel=1e-14)
    want = np.full((n, Cc), 1.0 / Cc)
    want[np.arange(n), labels] -= 1.0
    want *= mask[:, None] / 5.0
    np.testing.assert_allclose(G, want, rtol=1e-13, atol=1e-17)
    assert np.all(pred == 0)                                   # ties -> lowest index


def test_loss_invariants_and_torch_cross_entropy():
    rng = np.random.default_rng(7)
    n, Cc = 40, 9
    P = rng.standard_normal((n, Cc)) * 3
    labels = rng.integers(0, Cc, n).astype(np.int32)
    mask = (rng.random(n) < 0.6).astype(np.uint8)
    lo, G, pred, nc, T = orc.loss(P, labels, mask)
    np.testing.assert_allclose(G.sum(axis=1), 0, atol=1e-15)
    assert np.all(G[mask == 0] == 0)
    lo2, G2, *_ = orc.loss(P + rng.standard_normal((n, 1)) * 50, labels, mask)
    assert lo2 == pytest.approx(lo, rel=1e-12)
    np.testing.assert_allclose(G2, G, rtol=1e-9, atol=1e-14)
    Pt = torch.tensor(P, requires_grad=True)
    idx = torch.tensor(np.nonzero(mask)[0])
    lt = torch.nn.functional.cross_entropy(Pt[idx], torch.tensor(labels, dtype=torch.long)[idx])
    lt.backward()
    assert lo == pytest.approx(lt.item(), rel=1e-12)
    np.testing.assert_allclose(G, Pt.grad.numpy(), rtol=1e-10, atol=1e-15)
    assert np.array_equal(pred, P.argmax(axis=1))
    assert nc == int(np.sum((P.argmax(axis=1) == labels) & (mask == 1)))


# ----------------------------------------------------------------------- O5: backward

def _small_problem(seed, directed=False):
    rng = np.random.default_rng(seed)
    n, dims = 24, (5, 6, 4, 3)
    flags = orc.ADD_SELF_LOOPS | (0 if directed else orc.SYMMETRISE)
    src, dst = rng.integers(0, n, 70), rng.integers(0, n, 70)
    g = orc.graph_build(n, src, dst, flags)
    X = rng.standard_normal((n, dims[0]))
    Ws = [rng.standard_normal((dims[i], dims[i + 1])) * 0.7 for i in range(3)]
    bs = [rng.standard_normal(dims[i + 1]) * 0.3 for i in range(3)]
    labels = rng.integers(0, dims[-1], n).astype(np.int32)
    mask = (rng.random(n) < 0.5).astype(np.uint8)
    mask[0] = 1
    drop = [(rng.random((n, dims[i + 1])) < 0.7).astype(np.uint8) for i in range(2)]
    return g, (src, dst, not directed), X, Ws, bs, labels, mask, drop


@pytest.mark.parametrize("directed", [False, True])
def test_gradients_vs_finite_differences(directed):
    g, _, X, Ws, bs, labels, mask, drop = _small_problem(11, directed)
    ks = 1 / 0.7

    def f(Ws_, bs_):
        _, _, Xs = orc.forward(g, X, Ws_, bs_, drop, ks)
        return orc.loss(Xs[-1], labels, mask)[0]

    Zs, Ps, Xs = orc.forward(g, X, Ws, bs, drop, ks)
    _, G, *_ = orc.loss(Xs[-1], labels, mask)
    dWs, dbs = orc.backward(g, Zs, Ps, Ws, G, drop, ks)
    rng = np.random.default_rng(0)
    h = 1e-6
    for l in range(3):
        for _ in range(6):
            i, j = rng.integers(0, Ws[l].shape[0]), rng.integers(0, Ws[l].shape[1])
            Wp = [w.copy() for w in Ws]; Wm = [w.copy() for w in Ws]
            Wp[l][i, j] += h; Wm[l][i, j] -= h
            fd = (f(Wp, bs) - f(Wm, bs)) / (2 * h)
            assert dWs[l][i, j] == pytest.approx(fd, rel=2e-6, abs=1e-9)
        for j in range(len(bs[l])):
            bp = [b.copy() for b in bs]; bm = [b.copy() for b in bs]
            bp[l][j] += h; bm[l][j] -= h
            fd = (f(Ws, bp) - f(Ws, bm)) / (2 * h)
            assert dbs[l][j] == pytest.approx(fd, rel=2e-6, abs=1e-9)


@pytest.mark.parametrize("directed", [False, True])
def test_gradients_vs_torch_autograd_on_dense_ahat(directed):
    g, (src, dst, sym), X, Ws, bs, labels, mask, drop = _small_problem(12, directed)
    ks = 1 / 0.7
    Ah = torch.tensor(dense_ahat(g.n, src, dst, sym))
    Wt = [torch.tensor(w, requires_grad=True) for w in Ws]
    bt = [torch.tensor(b, requires_grad=True) for b in bs]
    H = torch.tensor(X)
    for l in range(3):
        H = Ah @ H @ Wt[l] + bt[l]
        if l < 2:
            H = torch.relu(H) * torch.tensor(drop[l], dtype=torch.float64) * ks
    idx = torch.tensor(np.nonzero(mask)[0])
    lt = torch.nn.functional.cross_entropy(H[idx], torch.tensor(labels, dtype=torch.long)[idx])
    lt.backward()
    res = orc.train_epoch(g, X, Ws, bs, labels, mask, masks=drop, keep_scale=ks)
    assert res["loss"] == pytest.approx(lt.item(), rel=1e-12)
    np.testing.assert_allclose(res["logits"], H.detach().numpy(), rtol=1e-11, atol=1e-13)
    for l in range(3):
        np.testing.assert_allclose(res["dW"][l], Wt[l].grad.numpy(), rtol=1e-9, atol=1e-13)
        np.testing.assert_allclose(res["db"][l], bt[l].grad.numpy(), rtol=1e-9, atol=1e-13)


# ----------------------------------------------------------------------- O6: Adam

def _dense_aggregator(n, src, dst, norm):
    A = np.zeros((n, n))
    A[src, dst] = 1.0; A[dst, src] = 1.0
    np.fill_diagonal(A, 0.0)
    if norm == "row":
        rs = A.sum(axis=1, keepdims=True)
        A = np.divide(A, rs, out=np.zeros_like(A), where=rs > 0)
    return A


def _small_model_problem(seed):
    rng = np.random.default_rng(seed)
    n, dims = 40, (6, 5, 4, 3)
    src, dst = rng.integers(0, 34, 120).astype(np.int32), rng.integers(0, 34, 120).astype(np.int32)
    keep = src != dst
    src, dst = src[keep], dst[keep]
    X = rng.standard_normal((n, dims[0]))
    y = rng.integers(0, dims[-1], n).astype(np.int32)
    m = (rng.random(n) < 0.5).astype(np.uint8); m[0] = 1
    return rng, n, dims, src, dst, X, y, m


def test_sage_gradients_vs_torch_autograd_on_dense_mean_matrix():
    """The oracle's GraphSAGE-mean iteration against autograd on the dense row-mean matrix."""
    rng, n, dims, src, dst, X, y, m = _small_model_problem(11)
    g = orc.graph_build(n, src, dst, orc.SYMMETRISE, norm="row")
    Ws = [rng.standard_normal((dims[i], dims[i + 1])) * 0.4 for i in range(3)]
    Wn = [rng.standard_normal((dims[i], dims[i + 1])) * 0.4 for i in range(3)]
    bs = [rng.standard_normal(dims[i + 1]) * 0.1 for i in range(3)]
    ref = orc.sage_epoch(g, X, Ws, Wn, bs, y, m)
    M = torch.tensor(_dense_aggregator(n, src, dst, "row"))
    tw = [torch.tensor(w, requires_grad=True) for w in Ws + Wn + bs]
    H = torch.tensor(X)
    for l in range(3):
        P = H @ tw[l] + (M @ H) @ tw[3 + l] + tw[6 + l]
        H = P if l == 2 else torch.relu(P)
    idx = torch.tensor(np.nonzero(m)[0])
    lt = torch.nn.functional.cross_entropy(H[idx], torch.tensor(y, dtype=torch.int64)[idx])
    lt.backward()
    assert abs(ref["loss"] - lt.item()) <= 1e-12 * abs(lt.item())
    for got, t_ in zip(ref["grads"], tw):
        assert np.allclose(got, t_.grad.numpy(), rtol=1e-10, atol=1e-13)
    # isolated nodes average nothing: their neighbour term is zero
    iso = np.setdiff1d(np.arange(n), np.union1d(src, dst))
    assert len(iso) > 0 and np.all(orc.aggregate(g, X)[iso] == 0.0)


@pytest.mark.parametrize("gin_eps", [0.0, 0.3])
def test_gin_gradients_vs_torch_autograd_on_dense_adjacency(gin_eps):
    """The oracle's GIN iteration against autograd on the dense adjacency matrix."""
    rng, n, dims, src, dst, X, y, m = _small_model_problem(12)
    g = orc.graph_build(n, src, dst, orc.SYMMETRISE, norm="none")
    hid = 7
    W1 = [rng.standard_normal((dims[i], hid)) * 0.3 for i in range(3)]
    b1 = [rng.standard_normal(hid) * 0.1 for i in range(3)]
    W2 = [rng.standard_normal((hid, dims[i + 1])) * 0.3 for i in range(3)]
    b2 = [rng.standard_normal(dims[i + 1]) * 0.1 for i in range(3)]
    ref = orc.gin_epoch(g, X, W1, b1, W2, b2, y, m, gin_eps=gin_eps)
    A = torch.tensor(_dense_aggregator(n, src, dst, "none"))
    tw = [torch.tensor(w, requires_grad=True) for w in W1 + b1 + W2 + b2]
    H = torch.tensor(X)
    for l in range(3):
        Z = (1.0 + gin_eps) * H + A @ H
        P = torch.relu(Z @ tw[l] + tw[3 + l]) @ tw[6 + l] + tw[9 + l]
        H = P if l == 2 else torch.relu(P)
    idx = torch.tensor(np.nonzero(m)[0])
    lt = torch.nn.functional.cross_entropy(H[idx], torch.tensor(y, dtype=torch.int64)[idx])
    lt.backward()
    assert abs(ref["loss"] - lt.item()) <= 1e-12 * abs(lt.item())
    for got, t_ in zip(ref["grads"], tw):
        assert np.allclose(got, t_.grad.numpy(), rtol=1e-10, atol=1e-13)


def test_adam_closed_forms():
    rng = np.random.default_rng(8)
    th0, g = rng.standard_normal(50), rng.standard_normal(50)
    lr, eps = 0.01, 1e-8
    th, m, v = orc.adam(th0, g, np.zeros(50), np.zeros(50), 1, lr=lr, eps=eps)
    np.testing.assert_allclose(th, th0 - lr * g / (np.abs(g) + eps), rtol=1e-13)
    # constant gradient: corrected moments are g and g^2 at every step
    th, m, v = th0, np.zeros(50), np.zeros(50)
    for t in range(1, 8):
        th, m, v = orc.adam(th, g, m, v, t, lr=lr, eps=eps)
        np.testing.assert_allclose(th, th0 - t * lr * g / (np.abs(g) + eps), rtol=1e-11)
    th, m, v = orc.adam(th0, np.zeros(50), np.zeros(50), np.zeros(50), 1)
    np.testing.assert_array_equal(th, th0)


def test_adam_vs_torch_optim():
    rng = np.random.default_rng(9)
    th0 = rng.standard_normal((6, 5))
    p = torch.tensor(th0.copy(), requires_grad=True)
    opt = torch.optim.Adam([p], lr=0.01, betas=(0.9, 0.999), eps=1e-8)
    th, m, v = th0, np.zeros_like(th0), np.zeros_like(th0)
    for t in range(1, 6):
        g = rng.standard_normal((6, 5))
        p.grad = torch.tensor(g)
        opt.step()
        th, m, v = orc.adam(th, g, m, v, t)
        np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-11, atol=1e-14)


# ----------------------------------------------------------------------- workload shapes

def test_workloads_take_the_papers_table_shapes():
    from paper_2501_01951_b200 import synth
    rows = {}
    for line in open(os.path.join(GOLD, "datasets_table.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, nodes, edges, feats, classes = line.split()
        rows[name] = (float(nodes), float(edges), int(feats), int(classes))
    c2, c5 = synth.CONFIGS["C2"], synth.CONFIGS["C5"]
    nodes, edges, feats, classes = rows["Reddit"]
    assert abs(c2.n - nodes) / nodes < 0.01 and abs(2 * c2.undirected_edges - edges) / edges < 0.01
    assert c2.dims[0] == feats and c2.classes == classes
    _, _, feats, classes = rows["ogbn-papers100M"]
    assert c5.dims[0] == feats and c5.classes == classes


# ----------------------------------------------------------------------- node reordering (Section 3.2.2)

def _brute_bandwidth(n, g, order):
    pos = np.empty(n, dtype=np.int64); pos[order] = np.arange(n)
    return max(abs(pos[u] - pos[v]) for u in range(n) for v in g.col[g.rowptr[u]:g.rowptr[u + 1]])


def test_bandwidth_closed_forms_and_bruteforce():
    n = 40
    s = np.arange(n - 1)
    path = orc.graph_build(n, s, s + 1)
    assert orc.bandwidth(path) == 1                                   # a path in its natural order
    assert orc.bandwidth(orc.graph_build(n, *ring(n))) == n - 1       # the closing edge of a ring
    assert orc.bandwidth(orc.graph_build(n, np.zeros(n - 1, np.int64), np.arange(1, n))) == n - 1    # star, centre first
    assert orc.bandwidth(orc.graph_build(n, [], [])) == 0
    rng = np.random.default_rng(5)
    g = orc.graph_build(n, rng.integers(0, n, 90), rng.integers(0, n, 90))
    order = rng.permutation(n)
    assert orc.bandwidth(g, order) == _brute_bandwidth(n, g, order)


def test_rcm_is_a_valid_order_and_matches_scipy_quality():
    from scipy.sparse.csgraph import reverse_cuthill_mckee
    rng = np.random.default_rng(6)
    for n, m in ((30, 40), (200, 400), (500, 700)):
        g = orc.graph_build(n, rng.integers(0, n, m), rng.integers(0, n, m))
        order = orc.rcm(g)
        assert np.array_equal(np.sort(order), np.arange(n))
        M = sp.csr_matrix((np.ones(g.nnz), g.col, g.rowptr), shape=(n, n))
        ref = reverse_cuthill_mckee(M, symmetric_mode=True)
        b_ours, b_ref, b_nat = orc.bandwidth(g, order), orc.bandwidth(g, ref.astype(np.int64)), orc.bandwidth(g)
        # tie-breaking rules differ between implementations, so compare the quality of the result
        assert b_ours <= 1.25 * b_ref + 2 and b_ours < b_nat


def test_rcm_on_structured_graphs():
    # a path given in scrambled labels is recovered as a path: bandwidth 1
    n = 64
    rng = np.random.default_rng(7)
    lab = rng.permutation(n)
    g = orc.graph_build(n, lab[:-1], lab[1:])
    assert orc.bandwidth(g) > 1 and orc.bandwidth(g, orc.rcm(g)) == 1
    # a 2-D grid r x c has bandwidth min(r, c) under the level order RCM produces
    r, c = 6, 9
    idx = np.arange(r * c).reshape(r, c)
    s = np.concatenate([idx[:, :-1].ravel(), idx[:-1, :].ravel()]); d = np.concatenate([idx[:, 1:].ravel(), idx[1:, :].ravel()])
    g = orc.graph_build(r * c, s, d)
    assert orc.bandwidth(g, orc.rcm(g)) <= min(r, c) + 1
    # components: every node appears once; isolated nodes are placed too
    g = orc.graph_build(10, [0, 1, 5], [1, 2, 6])
    assert np.array_equal(np.sort(orc.rcm(g)), np.arange(10))


def test_pipeline_stage_count():
    # the paper's remark: b = 0.8 n still allows a pipeline, with 2 / 0.2 = 10 stages
    assert orc.pipeline_stages(1000, 800) == 10
    assert orc.pipeline_stages(1000, 0) == 2 and orc.pipeline_stages(1000, 1) == 3
    assert orc.pipeline_stages(1000, 999) == 2000 and orc.pipeline_stages(1000, 1000) == -1
    for n, b in ((37, 5), (100, 33), (12345, 6789)):
        s = orc.pipeline_stages(n, b)
        assert (n - b) / (2 * n) >= 1 / s and (s == 1 or (n - b) / (2 * n) < 1 / (s - 1))
