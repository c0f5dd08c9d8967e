"""Python face of the CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Wraps ``gcn_oracle.c`` (plain C, fp64, definition-order loops) with numpy arrays and composes
its steps into whole forward / backward / training-epoch passes in the order Algorithm 2 of
the paper gives: for each layer aggregation then update, then the loss, the backward pass and
the weight update.  The forward is always evaluated as sigma((A_hat X) W + b) (Eq. 3, left to
right); the oracle never reorders the product.

Only tests, the smoke check and the benchmark's cpu-baseline leg import this module.  It
imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gcn_oracle.c")
_LIB = os.path.join(_HERE, "libgcn_oracle.so")

SYMMETRISE = 1
ADD_SELF_LOOPS = 2


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_graph_build.restype = C.c_int64
        _lib.oracle_loss.restype = C.c_int64
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def n_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or all cores)."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


# ------------------------------------------------------------------------------ graph

class Graph:
    """A_hat in CSR plus the independently built transposed structure (fp64 values)."""

    def __init__(self, n, rowptr, col, val, rowptr_t, col_t, val_t, deg, dinv32, val32, src_index_t):
        self.n, self.rowptr, self.col, self.val = n, rowptr, col, val
        self.rowptr_t, self.col_t, self.val_t = rowptr_t, col_t, val_t
        self.deg, self.dinv32, self.val32, self.src_index_t = deg, dinv32, val32, src_index_t

    @property
    def nnz(self):
        return int(self.rowptr[-1])


NORMS = {"sym": 0, "row": 1, "none": 2}


def graph_build(n, src, dst, flags=SYMMETRISE | ADD_SELF_LOOPS, norm="sym") -> Graph:
    """A_tilde = A + I and A_hat = D^-1/2 A_tilde D^-1/2 (Section 2.1) from an edge list.
    norm = "row": row-mean values (GraphSAGE mean aggregator); "none": ones (GIN sum aggregator)."""
    src = np.ascontiguousarray(src, dtype=np.int32)
    dst = np.ascontiguousarray(dst, dtype=np.int32)
    m = len(src)
    L = lib()
    rowptr = np.zeros(n + 1, dtype=np.int64)
    nnz = L.oracle_graph_build(C.c_int64(n), C.c_int64(m), _p(src, C.c_int32), _p(dst, C.c_int32),
                               C.c_uint32(flags), _p(rowptr, C.c_int64), None)
    if nnz < 0:
        raise ValueError("oracle_graph_build: bad edge list (code %d)" % nnz)
    col = np.zeros(max(nnz, 1), dtype=np.int32)
    L.oracle_graph_build(C.c_int64(n), C.c_int64(m), _p(src, C.c_int32), _p(dst, C.c_int32),
                         C.c_uint32(flags), _p(rowptr, C.c_int64), _p(col, C.c_int32))
    col = col[:nnz]
    return graph_from_csr(n, rowptr, col, norm)


def graph_from_csr(n, rowptr, col, norm="sym") -> Graph:
    L = lib()
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    col = np.ascontiguousarray(col, dtype=np.int32)
    nnz = int(rowptr[-1])
    val = np.zeros(max(nnz, 1), dtype=np.float64)
    val32 = np.zeros(max(nnz, 1), dtype=np.float32)
    dinv32 = np.zeros(n, dtype=np.float32)
    deg = np.zeros(n, dtype=np.int32)
    L.oracle_normalise(C.c_int64(n), _p(rowptr, C.c_int64), _p(col, C.c_int32), _p(val, C.c_double),
                       _p(dinv32, C.c_float), _p(val32, C.c_float), _p(deg, C.c_int32))
    if NORMS[norm] != 0:
        L.oracle_normalise_mode(C.c_int64(n), _p(rowptr, C.c_int64), C.c_int32(NORMS[norm]), _p(val, C.c_double), _p(val32, C.c_float))
    rowptr_t = np.zeros(n + 1, dtype=np.int64)
    col_t = np.zeros(max(nnz, 1), dtype=np.int32)
    sidx = np.zeros(max(nnz, 1), dtype=np.int64)
    L.oracle_transpose(C.c_int64(n), _p(rowptr, C.c_int64), _p(col, C.c_int32),
                       _p(rowptr_t, C.c_int64), _p(col_t, C.c_int32), _p(sidx, C.c_int64))
    val, val32, col_t, sidx = val[:nnz], val32[:nnz], col_t[:nnz], sidx[:nnz]
    return Graph(n, rowptr, col, val, rowptr_t, col_t, np.ascontiguousarray(val[sidx]), deg, dinv32, val32, sidx)


# ------------------------------------------------------------------------------ steps

def aggregate(g: Graph, X, transposed=False):
    """Z = A_hat X (or A_hat^T X), Algorithm 2 aggregation line."""
    X = _f64(X)
    n, d = X.shape
    Z = np.zeros((n, d), dtype=np.float64)
    rp, cl, vl = (g.rowptr_t, g.col_t, g.val_t) if transposed else (g.rowptr, g.col, g.val)
    lib().oracle_aggregate(C.c_int64(n), _p(rp, C.c_int64), _p(cl, C.c_int32), _p(vl, C.c_double),
                           C.c_int64(d), _p(X, C.c_double), C.c_int64(d), _p(Z, C.c_double), C.c_int64(d))
    return Z


def sampled_aggregate(g: Graph, X, M, transposed=False):
    """Z = (A_hat X) (.) M, the sampled aggregation of Eq. 4: M is a 0/1 array of Z's shape (1 = kept)."""
    return aggregate(g, X, transposed) * (np.asarray(M) != 0)


def aggregate_rows(g: Graph, X, rows, transposed=False):
    """Rows ``rows`` of A_hat X (or A_hat^T X) only; X may be any array indexable by node id
    whose needed rows are present (here: a full n x d array)."""
    X = _f64(X)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    d = X.shape[1]
    out = np.zeros((len(rows), d), dtype=np.float64)
    rp, cl, vl = (g.rowptr_t, g.col_t, g.val_t) if transposed else (g.rowptr, g.col, g.val)
    lib().oracle_aggregate_rows(C.c_int64(len(rows)), _p(rows, C.c_int64), _p(rp, C.c_int64),
                                _p(cl, C.c_int32), _p(vl, C.c_double), C.c_int64(d),
                                _p(X, C.c_double), C.c_int64(d), _p(out, C.c_double))
    return out


def update(Z, W, bias=None):
    """P = Z W + 1 b^T, Algorithm 2 update line before the activation."""
    Z, W = _f64(Z), _f64(W)
    n, d_in = Z.shape
    d_out = W.shape[1]
    assert W.shape[0] == d_in
    b = None if bias is None else _f64(bias)
    P = np.zeros((n, d_out), dtype=np.float64)
    lib().oracle_update(C.c_int64(n), C.c_int64(d_in), C.c_int64(d_out), _p(Z, C.c_double),
                        _p(W, C.c_double), _p(b, C.c_double), _p(P, C.c_double))
    return P


def activation(P, relu=True, mask=None, keep_scale=1.0):
    P = _f64(P)
    n, d = P.shape
    mk = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    out = np.zeros_like(P)
    lib().oracle_activation(C.c_int64(n), C.c_int64(d), _p(P, C.c_double), C.c_int(int(relu)),
                            _p(mk, C.c_uint8), C.c_double(keep_scale), _p(out, C.c_double))
    return out


def loss(P, labels, train_mask):
    """Masked softmax cross-entropy: returns (loss, G, pred, n_correct_on_mask, #T)."""
    P = _f64(P)
    n, Cc = P.shape
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    tm = np.ascontiguousarray(train_mask, dtype=np.uint8)
    G = np.zeros_like(P)
    pred = np.zeros(n, dtype=np.int32)
    lo = C.c_double(0.0)
    nc = C.c_int64(0)
    T = lib().oracle_loss(C.c_int64(n), C.c_int64(Cc), _p(P, C.c_double), _p(labels, C.c_int32),
                          _p(tm, C.c_uint8), C.byref(lo), _p(G, C.c_double), _p(pred, C.c_int32), C.byref(nc))
    return lo.value, G, pred, nc.value, int(T)


def update_bwd(Z, P, W, Gout, relu=True, mask=None, keep_scale=1.0, need_dZ=True):
    """dP, dW, db, dZ of one layer's update (chain rule on Eq. 3)."""
    Z, P, W, Gout = _f64(Z), _f64(P), _f64(W), _f64(Gout)
    n, d_in = Z.shape
    d_out = W.shape[1]
    mk = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    dP = np.zeros((n, d_out)); dW = np.zeros((d_in, d_out)); db = np.zeros(d_out)
    dZ = np.zeros((n, d_in)) if need_dZ else None
    lib().oracle_update_bwd(C.c_int64(n), C.c_int64(d_in), C.c_int64(d_out), _p(Z, C.c_double),
                            _p(P, C.c_double), _p(W, C.c_double), _p(Gout, C.c_double),
                            C.c_int(int(relu)), _p(mk, C.c_uint8), C.c_double(keep_scale),
                            _p(dP, C.c_double), _p(dW, C.c_double), _p(db, C.c_double), _p(dZ, C.c_double))
    return dP, dW, db, dZ


def adam(theta, g, m, v, t, lr=0.01, beta1=0.9, beta2=0.999, eps=1e-8):
    """One Adam step; returns new (theta, m, v) as fp64 copies."""
    theta, m, v = _f64(theta).copy(), _f64(m).copy(), _f64(v).copy()
    g = _f64(g)
    lib().oracle_adam(C.c_int64(theta.size), _p(theta, C.c_double), _p(g, C.c_double), _p(m, C.c_double),
                      _p(v, C.c_double), C.c_int64(t), C.c_double(lr), C.c_double(beta1),
                      C.c_double(beta2), C.c_double(eps))
    return theta, m, v


# ------------------------------------------------------------------------------ whole passes

def forward(g: Graph, X0, Ws, bs, masks=None, keep_scale=1.0):
    """All layers of Eq. 3 in Algorithm 2's order.  ReLU on every layer but the last.
    Returns the per-layer lists Z (aggregated input), P (pre-activation), X (activations,
    X[0] = input, X[L] = logits)."""
    L = len(Ws)
    Xs, Zs, Ps = [_f64(X0)], [], []
    for l in range(L):
        Z = aggregate(g, Xs[-1])
        P = update(Z, Ws[l], None if bs is None else bs[l])
        last = l == L - 1
        mk = None if (masks is None or last) else masks[l]
        Xn = P if last else activation(P, True, mk, keep_scale)
        Zs.append(Z); Ps.append(P); Xs.append(Xn)
    return Zs, Ps, Xs


def backward(g: Graph, Zs, Ps, Ws, G, masks=None, keep_scale=1.0):
    """Gradients of every W_l, b_l from the logits' gradient G (chain rule, last layer first).
    The first layer's input gradient is not computed (features are data)."""
    L = len(Ws)
    dWs, dbs = [None] * L, [None] * L
    Gout = G
    for l in range(L - 1, -1, -1):
        last = l == L - 1
        mk = None if (masks is None or last) else masks[l]
        _, dW, db, dZ = update_bwd(Zs[l], Ps[l], Ws[l], Gout, relu=not last, mask=mk,
                                   keep_scale=keep_scale, need_dZ=(l > 0))
        dWs[l], dbs[l] = dW, db
        if l > 0:
            Gout = aggregate(g, dZ, transposed=True)
    return dWs, dbs


def train_epoch(g: Graph, X0, Ws, bs, labels, train_mask, state=None, t=1, lr=0.01,
                beta1=0.9, beta2=0.999, eps=1e-8, masks=None, keep_scale=1.0):
    """One iteration of Algorithm 2's outer loop: forward, loss, backward, Adam on every W, b.
    ``state`` holds Adam moments (lists mW, vW, mb, vb) or None for zeros."""
    Ws = [_f64(W) for W in Ws]
    bs = [_f64(b) for b in bs]
    Zs, Ps, Xs = forward(g, X0, Ws, bs, masks, keep_scale)
    lo, G, pred, ncorrect, T = loss(Xs[-1], labels, train_mask)
    dWs, dbs = backward(g, Zs, Ps, Ws, G, masks, keep_scale)
    if state is None:
        state = dict(mW=[np.zeros_like(W) for W in Ws], vW=[np.zeros_like(W) for W in Ws],
                     mb=[np.zeros_like(b) for b in bs], vb=[np.zeros_like(b) for b in bs])
    newW, newb = [], []
    for l in range(len(Ws)):
        W2, state["mW"][l], state["vW"][l] = adam(Ws[l], dWs[l], state["mW"][l], state["vW"][l], t, lr, beta1, beta2, eps)
        b2, state["mb"][l], state["vb"][l] = adam(bs[l], dbs[l], state["mb"][l], state["vb"][l], t, lr, beta1, beta2, eps)
        newW.append(W2); newb.append(b2)
    return dict(loss=lo, logits=Xs[-1], pred=pred, n_correct=ncorrect, n_train=T, G=G,
                Zs=Zs, Ps=Ps, Xs=Xs, dW=dWs, db=dbs, W=newW, b=newb, state=state)


# ------------------------------------------------------------------------------ node reordering

# ------------------------------------------------------------------------------ GraphSAGE (mean) and GIN
# The paper evaluates these two architectures besides GCN (Section 5, "The Model and Datasets") and
# does not define them; the layers below are their textbook full-graph forms, built from the same
# aggregation and update steps as the GCN layer, on graphs made with norm="row" (mean of the
# neighbours, no self loops) and norm="none" (sum of the neighbours, no self loops).

def _adam_all(params, grads, state, t, lr, beta1, beta2, eps):
    if state is None:
        state = dict(m=[np.zeros_like(p) for p in params], v=[np.zeros_like(p) for p in params])
    new = []
    for i, (p, g) in enumerate(zip(params, grads)):
        p2, state["m"][i], state["v"][i] = adam(p, g, state["m"][i], state["v"][i], t, lr, beta1, beta2, eps)
        new.append(p2)
    return new, state


def sage_epoch(g_mean: Graph, X0, Ws_self, Ws_neigh, bs, labels, train_mask, state=None, t=1, lr=0.01,
               beta1=0.9, beta2=0.999, eps=1e-8):
    """One training iteration of a mean-aggregator GraphSAGE: H' = sigma(H W_self + (M H) W_neigh + b),
    M = D^-1 A the row mean over the neighbours, ReLU on every layer but the last; masked softmax
    cross-entropy; Adam.  Parameter order of the returned lists: W_self[0..L), W_neigh[0..L), b[0..L)."""
    L = len(Ws_self)
    Ws_self, Ws_neigh, bs = [_f64(w) for w in Ws_self], [_f64(w) for w in Ws_neigh], [_f64(b) for b in bs]
    Hs, MHs, Ps = [_f64(X0)], [], []
    for l in range(L):
        MH = aggregate(g_mean, Hs[-1])
        P = Hs[-1] @ Ws_self[l] + MH @ Ws_neigh[l] + bs[l]
        MHs.append(MH); Ps.append(P)
        Hs.append(P if l == L - 1 else np.maximum(P, 0.0))
    lo, G, pred, ncorrect, T = loss(Hs[-1], labels, train_mask)
    dS, dN, db = [None] * L, [None] * L, [None] * L
    Gout = G
    for l in range(L - 1, -1, -1):
        dP = Gout if l == L - 1 else Gout * (Ps[l] > 0)
        dS[l], dN[l], db[l] = Hs[l].T @ dP, MHs[l].T @ dP, dP.sum(axis=0)
        if l > 0:
            Gout = dP @ Ws_self[l].T + aggregate(g_mean, dP @ Ws_neigh[l].T, transposed=True)
    params, grads = Ws_self + Ws_neigh + bs, dS + dN + db
    new, state = _adam_all(params, grads, state, t, lr, beta1, beta2, eps)
    return dict(loss=lo, logits=Hs[-1], pred=pred, n_correct=ncorrect, G=G, grads=grads, params=new, state=state)


def gin_epoch(g_sum: Graph, X0, W1s, b1s, W2s, b2s, labels, train_mask, gin_eps=0.0, state=None, t=1, lr=0.01,
              beta1=0.9, beta2=0.999, eps=1e-8):
    """One training iteration of GIN: Z = (1 + gin_eps) H + A H (sum over the neighbours), then a
    two-layer perceptron H' = sigma(relu(Z W1 + b1) W2 + b2), sigma = ReLU on every layer but the last
    (gin_eps is a constant here).  Parameter order: W1[0..L), b1[0..L), W2[0..L), b2[0..L)."""
    L = len(W1s)
    W1s, b1s, W2s, b2s = ([_f64(x) for x in lst] for lst in (W1s, b1s, W2s, b2s))
    Hs, Zs, Ts, Ps = [_f64(X0)], [], [], []
    for l in range(L):
        Z = (1.0 + gin_eps) * Hs[-1] + aggregate(g_sum, Hs[-1])
        Tl = np.maximum(Z @ W1s[l] + b1s[l], 0.0)
        P = Tl @ W2s[l] + b2s[l]
        Zs.append(Z); Ts.append(Tl); Ps.append(P)
        Hs.append(P if l == L - 1 else np.maximum(P, 0.0))
    lo, G, pred, ncorrect, T = loss(Hs[-1], labels, train_mask)
    dW1, db1, dW2, db2 = [None] * L, [None] * L, [None] * L, [None] * L
    Gout = G
    for l in range(L - 1, -1, -1):
        dP = Gout if l == L - 1 else Gout * (Ps[l] > 0)
        dW2[l], db2[l] = Ts[l].T @ dP, dP.sum(axis=0)
        dT = (dP @ W2s[l].T) * (Ts[l] > 0)
        dW1[l], db1[l] = Zs[l].T @ dT, dT.sum(axis=0)
        if l > 0:
            dZ = dT @ W1s[l].T
            Gout = (1.0 + gin_eps) * dZ + aggregate(g_sum, dZ, transposed=True)
    params, grads = W1s + b1s + W2s + b2s, dW1 + db1 + dW2 + db2
    new, state = _adam_all(params, grads, state, t, lr, beta1, beta2, eps)
    return dict(loss=lo, logits=Hs[-1], pred=pred, n_correct=ncorrect, G=G, grads=grads, params=new, state=state)


def bandwidth(g: Graph, order=None) -> int:
    """b = max over stored entries (u,v) of p_v - p_u (Section 3.2.2); order[k] = node at position k."""
    pos = None
    if order is not None:
        pos = np.empty(g.n, dtype=np.int64)
        pos[np.asarray(order, dtype=np.int64)] = np.arange(g.n, dtype=np.int64)
    L = lib()
    L.oracle_bandwidth.restype = C.c_int64
    return int(L.oracle_bandwidth(C.c_int64(g.n), _p(g.rowptr, C.c_int64), _p(g.col, C.c_int32), _p(pos, C.c_int64)))


def rcm(g: Graph):
    """Reverse Cuthill-McKee order of a symmetric graph: order[k] = node at position k."""
    order = np.zeros(g.n, dtype=np.int64)
    lib().oracle_rcm(C.c_int64(g.n), _p(g.rowptr, C.c_int64), _p(g.col, C.c_int32), _p(order, C.c_int64))
    return order


def pipeline_stages(n: int, b: int) -> int:
    """ceil(2n / (n - b)) (Proposition 3.5 and the stage count of the evaluation)."""
    L = lib()
    L.oracle_pipeline_stages.restype = C.c_int64
    return int(L.oracle_pipeline_stages(C.c_int64(n), C.c_int64(b)))
