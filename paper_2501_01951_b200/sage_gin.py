"""Buffer plumbing for the two other architectures the paper's evaluation names (Section 5, "The Model
and Datasets"): mean-aggregator GraphSAGE and GIN, full-graph training.  The paper does not define
them; the layers are their textbook forms, built from the same C-ABI steps as the GCN layer:

  GraphSAGE (mean):  H' = sigma([H | M H] [W_self; W_neigh] + b),  M = D^-1 A on a graph made with
                     GRAPH_NORM_ROW (no self loops);
  GIN:               H' = sigma(relu(((1 + eps) H + A H) W1 + b1) W2 + b2),  A on a graph made with
                     GRAPH_NORM_NONE (no self loops); the (1 + eps) H term is the aggregation
                     epilogue's residual.

As in ``train.py`` nothing is computed here: every value comes out of a kernel of ``libmixgcn.so``
(``spmm``, ``gemm``, ``colsum``, ``loss_softmax_xent``, ``adam_step``).
"""
from __future__ import annotations

import torch

from . import binding as mg


def round4(x: int) -> int:
    return (x + 3) // 4 * 4


class _Base:
    def __init__(self, ctx, graph, dims, precision):
        self.ctx, self.g, self.precision = ctx, graph, precision
        self.dims = tuple(int(d) for d in dims)
        self.L = len(self.dims) - 1
        self.n = graph.n
        self.device = torch.device("cuda", ctx.device)
        self.ld = [round4(d) for d in self.dims]
        self.loss = torch.zeros(1, dtype=torch.float32, device=self.device)
        self.pred = torch.zeros(self.n, dtype=torch.int32, device=self.device)
        self.n_correct = torch.zeros(1, dtype=torch.int64, device=self.device)
        self.params, self.grads, self.m, self.v = [], [], [], []

    def _z(self, r, c):
        return torch.zeros((r, c), dtype=torch.float32, device=self.device)

    def _set_params(self, tensors):
        self.params = [t.to(self.device, torch.float32).contiguous().clone() for t in tensors]
        self.grads = [torch.zeros_like(t) for t in self.params]
        self.m = [torch.zeros_like(t) for t in self.params]
        self.v = [torch.zeros_like(t) for t in self.params]

    def compute_loss(self):
        mg.loss_softmax_xent(self.ctx, self.logits, self.labels, self.train_mask, self.loss, dlogits=self.logits,
                             pred=self.pred, n_correct=self.n_correct, C_=self.dims[-1])

    def step(self, t, lr=0.01, beta1=0.9, beta2=0.999, eps=1e-8):
        mg.adam_step(self.ctx, self.params, self.grads, self.m, self.v, t, lr, beta1, beta2, eps)

    def epoch(self, t, lr=0.01):
        self.forward()
        self.compute_loss()
        self.backward()
        self.step(t, lr)


class SageTrainer(_Base):
    """Mean-aggregator GraphSAGE.  ``graph`` must carry row-mean values (GRAPH_NORM_ROW, no self loops).
    Layer l keeps S_l = [H_l | M H_l] (n x 2 ld_l): the left half is written by the layer below (or is
    the input), the right half by the aggregation, and one product with W_l = [W_self; W_neigh]
    (2 d_l x d_{l+1}) does the update."""

    def __init__(self, ctx, graph, dims, precision=mg.PREC_FP32):
        super().__init__(ctx, graph, dims, precision)
        n, L, ld = self.n, self.L, self.ld
        self.S = [self._z(n, 2 * ld[l]) for l in range(L)]
        self.logits = self._z(n, ld[L])
        wmax = max(ld[1:L]) if L >= 2 else 4
        self.dS = self._z(n, 2 * wmax)                     # gradient w.r.t. [H_l | M H_l]
        self.Ga, self.Gb = self._z(n, wmax), self._z(n, wmax)

    def set_params(self, Ws_self, Ws_neigh, bs):
        """Parameter order: W_cat[0..L) (rows [W_self; W_neigh]), b[0..L)."""
        cats = []
        for l in range(self.L):
            W = torch.zeros(2 * self.ld[l], self.dims[l + 1])
            W[: self.dims[l]] = Ws_self[l]
            W[self.ld[l]: self.ld[l] + self.dims[l]] = Ws_neigh[l]
            cats.append(W)
        self._set_params(cats + list(bs))

    def set_inputs(self, X0, labels, train_mask):
        """X0: n x ld[0] device tensor (pads zero); it is copied once into the left half of S_0."""
        self.S[0][:, : self.ld[0]].copy_(X0)
        self.labels, self.train_mask = labels, train_mask

    def forward(self):
        L, ld = self.L, self.ld
        for l in range(L):
            S, d = self.S[l], ld[l]
            mg.spmm(self.ctx, self.g, S[:, :d], S[:, d:], self.dims[l])
            last = l == L - 1
            out = self.logits if last else self.S[l + 1][:, : ld[l + 1]]
            mg.gemm(self.ctx, self.precision, False, False, self.n, self.dims[l + 1], 2 * d, S, self.params[l], out,
                    epi=mg.make_epilogue(bias=self.params[L + l], relu=not last))

    def backward(self):
        L, ld = self.L, self.ld
        G = self.logits                                     # gradient w.r.t. the layer's pre-activation
        for l in range(L - 1, -1, -1):
            d, dout = ld[l], self.dims[l + 1]
            mg.colsum(self.ctx, G, self.grads[L + l], dout)
            mg.gemm(self.ctx, self.precision, True, False, 2 * d, dout, self.n, self.S[l], G, self.grads[l])
            if l > 0:
                dS = self.dS[:, : 2 * d]
                mg.gemm(self.ctx, self.precision, False, True, self.n, 2 * d, dout, G, self.params[l], dS)
                Gn = (self.Ga if (L - 1 - l) % 2 == 0 else self.Gb)[:, :d]   # the two buffers alternate
                # G_in = relu'(H_l) * (dS_left + M^T dS_right): residual and gate in the aggregation's epilogue
                mg.spmm(self.ctx, self.g, dS[:, d:], Gn, self.dims[l], transposed=True,
                        epi=mg.make_epilogue(residual=dS[:, :d], residual_scale=1.0, gate=self.S[l][:, :d], gate_scale=1.0))
                G = Gn


class GinTrainer(_Base):
    """GIN with a two-layer perceptron per layer.  ``graph`` must carry unit values (GRAPH_NORM_NONE, no
    self loops); ``gin_eps`` is the constant eps of the (1 + eps) self term."""

    def __init__(self, ctx, graph, dims, hidden, precision=mg.PREC_FP32, gin_eps=0.0):
        super().__init__(ctx, graph, dims, precision)
        n, L, ld = self.n, self.L, self.ld
        self.hidden, self.ldh, self.gin_eps = int(hidden), round4(hidden), float(gin_eps)
        self.H = [None] + [self._z(n, ld[l]) for l in range(1, L)]
        self.Z = [self._z(n, ld[l]) for l in range(L)]
        self.T = [self._z(n, self.ldh) for l in range(L)]
        self.logits = self._z(n, ld[L])
        wmax = max(ld[1:L]) if L >= 2 else 4
        self.dT, self.dZ = self._z(n, self.ldh), self._z(n, wmax)
        self.Ga, self.Gb = self._z(n, wmax), self._z(n, wmax)

    def set_params(self, W1s, b1s, W2s, b2s):
        """Parameter order: W1[0..L), b1[0..L), W2[0..L), b2[0..L)."""
        self._set_params(list(W1s) + list(b1s) + list(W2s) + list(b2s))

    def set_inputs(self, X0, labels, train_mask):
        self.H[0], self.labels, self.train_mask = X0, labels, train_mask

    def forward(self):
        L = self.L
        for l in range(L):
            H, d = self.H[l], self.dims[l]
            mg.spmm(self.ctx, self.g, H, self.Z[l], d, epi=mg.make_epilogue(residual=H, residual_scale=1.0 + self.gin_eps))
            mg.gemm(self.ctx, self.precision, False, False, self.n, self.hidden, d, self.Z[l], self.params[l], self.T[l],
                    epi=mg.make_epilogue(bias=self.params[L + l], relu=True))
            last = l == L - 1
            out = self.logits if last else self.H[l + 1]
            mg.gemm(self.ctx, self.precision, False, False, self.n, self.dims[l + 1], self.hidden, self.T[l],
                    self.params[2 * L + l], out, epi=mg.make_epilogue(bias=self.params[3 * L + l], relu=not last))

    def backward(self):
        L = self.L
        G = self.logits
        for l in range(L - 1, -1, -1):
            d, dout, h = self.dims[l], self.dims[l + 1], self.hidden
            mg.colsum(self.ctx, G, self.grads[3 * L + l], dout)
            mg.gemm(self.ctx, self.precision, True, False, h, dout, self.n, self.T[l], G, self.grads[2 * L + l])
            # dT = relu'(T) * (dP W2^T)
            mg.gemm(self.ctx, self.precision, False, True, self.n, h, dout, G, self.params[2 * L + l], self.dT,
                    epi=mg.make_epilogue(gate=self.T[l], gate_scale=1.0))
            mg.colsum(self.ctx, self.dT, self.grads[L + l], h)
            mg.gemm(self.ctx, self.precision, True, False, d, h, self.n, self.Z[l], self.dT, self.grads[l])
            if l > 0:
                dZ = self.dZ[:, : self.ld[l]]
                mg.gemm(self.ctx, self.precision, False, True, self.n, d, h, self.dT, self.params[l], dZ)
                Gn = (self.Ga if (L - 1 - l) % 2 == 0 else self.Gb)[:, : self.ld[l]]   # the two buffers alternate
                # G_in = relu'(H_l) * ((1 + eps) dZ + A^T dZ)
                mg.spmm(self.ctx, self.g, dZ, Gn, d, transposed=True,
                        epi=mg.make_epilogue(residual=dZ, residual_scale=1.0 + self.gin_eps, gate=self.H[l], gate_scale=1.0))
                G = Gn
