"""Buffer plumbing for one full-graph GCN training iteration (the loop body of Algorithm 2).

``GcnTrainer`` owns torch device buffers and calls the C-ABI in the order the algorithm
gives -- for each layer aggregation+update (``layer_fwd``), then the loss, the backward pass
(``layer_bwd``, last layer first) and the weight update (``adam_step``).  It performs no
arithmetic itself: every value is produced by a kernel of ``libmixgcn.so``.
"""
from __future__ import annotations

import torch

from . import binding as mg


def round4(x: int) -> int:
    return (x + 3) // 4 * 4


def round8(x: int) -> int:
    return (x + 7) // 8 * 8


class GcnTrainer:
    def __init__(self, ctx: mg.Ctx, graph: mg.Graph, dims, precision=mg.PREC_FP32, order=mg.ORDER_AUTO,
                 n_chunks=0, fuse_gate=True, keep_scale=1.0, device=None, row_sparse="auto",
                 train_rows_only=False, row_plans=True, cache_first_aggregation=False, lp_copies=True, saved_lp_only=True, sign_bitmaps=True):
        self.ctx, self.g = ctx, graph
        self.dims = tuple(int(d) for d in dims)
        self.L = len(self.dims) - 1
        self.n = graph.n
        self.device = torch.device("cuda", ctx.device) if device is None else device
        self.ld = [round4(d) for d in self.dims]
        self.fuse_gate = fuse_gate
        self.row_sparse = row_sparse          # "auto" | number of layers (from the top) whose backward gets a row mask
        self.row_masks = None
        # opt-in: the last layer's output, the loss and its gradient on train rows only (needs a
        # row-sparse backward for the last layer; predictions exist for train rows only)
        self.train_rows_only = bool(train_rows_only)
        # row plans: the row-sparse backward on restricted matrices built once per (graph, train mask);
        # False = the masks are tested inside the aggregation kernel every iteration
        self.use_row_plans = bool(row_plans)
        # opt-in: keep A_hat X^(0) of an agg-first first layer across iterations (features and graph are
        # the same every epoch); the paper recomputes it
        self.cache_first_aggregation = bool(cache_first_aggregation)
        self._first_aggregation_valid = False
        n, L = self.n, self.L
        orders = order if isinstance(order, (list, tuple)) else [order] * L
        self.descs, self.orders = [], []
        for l in range(L):
            flags = (mg.LAYER_RELU if l < L - 1 else 0) | (mg.LAYER_FIRST if l == 0 else 0)
            if fuse_gate:
                if l >= 1:
                    flags |= mg.LAYER_GATE_GIN      # apply layer l-1's ReLU mask while producing G_in
                if l < L - 1:
                    flags |= mg.LAYER_GOUT_GATED    # ... so that layer l receives a gated G_out
            d = mg.layer_desc(self.dims[l], self.dims[l + 1], self.ld[l], self.ld[l + 1], 4, orders[l], precision,
                              flags, keep_scale if l < L - 1 else 1.0, keep_scale if l >= 1 else 1.0, n_chunks)
            o, cols = mg.layer_plan(d)
            d.ld_saved = round4(cols)
            d.order = o
            self.descs.append(d)
            self.orders.append(o)
        z = lambda r, c: torch.zeros((r, c), dtype=torch.float32, device=self.device)
        self.X = [None] + [z(n, self.ld[l]) for l in range(1, L + 1)]
        self.saved = [z(n, self.descs[l].ld_saved) for l in range(L)]
        # gradient buffers: the logits' gradient is written over the logits; the input gradients of
        # layers L-1, L-2, ... alternate between GA and GB (GB lives in the logits buffer when it fits)
        self.G = [None] * (L + 1)
        self.G[L] = self.X[L]
        pool = []
        if L >= 2:
            wmax = max(self.ld[1:L])
            pool.append(z(n, wmax))
            if L >= 3:
                if self.ld[L] >= wmax:
                    pool.append(self.X[L])
                else:
                    pool.append(z(n, wmax))
        for i, l in enumerate(range(L - 1, 0, -1)):
            buf = pool[i % 2]
            self.G[l] = buf.view(-1)[: n * self.ld[l]].view(n, self.ld[l])
        # BF16 products: bf16 companions of the activations, written by the kernels that produce them
        # (buffers only; lp_copies=False leaves them out and the library converts operands on the fly)
        self.lp = []
        self.saved_lp = [None] * L       # bf16 copy of saved[l], where there is one
        # with bf16 companions an agg-first layer's A_hat X is read only as bf16: its fp32 copy need not be written
        # (set per iteration in forward(): only where the backward is dense and nothing else reads `saved`)
        self.saved_lp_only = bool(saved_lp_only) and precision == mg.PREC_BF16 and lp_copies and n_chunks <= 1
        if precision == mg.PREC_BF16 and lp_copies:
            zb = lambda c: torch.zeros((n, round8(c)), dtype=torch.bfloat16, device=self.device)
            keep = lambda t: (self.lp.append(t), t)[1]
            x_lp = [None] * (L + 1)      # copy of X[l], wanted where layer l multiplies X[l] itself (upd-first)
            g_lp = [None] * (L + 1)      # copy of G[l], wanted where layer l-1 multiplies G[l] itself (agg-first, gated on arrival)
            for l in range(1, L):
                if self.orders[l] == mg.ORDER_UPD_FIRST:
                    x_lp[l] = keep(zb(self.dims[l]))
                if self.orders[l - 1] == mg.ORDER_AGG_FIRST and fuse_gate:
                    g_lp[l] = keep(zb(self.dims[l]))
            for l, d in enumerate(self.descs):
                cols = self.dims[l] if self.orders[l] == mg.ORDER_AGG_FIRST else self.dims[l + 1]
                t = keep(zb(cols))
                self.saved_lp[l] = t
                d.saved_lp, d.ld_saved_lp = t.data_ptr(), t.stride(0)
                d.ld_in_lp, d.ld_out_lp = round8(self.dims[l]), round8(self.dims[l + 1])
                if x_lp[l] is not None:
                    d.x_in_lp = x_lp[l].data_ptr()
                if x_lp[l + 1] is not None:
                    d.x_out_lp = x_lp[l + 1].data_ptr()
                if g_lp[l + 1] is not None:
                    d.g_out_lp = g_lp[l + 1].data_ptr()
                if g_lp[l] is not None:
                    d.g_in_lp = g_lp[l].data_ptr()
        # Sign bitmaps of the hidden activations (one bit per element): written by the forward kernel that produces
        # X[l], read by the backward kernel that gates the gradient w.r.t. X[l] instead of the fp32 tensor
        self.xbits = [None] * (L + 1)
        if fuse_gate and sign_bitmaps:
            for l in range(1, L):
                # where a dense product produces X[l] (agg-first layer l-1) its epilogue writes the bitmap for free;
                # an aggregation would need one more pass over X[l], which costs what the bitmap saves
                if self.orders[l - 1] != mg.ORDER_AGG_FIRST:
                    continue
                t = torch.zeros((n, (self.dims[l] + 31) // 32), dtype=torch.int32, device=self.device)
                self.xbits[l] = t
                self.descs[l - 1].x_out_bits, self.descs[l - 1].ld_out_bits = t.data_ptr(), t.stride(0)
                self.descs[l].x_in_bits, self.descs[l].ld_in_bits = t.data_ptr(), t.stride(0)
        self.loss = torch.zeros(1, dtype=torch.float32, device=self.device)
        self.pred = torch.zeros(n, dtype=torch.int32, device=self.device)
        self.n_correct = torch.zeros(1, dtype=torch.int64, device=self.device)
        self.W = self.b = self.dW = self.db = None
        self.masks = [None] * L

    # -- parameters -----------------------------------------------------------------------------
    def set_params(self, Ws, bs):
        dev = self.device
        self.W = [w.to(dev, torch.float32).contiguous().clone() for w in Ws]
        self.b = [b.to(dev, torch.float32).contiguous().clone() for b in bs]
        self.dW = [torch.zeros_like(w) for w in self.W]
        self.db = [torch.zeros_like(b) for b in self.b]
        self.mW = [torch.zeros_like(w) for w in self.W]
        self.vW = [torch.zeros_like(w) for w in self.W]
        self.mb = [torch.zeros_like(b) for b in self.b]
        self.vb = [torch.zeros_like(b) for b in self.b]

    def set_inputs(self, X0, labels, train_mask, drop_masks=None):
        """X0: n x ld[0] device tensor (row-major, pads zero); labels int32; train_mask uint8."""
        assert X0.shape == (self.n, self.ld[0]) and X0.stride(1) == 1
        self.X[0], self.labels, self.train_mask = X0, labels, train_mask
        if drop_masks is not None:
            self.masks = list(drop_masks) + [None] * (self.L - len(drop_masks))
        self._first_aggregation_valid = False
        self.descs[0].flags &= ~mg.LAYER_SAVED_IS_VALID
        self._plan_row_sparsity()

    def configure(self, train_rows_only=None, cache_first_aggregation=None, row_sparse=None):
        """Switch the opt-in variants of an existing trainer (buffers and inputs stay); rebuilds the row plans."""
        if train_rows_only is not None:
            self.train_rows_only = bool(train_rows_only)
        if cache_first_aggregation is not None:
            self.cache_first_aggregation = bool(cache_first_aggregation)
            self._first_aggregation_valid = False
        if row_sparse is not None:
            self.row_sparse = row_sparse
        self._plan_row_sparsity()

    def _plan_row_sparsity(self):
        """The loss gradient is non-zero on train rows only; one aggregation later on their neighbours
        only.  Hand those row masks to layer_bwd for the top `levels` layers (plumbing: the masks are
        the train mask and byte arrays the library fills)."""
        n, L = self.n, self.L
        n_train = int(self.train_mask.sum().item())
        frac = n_train / max(n, 1)
        levels = self.row_sparse
        if levels == "auto":
            mean_entries = self.g.nnz / max(n, 1)
            levels = 0 if frac >= 0.25 else (2 if frac * mean_entries < 0.5 else 1)
        if self.train_rows_only and self.row_sparse == "auto" and levels == 0:
            levels = 1
        levels = max(0, min(int(levels), L))
        self.row_sparse_levels = levels
        self.row_masks = [None] * (L + 1)
        self.row_plans = [None] * L
        for d in self.descs:
            d.gout_row_mask, d.gout_row_count, d.gin_row_mask, d.gout_plan = None, 0, None, None
            d.flags &= ~(mg.LAYER_OUT_ROWS_ONLY | mg.LAYER_GIN_ROWS_ONLY)
        if self.train_rows_only:
            if levels == 0 or n_train == 0 or self.masks[L - 1] is not None:
                raise ValueError("train_rows_only needs a row-sparse backward (row_sparse >= 1), a non-empty "
                                 "train mask and no dropout mask on the last layer")
            self.descs[L - 1].flags |= mg.LAYER_OUT_ROWS_ONLY
        if levels == 0:
            return
        self.row_masks[L] = self.train_mask
        for i in range(levels):
            l = L - 1 - i                                 # layer whose backward receives row_masks[l + 1]
            d = self.descs[l]
            d.gout_row_mask = self.row_masks[l + 1].data_ptr()
            if self.use_row_plans and n_train > 0:
                # everything that depends on the graph and the mask only, computed once
                plan = mg.rowplan_create(self.ctx, self.g, self.row_masks[l + 1])
                self.row_plans[l] = plan
                d.gout_plan = plan.h
                d.gout_row_count = plan.in_count
                if l > 0 and i + 1 < levels:
                    self.row_masks[l] = plan.out_row_mask()
                    d.flags |= mg.LAYER_GIN_ROWS_ONLY     # the layer below gathers exactly these rows of G_in
            else:
                d.gout_row_count = n_train if i == 0 else 0
                if l > 0 and i + 1 < levels:
                    self.row_masks[l] = torch.zeros(n, dtype=torch.uint8, device=self.device)
                    d.gin_row_mask = self.row_masks[l].data_ptr()

    # -- the iteration --------------------------------------------------------------------------
    def last_layer_takes_the_loss(self):
        """Whether forward_and_loss() hands the last layer and the loss to ONE library call (which takes the loss
        where the logits are produced, without writing them, wherever its kernels can)."""
        return self.masks[self.L - 1] is None and not self.train_rows_only

    def forward_and_loss(self):
        """forward() + compute_loss() with the same results; X[L] then holds the gradient w.r.t. the logits."""
        if not self.last_layer_takes_the_loss():
            self.forward()
            self.compute_loss()
            return
        L = self.L
        self.forward(upto=L - 1)
        d = self.descs[L - 1]
        d.flags &= ~(mg.LAYER_SAVED_LP_ONLY | mg.LAYER_SAVED_IS_VALID)
        # rows the backward never reads need no zeros (same rule as compute_loss)
        leave = self.row_plans[L - 1] is not None
        if leave:
            mg.ctx_set_option(self.ctx, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 2)
        try:
            mg.layer_fwd_loss(self.ctx, self.g, d, self.X[L - 1], self.W[L - 1], self.b[L - 1], self.saved[L - 1],
                              self.X[L], self.labels, self.train_mask, self.loss, self.pred, self.n_correct)
        finally:
            if leave:
                mg.ctx_set_option(self.ctx, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 0)
        if L == 1:
            self._first_aggregation_valid = self.orders[0] == mg.ORDER_AGG_FIRST

    def forward(self, upto=None):
        d0 = self.descs[0]
        reuse = self.cache_first_aggregation and self._first_aggregation_valid and self.orders[0] == mg.ORDER_AGG_FIRST
        d0.flags = (d0.flags | mg.LAYER_SAVED_IS_VALID) if reuse else (d0.flags & ~mg.LAYER_SAVED_IS_VALID)
        for l in range(self.L if upto is None else upto):
            d = self.descs[l]
            lp_only = (self.saved_lp_only and self.orders[l] == mg.ORDER_AGG_FIRST and not d.gout_row_mask and not d.gout_plan
                       and not (d.flags & (mg.LAYER_OUT_ROWS_ONLY | mg.LAYER_SAVED_IS_VALID))
                       and not (l == 0 and self.cache_first_aggregation))
            d.flags = (d.flags | mg.LAYER_SAVED_LP_ONLY) if lp_only else (d.flags & ~mg.LAYER_SAVED_LP_ONLY)
            mg.layer_fwd(self.ctx, self.g, d, self.X[l], self.W[l], self.b[l], self.masks[l],
                         self.saved[l], self.X[l + 1])
        # saved[0] now holds A_hat X^(0) unless the single layer of a one-layer model also restricted it to train rows
        self._first_aggregation_valid = self.orders[0] == mg.ORDER_AGG_FIRST and not (d0.flags & mg.LAYER_OUT_ROWS_ONLY)

    def aggregation_of(self, l):
        """The tensor that holds A_hat X^(l) after forward() for an agg-first layer: `saved[l]`, or its bf16
        copy where only that was written."""
        return self.saved_lp[l] if self.descs[l].flags & mg.LAYER_SAVED_LP_ONLY else self.saved[l]

    def compute_loss(self):
        if self.train_rows_only:
            mg.ctx_set_option(self.ctx, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 1)
            try:
                mg.loss_softmax_xent(self.ctx, self.X[self.L], self.labels, self.train_mask, self.loss,
                                     dlogits=self.X[self.L], pred=self.pred, n_correct=self.n_correct, C_=self.dims[-1])
            finally:
                mg.ctx_set_option(self.ctx, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 0)
            return
        if self.row_plans[self.L - 1] is not None:
            # the last layer's backward reads the plan's (train) rows of the gradient only: no need to
            # write zeros into the other rows; the logits of every node are still read for `pred`
            mg.ctx_set_option(self.ctx, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 2)
            try:
                mg.loss_softmax_xent(self.ctx, self.X[self.L], self.labels, self.train_mask, self.loss,
                                     dlogits=self.X[self.L], pred=self.pred, n_correct=self.n_correct, C_=self.dims[-1])
            finally:
                mg.ctx_set_option(self.ctx, mg.OPT_LOSS_TRAIN_ROWS_ONLY, 0)
            return
        mg.loss_softmax_xent(self.ctx, self.X[self.L], self.labels, self.train_mask, self.loss,
                             dlogits=self.X[self.L], pred=self.pred, n_correct=self.n_correct, C_=self.dims[-1])

    def backward(self, on_layer=None):
        """on_layer(l, "before" | "after"), if given, is called around each layer's backward call (tests
        use it to look at a layer's operands before the call consumes them)."""
        for l in range(self.L - 1, -1, -1):
            d = self.descs[l]
            if d.gout_row_mask and d.gout_row_count == 0 and self.row_masks[l + 1] is not self.train_mask:
                # A row mask the library reported one layer up.  It depends on the graph and the train
                # mask only, so its count is taken once (a stream synchronisation) and kept; with the
                # count layer_bwd can run its dense products on the compacted rows.
                d.gout_row_count = mg.count_rows(self.ctx, self.row_masks[l + 1])
            if on_layer is not None:
                on_layer(l, "before")
            mg.layer_bwd(self.ctx, self.g, d, self.X[l], self.saved[l], self.X[l + 1], self.masks[l],
                         self.W[l], self.G[l + 1], self.G[l] if l > 0 else None, self.dW[l], self.db[l])
            if on_layer is not None:
                on_layer(l, "after")

    def step(self, t, lr=0.01, beta1=0.9, beta2=0.999, eps=1e-8):
        mg.adam_step(self.ctx, self.W + self.b, self.dW + self.db, self.mW + self.mb, self.vW + self.vb, t,
                     lr, beta1, beta2, eps)

    def epoch(self, t, lr=0.01):
        self.forward_and_loss()
        self.backward()
        self.step(t, lr)
