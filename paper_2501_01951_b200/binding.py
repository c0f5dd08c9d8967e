"""ctypes binding of ``include/mixgcn.h`` -- argument marshalling only.

Every function here has the name of the C entry point without the ``mixgcn_`` prefix, takes
torch tensors (device memory owned by the caller) and forwards raw pointers, sizes and the
current torch CUDA stream.  No arithmetic of the method happens in Python.  Importing this
module without a built ``libmixgcn.so`` raises: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MIXGCN_LIBRARY=debug loads the bounds-checked build of the same sources (libmixgcn_debug.so) instead
_VARIANT = os.environ.get("MIXGCN_LIBRARY", "")
if _VARIANT not in ("", "debug"):
    raise ImportError(f"MIXGCN_LIBRARY={_VARIANT!r}: the only other build is 'debug'")
LIB_PATH = os.path.join(_HERE, "libmixgcn_debug.so" if _VARIANT == "debug" else "libmixgcn.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2501_01951_b200.build` "
        "(there is no CPU or PyTorch fallback for this library)")

lib = C.CDLL(LIB_PATH)

OK, EINVAL, ENOMEM, ECUDA, EUNSUPPORTED, EBADGRAPH, ETIMEOUT, EDEVICE = range(8)
GRAPH_SYMMETRISE, GRAPH_ADD_SELF_LOOPS, GRAPH_EDGES_ON_DEVICE = 1, 2, 4
GRAPH_NORM_ROW, GRAPH_NORM_NONE = 8, 16
PREC_FP32, PREC_TF32, PREC_BF16 = 0, 1, 2
ORDER_AUTO, ORDER_AGG_FIRST, ORDER_UPD_FIRST = 0, 1, 2
LAYER_RELU, LAYER_FIRST, LAYER_GATE_GIN, LAYER_GOUT_GATED, LAYER_OUT_ROWS_ONLY, LAYER_GIN_ROWS_ONLY = 1, 2, 4, 8, 16, 32
LAYER_SAVED_IS_VALID = 64
LAYER_SAVED_LP_ONLY = 128
N_PHASES = 7
PHASES = ("spmm", "gemm", "elementwise", "loss", "adam", "graph", "spmm_sparse")
PRECISIONS = {"fp32": PREC_FP32, "tf32": PREC_TF32, "bf16": PREC_BF16}

# every symbol include/mixgcn.h declares
SYMBOLS = (
    "mixgcn_status_string", "mixgcn_last_error", "mixgcn_ctx_create", "mixgcn_ctx_destroy",
    "mixgcn_ctx_reserve", "mixgcn_ctx_poll_status", "mixgcn_ctx_profile_enable", "mixgcn_ctx_profile_read",
    "mixgcn_graph_create", "mixgcn_graph_create_from_csr", "mixgcn_graph_info", "mixgcn_graph_export",
    "mixgcn_graph_export_schedule", "mixgcn_graph_destroy", "mixgcn_spmm", "mixgcn_gemm",
    "mixgcn_layer_plan", "mixgcn_layer_fwd", "mixgcn_layer_bwd", "mixgcn_loss_softmax_xent",
    "mixgcn_adam_step", "mixgcn_train_step_host", "mixgcn_loss_softmax_xent_noalloc", "mixgcn_ctx_set_option",
    "mixgcn_graph_bandwidth", "mixgcn_graph_rcm", "mixgcn_pipeline_stages", "mixgcn_graph_create_permuted",
    "mixgcn_count_rows", "mixgcn_rowplan_create", "mixgcn_rowplan_destroy", "mixgcn_rowplan_info",
    "mixgcn_rowplan_export", "mixgcn_spmm_rowplan", "mixgcn_colsum", "mixgcn_ctx_gemm_paths",
    "mixgcn_train_step_host_prefetch", "mixgcn_probe_gather", "mixgcn_spmm_sampled", "mixgcn_mask_pack",
    "mixgcn_build_info", "mixgcn_debug_poke_col", "mixgcn_layer_fwd_loss",
)


class Epilogue(C.Structure):
    _fields_ = [("bias", C.c_void_p), ("relu", C.c_int32), ("drop_mask", C.c_void_p),
                ("keep_scale", C.c_float), ("gate", C.c_void_p), ("ld_gate", C.c_int64),
                ("gate_scale", C.c_float), ("residual", C.c_void_p), ("ld_residual", C.c_int64),
                ("residual_scale", C.c_float), ("gate_bits", C.c_void_p), ("ld_gate_bits", C.c_int64),
                ("sign_bits", C.c_void_p), ("ld_sign_bits", C.c_int64)]


class LayerDesc(C.Structure):
    _fields_ = [("d_in", C.c_int32), ("d_out", C.c_int32), ("ld_in", C.c_int64), ("ld_out", C.c_int64),
                ("ld_saved", C.c_int64), ("order", C.c_int32), ("precision", C.c_int32),
                ("flags", C.c_uint32), ("keep_scale", C.c_float), ("in_scale", C.c_float),
                ("n_chunks", C.c_int32), ("gout_row_mask", C.c_void_p), ("gout_row_count", C.c_int64),
                ("gin_row_mask", C.c_void_p), ("gout_plan", C.c_void_p),
                ("saved_lp", C.c_void_p), ("ld_saved_lp", C.c_int64), ("x_in_lp", C.c_void_p), ("ld_in_lp", C.c_int64),
                ("x_out_lp", C.c_void_p), ("ld_out_lp", C.c_int64), ("g_out_lp", C.c_void_p), ("g_in_lp", C.c_void_p),
                ("x_out_bits", C.c_void_p), ("ld_out_bits", C.c_int64), ("x_in_bits", C.c_void_p), ("ld_in_bits", C.c_int64)]


lib.mixgcn_status_string.restype = C.c_char_p
lib.mixgcn_last_error.restype = C.c_char_p
for _name in SYMBOLS[2:]:
    getattr(lib, _name).restype = C.c_int


class MixgcnError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        msg = lib.mixgcn_last_error().decode()
        super().__init__(f"{lib.mixgcn_status_string(status).decode()} ({status}): {msg}")


def _check(status: int):
    if status != OK:
        raise MixgcnError(status)


def _ptr(t):
    """Device or host pointer of a tensor (None -> NULL)."""
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t, dtype, name):
    if not t.is_cuda or t.dtype != dtype:
        raise TypeError(f"{name}: expected a CUDA tensor of {dtype}, got {t.dtype} on {t.device}")
    return t


def _mat(t, name):
    """2-D fp32 CUDA tensor with unit column stride -> (tensor, ld)."""
    _dev(t, torch.float32, name)
    if t.dim() != 2 or t.stride(1) != 1:
        raise TypeError(f"{name}: expected a row-major 2-D tensor")
    return t, t.stride(0)


# ------------------------------------------------------------------------------ context

class Ctx:
    def __init__(self, device: int = 0):
        self.h = C.c_void_p()
        _check(lib.mixgcn_ctx_create(C.byref(self.h), C.c_int(device)))
        self.device = device

    def close(self):
        if self.h:
            lib.mixgcn_ctx_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ctx_create(device: int = 0) -> Ctx:
    return Ctx(device)


def ctx_reserve(ctx: Ctx, nbytes: int):
    _check(lib.mixgcn_ctx_reserve(ctx.h, C.c_int64(nbytes)))


def ctx_poll_status(ctx: Ctx, raise_on_error: bool = True) -> int:
    code = C.c_int32(0)
    st = lib.mixgcn_ctx_poll_status(ctx.h, C.byref(code))
    if raise_on_error:
        _check(st)
    return code.value


OPT_SPMM_SLICE_COLS = 1
OPT_LOSS_TRAIN_ROWS_ONLY = 2
OPT_DEBUG_WAIT_LIMIT = 3
OPT_DEBUG_DROP_LOAD = 4
OPT_GEMM_CTA_PAIRS = 5


def ctx_set_option(ctx: Ctx, option: int, value: int):
    _check(lib.mixgcn_ctx_set_option(ctx.h, C.c_int32(option), C.c_int64(value)))


def ctx_gemm_paths(ctx: Ctx) -> dict:
    """Dense products served so far by the fp32 FMA kernel, the tcgen05 TF32 kernels, the tcgen05 BF16 kernels."""
    counts = (C.c_int64 * 4)()
    _check(lib.mixgcn_ctx_gemm_paths(ctx.h, counts))
    return dict(simt=int(counts[0]), tc_tf32=int(counts[1]), tc_bf16=int(counts[2]), cta_pairs=int(counts[3]))


def ctx_profile_enable(ctx: Ctx, enable: bool = True):
    _check(lib.mixgcn_ctx_profile_enable(ctx.h, C.c_int(int(enable))))


def ctx_profile_read(ctx: Ctx):
    """-> ({phase: ms}, {phase: launches}, launches_total)."""
    ms = (C.c_double * N_PHASES)()
    ln = (C.c_int64 * N_PHASES)()
    tot = C.c_int64(0)
    _check(lib.mixgcn_ctx_profile_read(ctx.h, ms, ln, C.byref(tot)))
    return dict(zip(PHASES, list(ms))), dict(zip(PHASES, list(ln))), tot.value


# ------------------------------------------------------------------------------ graph

class Graph:
    def __init__(self, ctx: Ctx, handle):
        self.ctx, self.h = ctx, handle
        n, nnz, md, sym = C.c_int64(), C.c_int64(), C.c_int32(), C.c_int32()
        _check(lib.mixgcn_graph_info(self.h, C.byref(n), C.byref(nnz), C.byref(md), C.byref(sym)))
        self.n, self.nnz, self.max_deg, self.symmetric = n.value, nnz.value, md.value, bool(sym.value)

    def close(self):
        if self.h:
            lib.mixgcn_graph_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def graph_create(ctx: Ctx, n: int, src: torch.Tensor, dst: torch.Tensor,
                 flags: int = GRAPH_SYMMETRISE | GRAPH_ADD_SELF_LOOPS) -> Graph:
    """src/dst: int32 tensors, both on the host or both on the context's device."""
    if src.dtype != torch.int32 or dst.dtype != torch.int32 or src.numel() != dst.numel():
        raise TypeError("graph_create: src and dst must be int32 tensors of equal length")
    if src.is_cuda != dst.is_cuda:
        raise TypeError("graph_create: src and dst must live on the same side")
    src, dst = src.contiguous(), dst.contiguous()
    if src.is_cuda:
        flags |= GRAPH_EDGES_ON_DEVICE
        torch.cuda.current_stream().synchronize()
    h = C.c_void_p()
    _check(lib.mixgcn_graph_create(ctx.h, C.c_int64(n), C.c_int64(src.numel()), _ptr(src), _ptr(dst),
                                   C.c_uint32(flags), C.byref(h)))
    return Graph(ctx, h)


def graph_create_from_csr(ctx: Ctx, n: int, rowptr: torch.Tensor, col: torch.Tensor, flags: int = 0) -> Graph:
    if rowptr.dtype != torch.int64 or col.dtype != torch.int32 or rowptr.numel() != n + 1:
        raise TypeError("graph_create_from_csr: rowptr int64[n+1], col int32[nnz]")
    rowptr, col = rowptr.contiguous(), col.contiguous()
    flags = (flags & (GRAPH_NORM_ROW | GRAPH_NORM_NONE)) | (GRAPH_EDGES_ON_DEVICE if rowptr.is_cuda else 0)
    if rowptr.is_cuda:
        torch.cuda.current_stream().synchronize()
    h = C.c_void_p()
    _check(lib.mixgcn_graph_create_from_csr(ctx.h, C.c_int64(n), _ptr(rowptr), _ptr(col), C.c_uint32(flags), C.byref(h)))
    return Graph(ctx, h)


def graph_export(g: Graph, transposed: bool = False):
    """-> dict of host tensors rowptr, col, val, deg, dinv."""
    out = dict(rowptr=torch.empty(g.n + 1, dtype=torch.int64), col=torch.empty(g.nnz, dtype=torch.int32),
               val=torch.empty(g.nnz, dtype=torch.float32), deg=torch.empty(g.n, dtype=torch.int32),
               dinv=torch.empty(g.n, dtype=torch.float32))
    _check(lib.mixgcn_graph_export(g.h, C.c_int(int(transposed)), _ptr(out["rowptr"]), _ptr(out["col"]),
                                   _ptr(out["val"]), _ptr(out["deg"]), _ptr(out["dinv"])))
    return out


def graph_degrees(g: Graph) -> torch.Tensor:
    """Entries per row of the stored matrix (host int32); on a symmetric graph also the number of rows that gather node v."""
    deg = torch.empty(g.n, dtype=torch.int32)
    _check(lib.mixgcn_graph_export(g.h, C.c_int(0), None, None, None, _ptr(deg), None))
    return deg


def graph_export_schedule(g: Graph, transposed: bool = False) -> torch.Tensor:
    perm = torch.empty(g.n, dtype=torch.int32)
    _check(lib.mixgcn_graph_export_schedule(g.h, C.c_int(int(transposed)), _ptr(perm)))
    return perm


def build_info() -> dict:
    """Which build of the library is loaded: {"debug_bounds": bool}."""
    flag = C.c_int32(0)
    _check(lib.mixgcn_build_info(C.byref(flag)))
    return {"debug_bounds": bool(flag.value)}


def debug_poke_col(g: Graph, entry: int, value: int) -> int:
    """Bounds-checked debug build only: overwrite one column id of the forward CSR; returns the old one."""
    old = C.c_int32(0)
    _check(lib.mixgcn_debug_poke_col(g.h, C.c_int64(entry), C.c_int32(value), C.byref(old)))
    return old.value


def graph_bandwidth(g: Graph, order: torch.Tensor | None = None) -> int:
    """b = max over stored entries of p_v - p_u for the processing sequence `order` (host int32; None = identity)."""
    if order is not None and (order.is_cuda or order.dtype != torch.int32 or order.numel() != g.n):
        raise TypeError("order: host int32 tensor of length n")
    b = C.c_int64(0)
    _check(lib.mixgcn_graph_bandwidth(g.h, _ptr(None if order is None else order.contiguous()), C.byref(b)))
    return b.value


def graph_rcm(g: Graph) -> torch.Tensor:
    """Reverse Cuthill-McKee order (host int32 tensor, order[k] = node at position k)."""
    order = torch.empty(g.n, dtype=torch.int32)
    _check(lib.mixgcn_graph_rcm(g.h, _ptr(order)))
    return order


def pipeline_stages(n: int, b: int) -> int:
    s = C.c_int64(0)
    _check(lib.mixgcn_pipeline_stages(C.c_int64(n), C.c_int64(b), C.byref(s)))
    return s.value


def graph_create_permuted(ctx: Ctx, g: Graph, order: torch.Tensor) -> Graph:
    if order.is_cuda or order.dtype != torch.int32 or order.numel() != g.n:
        raise TypeError("order: host int32 tensor of length n")
    h = C.c_void_p()
    _check(lib.mixgcn_graph_create_permuted(ctx.h, g.h, _ptr(order.contiguous()), C.byref(h)))
    return Graph(ctx, h)


# ------------------------------------------------------------------------------ building blocks

def make_epilogue(bias=None, relu=False, drop_mask=None, keep_scale=1.0, gate=None, gate_scale=1.0,
                  residual=None, residual_scale=1.0, gate_bits=None, sign_bits=None):
    e = Epilogue()
    e.bias = None if bias is None else _dev(bias, torch.float32, "bias").data_ptr()
    e.relu = int(relu)
    e.drop_mask = None if drop_mask is None else _dev(drop_mask, torch.uint8, "drop_mask").data_ptr()
    e.keep_scale = keep_scale
    if gate is not None:
        gate, ldg = _mat(gate, "gate")
        e.gate, e.ld_gate = gate.data_ptr(), ldg
    e.gate_scale = gate_scale
    if residual is not None:
        residual, ldr = _mat(residual, "residual")
        e.residual, e.ld_residual = residual.data_ptr(), ldr
    e.residual_scale = residual_scale
    for name, t in (("gate_bits", gate_bits), ("sign_bits", sign_bits)):      # n x ld words of 32 bits (torch int32)
        if t is not None:
            _dev(t, torch.int32, name)
            if t.dim() != 2 or t.stride(1) != 1:
                raise TypeError(f"{name}: expected a row-major 2-D int32 tensor")
            setattr(e, name, t.data_ptr()); setattr(e, "ld_" + name, t.stride(0))
    e._keep = (bias, drop_mask, gate, residual, gate_bits, sign_bits)
    return e


def spmm(ctx: Ctx, g: Graph, Y: torch.Tensor, Z: torch.Tensor, w: int, transposed: bool = False, epi: Epilogue | None = None):
    Y, ldy = _mat(Y, "Y")
    Z, ldz = _mat(Z, "Z")
    _check(lib.mixgcn_spmm(ctx.h, g.h, C.c_int(int(transposed)), C.c_int32(w), _ptr(Y), C.c_int64(ldy),
                           _ptr(Z), C.c_int64(ldz), None if epi is None else C.byref(epi), _stream()))


def gemm(ctx: Ctx, precision: int, trans_a: bool, trans_b: bool, M: int, N: int, K: int,
         A: torch.Tensor, B: torch.Tensor, Cm: torch.Tensor, epi: Epilogue | None = None):
    A, lda = _mat(A, "A")
    B, ldb = _mat(B, "B")
    Cm, ldc = _mat(Cm, "C")
    _check(lib.mixgcn_gemm(ctx.h, C.c_int32(precision), C.c_int32(int(trans_a)), C.c_int32(int(trans_b)),
                           C.c_int64(M), C.c_int64(N), C.c_int64(K), _ptr(A), C.c_int64(lda), _ptr(B),
                           C.c_int64(ldb), _ptr(Cm), C.c_int64(ldc), None if epi is None else C.byref(epi), _stream()))


# ------------------------------------------------------------------------------ layers

def colsum(ctx: Ctx, X: torch.Tensor, out: torch.Tensor, d: int):
    """out[j] = sum over rows of X[:, j], j < d."""
    X, ld = _mat(X, "X")
    _dev(out, torch.float32, "out")
    _check(lib.mixgcn_colsum(ctx.h, C.c_int64(X.shape[0]), C.c_int32(d), _ptr(X), C.c_int64(ld), _ptr(out), _stream()))


def layer_desc(d_in, d_out, ld_in, ld_out, ld_saved, order=ORDER_AUTO, precision=PREC_FP32, flags=0,
               keep_scale=1.0, in_scale=1.0, n_chunks=0) -> LayerDesc:
    return LayerDesc(d_in, d_out, ld_in, ld_out, ld_saved, order, precision, flags, keep_scale, in_scale, n_chunks,
                     None, 0, None)


def layer_plan(desc: LayerDesc):
    order, cols = C.c_int32(), C.c_int32()
    _check(lib.mixgcn_layer_plan(C.byref(desc), C.byref(order), C.byref(cols)))
    return order.value, cols.value


def layer_fwd(ctx: Ctx, g: Graph, desc: LayerDesc, X_in, W, bias, drop_mask, saved, X_out):
    _mat(X_in, "X_in"); _mat(saved, "saved"); _mat(X_out, "X_out"); _dev(W, torch.float32, "W")
    if not W.is_contiguous():
        raise TypeError("W must be dense row-major")
    _check(lib.mixgcn_layer_fwd(ctx.h, g.h, C.byref(desc), _ptr(X_in), _ptr(W), _ptr(bias), _ptr(drop_mask),
                                _ptr(saved), _ptr(X_out), _stream()))


def layer_fwd_loss(ctx: Ctx, g: Graph, desc: LayerDesc, X_in, W, bias, saved, dlogits, labels, train_mask, loss, pred,
                   n_correct=None):
    """Last layer (update-first) with the loss taken inside its aggregation; raises EUNSUPPORTED if the layer does not qualify."""
    _mat(X_in, "X_in"); _mat(saved, "saved"); _mat(dlogits, "dlogits"); _dev(W, torch.float32, "W")
    if not W.is_contiguous():
        raise TypeError("W must be dense row-major")
    _dev(labels, torch.int32, "labels"); _dev(train_mask, torch.uint8, "train_mask"); _dev(loss, torch.float32, "loss")
    _dev(pred, torch.int32, "pred")
    _check(lib.mixgcn_layer_fwd_loss(ctx.h, g.h, C.byref(desc), _ptr(X_in), _ptr(W), _ptr(bias), _ptr(saved), _ptr(dlogits),
                                     _ptr(labels), _ptr(train_mask), _ptr(loss), _ptr(pred), _ptr(n_correct), _stream()))


def layer_bwd(ctx: Ctx, g: Graph, desc: LayerDesc, X_in, saved, X_out, drop_mask, W, G_out, G_in, dW, dbias):
    _mat(X_in, "X_in"); _mat(saved, "saved"); _mat(X_out, "X_out"); _mat(G_out, "G_out")
    if G_in is not None:
        _mat(G_in, "G_in")
    if not (W.is_contiguous() and dW.is_contiguous()):
        raise TypeError("W and dW must be dense row-major")
    _check(lib.mixgcn_layer_bwd(ctx.h, g.h, C.byref(desc), _ptr(X_in), _ptr(saved), _ptr(X_out), _ptr(drop_mask),
                                _ptr(W), _ptr(G_out), _ptr(G_in), _ptr(dW), _ptr(dbias), _stream()))


def loss_softmax_xent(ctx: Ctx, logits, labels, train_mask, loss, dlogits=None, pred=None, n_correct=None, C_=None):
    logits, ld = _mat(logits, "logits")
    n = logits.shape[0]
    Cc = logits.shape[1] if C_ is None else C_
    _dev(labels, torch.int32, "labels"); _dev(train_mask, torch.uint8, "train_mask"); _dev(loss, torch.float32, "loss")
    if dlogits is not None:
        dlogits, ldd = _mat(dlogits, "dlogits")
        if ldd != ld:
            raise TypeError("dlogits must share the logits' leading dimension")
    _check(lib.mixgcn_loss_softmax_xent(ctx.h, C.c_int64(n), C.c_int32(Cc), _ptr(logits), C.c_int64(ld), _ptr(labels),
                                        _ptr(train_mask), _ptr(loss), _ptr(dlogits), _ptr(pred), _ptr(n_correct), _stream()))


def loss_softmax_xent_noalloc(logits, labels, train_mask, loss, dlogits=None, pred=None, n_correct=None,
                              status=None, C_=None):
    """The loss for callers that cannot allocate device memory: no context, scratch inside the
    library image.  Runs on torch's current device; at most 33,554,432 rows."""
    logits, ld = _mat(logits, "logits")
    n = logits.shape[0]
    Cc = logits.shape[1] if C_ is None else C_
    _dev(labels, torch.int32, "labels"); _dev(train_mask, torch.uint8, "train_mask"); _dev(loss, torch.float32, "loss")
    if dlogits is not None:
        dlogits, ldd = _mat(dlogits, "dlogits")
        if ldd != ld:
            raise TypeError("dlogits must share the logits' leading dimension")
    _check(lib.mixgcn_loss_softmax_xent_noalloc(C.c_int64(n), C.c_int32(Cc), _ptr(logits), C.c_int64(ld), _ptr(labels),
                                                _ptr(train_mask), _ptr(loss), _ptr(dlogits), _ptr(pred), _ptr(n_correct),
                                                _ptr(status), _stream()))


def adam_step(ctx: Ctx, params, grads, ms, vs, t, lr=0.01, beta1=0.9, beta2=0.999, eps=1e-8):
    k = len(params)
    for lst in (params, grads, ms, vs):
        for x in lst:
            _dev(x, torch.float32, "adam tensor")
            if not x.is_contiguous():
                raise TypeError("adam tensors must be contiguous")
    arr = lambda lst: (C.c_void_p * k)(*[x.data_ptr() for x in lst])
    numel = (C.c_int64 * k)(*[x.numel() for x in params])
    _check(lib.mixgcn_adam_step(ctx.h, C.c_int32(k), arr(params), arr(grads), arr(ms), arr(vs), numel, C.c_int64(t),
                                C.c_float(lr), C.c_float(beta1), C.c_float(beta2), C.c_float(eps), _stream()))


class RowPlan:
    """Row plan of a row-sparse aggregation (see mixgcn_rowplan_create)."""

    def __init__(self, ctx: Ctx, g: Graph, handle):
        self.ctx, self.g, self.h = ctx, g, handle
        a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
        _check(lib.mixgcn_rowplan_info(self.h, C.byref(a), C.byref(b), C.byref(c)))
        self.in_count, self.out_count, self.nnz = a.value, b.value, c.value

    def in_rows(self) -> torch.Tensor:
        out = torch.empty(self.in_count, dtype=torch.int32, device=torch.device("cuda", self.ctx.device))
        _check(lib.mixgcn_rowplan_export(self.h, _ptr(out), None, _stream()))
        return out

    def out_row_mask(self) -> torch.Tensor:
        out = torch.empty(self.g.n, dtype=torch.uint8, device=torch.device("cuda", self.ctx.device))
        _check(lib.mixgcn_rowplan_export(self.h, None, _ptr(out), _stream()))
        return out

    def close(self):
        if self.h:
            lib.mixgcn_rowplan_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def rowplan_create(ctx: Ctx, g: Graph, in_row_mask: torch.Tensor, transposed: bool = True) -> RowPlan:
    _dev(in_row_mask, torch.uint8, "in_row_mask")
    if in_row_mask.numel() != g.n:
        raise ValueError("rowplan_create: the mask needs one byte per node")
    torch.cuda.current_stream().synchronize()
    h = C.c_void_p()
    _check(lib.mixgcn_rowplan_create(ctx.h, g.h, C.c_int(1 if transposed else 0), _ptr(in_row_mask), C.byref(h)))
    return RowPlan(ctx, g, h)


def spmm_rowplan(ctx: Ctx, plan: RowPlan, Yc: torch.Tensor, Z: torch.Tensor, w: int, epi=None, rows_only=False):
    """Z = epilogue(A_restricted Yc) with Yc the compacted input (plan.in_count rows)."""
    _dev(Yc, torch.float32, "Yc"); _dev(Z, torch.float32, "Z")
    if Yc.shape[0] != plan.in_count or Z.shape[0] != plan.g.n:
        raise ValueError("spmm_rowplan: Yc needs plan.in_count rows and Z one row per node")
    _check(lib.mixgcn_spmm_rowplan(ctx.h, plan.h, C.c_int32(w), _ptr(Yc), C.c_int64(Yc.stride(0)), _ptr(Z),
                                   C.c_int64(Z.stride(0)), C.byref(epi) if epi is not None else None,
                                   C.c_int32(1 if rows_only else 0), _stream()))


def count_rows(ctx: Ctx, row_mask) -> int:
    """Non-zero bytes of a device uint8 row mask (synchronises the current stream)."""
    _dev(row_mask, torch.uint8, "row_mask")
    out = C.c_int64(0)
    _check(lib.mixgcn_count_rows(ctx.h, C.c_int64(row_mask.numel()), _ptr(row_mask), C.byref(out), _stream()))
    return out.value


def train_step_host(ctx: Ctx, g: Graph, dims, precision, X, labels, train_mask, W, b, mW, vW, mb, vb, t,
                    lr=0.01, beta1=0.9, beta2=0.999, eps=1e-8, pred=None) -> float:
    """All tensors are HOST tensors (pinned memory makes the copies faster); W, b and the Adam
    moments are updated in place.  Returns the loss."""
    L = len(dims) - 1
    for x in [X, labels, train_mask, *W, *b, *mW, *vW, *mb, *vb]:
        if x.is_cuda or not x.is_contiguous():
            raise TypeError("train_step_host takes contiguous host tensors")
    dims_a = (C.c_int32 * (L + 1))(*dims)
    arr = lambda lst: (C.c_void_p * L)(*[x.data_ptr() for x in lst])
    loss = C.c_float(0.0)
    _check(lib.mixgcn_train_step_host(ctx.h, g.h, C.c_int32(L), dims_a, C.c_int32(precision), _ptr(X), _ptr(labels),
                                      _ptr(train_mask), arr(W), arr(b), arr(mW), arr(vW), arr(mb), arr(vb),
                                      C.c_int64(t), C.c_float(lr), C.c_float(beta1), C.c_float(beta2), C.c_float(eps),
                                      C.byref(loss), _ptr(pred)))
    return loss.value


def train_step_host_prefetch(ctx: Ctx, X_next):
    """Announce the (pinned) host features of the next train_step_host call so that the call before it overlaps their copy."""
    if X_next is not None and (X_next.is_cuda or not X_next.is_contiguous()):
        raise TypeError("train_step_host_prefetch takes a contiguous host tensor")
    _check(lib.mixgcn_train_step_host_prefetch(ctx.h, _ptr(X_next)))


def probe_gather(ctx: Ctx, table: torch.Tensor, gathers_per_warp: int, sink: torch.Tensor, seed: int = 1) -> int:
    """Enqueue the row-gather probe on a rows x 128 fp32 table; returns the number of rows it reads."""
    table, ld = _mat(table, "table")
    if ld != 128 or table.shape[1] != 128:
        raise TypeError("table: expected a dense rows x 128 fp32 tensor")
    total = C.c_int64(0)
    _check(lib.mixgcn_probe_gather(ctx.h, _ptr(table), C.c_int64(table.shape[0]), C.c_int64(gathers_per_warp),
                                   C.c_uint64(seed), _ptr(sink), C.byref(total), _stream()))
    return total.value


def mask_pack(ctx: Ctx, w: int, bits: torch.Tensor, X: torch.Tensor | None = None, bytes_mask: torch.Tensor | None = None):
    """bits (n x ld_bits int32 device tensor) <- bitmap of (X > 0) and / or (bytes_mask != 0)."""
    _dev(bits, torch.int32, "bits")
    n, ld_bits = bits.shape[0], bits.stride(0)
    ldx = 0
    if X is not None:
        X, ldx = _mat(X, "X")
    if bytes_mask is not None:
        _dev(bytes_mask, torch.uint8, "bytes_mask")
    _check(lib.mixgcn_mask_pack(ctx.h, C.c_int64(n), C.c_int32(w), _ptr(X), C.c_int64(ldx), _ptr(bytes_mask), _ptr(bits),
                                C.c_int64(ld_bits), _stream()))


def spmm_sampled(ctx: Ctx, g: Graph, Y: torch.Tensor, Z: torch.Tensor, w: int, bits: torch.Tensor, transposed: bool = False,
                 epi: Epilogue | None = None):
    """Z = (A_hat Y) (.) M with M given as a bitmap (n x ld_bits int32 words)."""
    Y, ldy = _mat(Y, "Y")
    Z, ldz = _mat(Z, "Z")
    _dev(bits, torch.int32, "bits")
    _check(lib.mixgcn_spmm_sampled(ctx.h, g.h, C.c_int(int(transposed)), C.c_int32(w), _ptr(Y), C.c_int64(ldy), _ptr(Z),
                                   C.c_int64(ldz), _ptr(bits), C.c_int64(bits.stride(0)), None if epi is None else C.byref(epi),
                                   _stream()))
