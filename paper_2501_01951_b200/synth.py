"""Seeded synthetic inputs for full-graph GCN training.

This module only *draws inputs*: R-MAT edge lists, N(0,1) features, uniform labels,
Bernoulli train masks and Glorot-uniform weights.  It contains none of the method's
arithmetic (no normalisation, aggregation, update, loss or optimiser step) and imports
neither the CUDA binding nor the CPU oracle; both sides of a parity test receive the very
same arrays produced here.

Every draw is a pure function of ``(seed, element index)`` through a counter-based
generator (splitmix64 on 64-bit integers, written with torch integer ops), so a result does
not depend on chunk sizes, thread counts or the device it is generated on.  Integer-valued
outputs (edges, labels, masks) are bit-identical on CPU and GPU; the Glorot weights are
rounded once from an exact fp64 expression and are bit-identical as well; the normal
features go through ``log``/``cos`` in fp32 and may differ in the last bit between devices,
so a test generates them once and hands the same tensor to both sides.

The five workloads (``CONFIGS``) take their shapes from the datasets table of the paper
(Table 2: nodes / edges / feature width / classes); no item of any dataset is reproduced.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

_M64 = (1 << 64) - 1


def _i64(x: int) -> int:
    """Python int -> the signed 64-bit value with the same bit pattern."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _i64(0x9E3779B97F4A7C15)
_MUL1 = _i64(0xBF58476D1CE4E5B9)
_MUL2 = _i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor (torch's >> is arithmetic)."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def splitmix64(x: torch.Tensor) -> torch.Tensor:
    """One splitmix64 output step on an int64 tensor (wrap-around arithmetic)."""
    z = x + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def _splitmix64_int(x: int) -> int:
    z = (x + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _stream_key(seed: int, stream: int) -> int:
    """A 64-bit key for (seed, stream), as a signed python int."""
    return _i64(_splitmix64_int(_splitmix64_int(seed & _M64) ^ (stream * 0xD1B54A32D192ED03 & _M64)))


def hash_index(seed: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """64 pseudo-random bits per element of ``idx`` (int64), keyed by (seed, stream)."""
    return splitmix64(splitmix64(idx ^ _stream_key(seed, stream)))


# ----------------------------------------------------------------------------- graphs

RMAT_ABCD = (0.57, 0.19, 0.19, 0.05)


def _scramble_ids(x: torch.Tensor, s: int, seed: int) -> torch.Tensor:
    """A seeded bijection on [0, 2**s): odd-multiplier affine maps and xor-shifts."""
    mask = (1 << s) - 1
    a = (_splitmix64_int(seed ^ 0xA5A5) | 1) & mask
    b = _splitmix64_int(seed ^ 0x5A5A) & mask
    c = (_splitmix64_int(seed ^ 0x1234) | 1) & mask
    k1 = max(1, s // 2)
    k2 = max(1, s // 2 + 1)
    x = (x * a + b) & mask
    x = x ^ (x >> k1)
    x = (x * c) & mask
    x = x ^ (x >> k2)
    return x & mask


def rmat_candidates(seed: int, first: int, count: int, scale: int, device="cpu"):
    """Candidate edges ``first .. first+count-1`` of the R-MAT stream: int64 (u, v) in
    [0, 2**scale), before id scrambling.  One 16-bit draw per level, four per hash."""
    a, b, c, _ = RMAT_ABCD
    ta = int(round(a * 65536))
    tab = int(round((a + b) * 65536))
    tabc = int(round((a + b + c) * 65536))
    i = torch.arange(first, first + count, dtype=torch.int64, device=device)
    u = torch.zeros_like(i)
    v = torch.zeros_like(i)
    words = (scale + 3) // 4
    level = 0
    for wd in range(words):
        h = hash_index(seed, 100 + wd, i)
        for q in range(4):
            if level >= scale:
                break
            r = _lsr(h, 16 * q) & 0xFFFF
            ub = (r >= tab).to(torch.int64)
            vb = (((r >= ta) & (r < tab)) | (r >= tabc)).to(torch.int64)
            u = u * 2 + ub
            v = v * 2 + vb
            level += 1
    return u, v


def rmat_graph(n: int, target_undirected: int, seed: int, device="cpu", batch: int | None = None):
    """Seeded R-MAT graph on ``n`` nodes with at least ``target_undirected`` distinct
    undirected edges (no self-loops).  Candidates are drawn in fixed-size batches; ids pass
    through a seeded bijection so that degree is uncorrelated with id; pairs with an id >= n
    or u == v are rejected; duplicates collapse.  Batches are added until the distinct count
    first reaches the target, so the overshoot is below one batch.

    Returns (src, dst) int32 tensors with src < dst, sorted by (src, dst).
    """
    scale = max(1, math.ceil(math.log2(n)))
    if batch is None:
        batch = 1 << max(12, math.ceil(math.log2(max(target_undirected, 1))) - 3)
    keys = torch.empty(0, dtype=torch.int64, device=device)
    first = 0
    max_batches = 4096
    for _ in range(max_batches):
        u, v = rmat_candidates(seed, first, batch, scale, device)
        first += batch
        u = _scramble_ids(u, scale, seed)
        v = _scramble_ids(v, scale, seed)
        ok = (u < n) & (v < n) & (u != v)
        lo = torch.minimum(u, v)[ok]
        hi = torch.maximum(u, v)[ok]
        del u, v, ok
        keys = torch.unique(torch.cat([keys, (lo << 32) | hi]))
        del lo, hi
        if keys.numel() >= target_undirected:
            break
    else:
        raise RuntimeError("R-MAT generator did not reach the target edge count")
    src = (keys >> 32).to(torch.int32)
    dst = (keys & 0xFFFFFFFF).to(torch.int32)
    return src, dst


# ----------------------------------------------------------------------------- tensors

def _uniform24(seed: int, stream: int, idx: torch.Tensor, shift: int) -> torch.Tensor:
    return _lsr(hash_index(seed, stream, idx), shift) & 0xFFFFFF


def normal_features(n: int, d: int, seed: int, device="cpu", ld: int | None = None,
                    rows_per_chunk: int = 1 << 18, out: torch.Tensor | None = None) -> torch.Tensor:
    """n x d fp32 i.i.d. N(0,1) (Box-Muller on two 24-bit uniforms keyed by (seed, row*d+col)),
    stored row-major with leading dimension ``ld`` (>= d; pad columns are zero)."""
    ld = d if ld is None else ld
    if out is None:
        out = torch.zeros((n, ld), dtype=torch.float32, device=device)
    for r0 in range(0, n, rows_per_chunk):
        r1 = min(n, r0 + rows_per_chunk)
        idx = torch.arange(r0 * d, r1 * d, dtype=torch.int64, device=device)
        h = hash_index(seed, 200, idx)
        u1 = ((_lsr(h, 40) & 0xFFFFFF) + 1).to(torch.float32) * (1.0 / 16777216.0)
        u2 = (_lsr(h, 16) & 0xFFFFFF).to(torch.float32) * (1.0 / 16777216.0)
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        out[r0:r1, :d] = z.view(r1 - r0, d)
        del idx, h, u1, u2, z
    return out


def uniform_labels(n: int, classes: int, seed: int, device="cpu") -> torch.Tensor:
    idx = torch.arange(n, dtype=torch.int64, device=device)
    return (_lsr(hash_index(seed, 300, idx), 8) % classes).to(torch.int32)


def bernoulli_mask(n: int, p: float, seed: int, device="cpu") -> torch.Tensor:
    idx = torch.arange(n, dtype=torch.int64, device=device)
    return (_uniform24(seed, 400, idx, 20) < int(round(p * 16777216))).to(torch.uint8)


def glorot_uniform(d_in: int, d_out: int, seed: int, device="cpu") -> torch.Tensor:
    """d_in x d_out fp32, U(-a, a) with a = sqrt(6 / (d_in + d_out))."""
    idx = torch.arange(d_in * d_out, dtype=torch.int64, device=device)
    u = _uniform24(seed, 500, idx, 24).to(torch.float64) * (1.0 / 16777216.0)
    a = math.sqrt(6.0 / (d_in + d_out))
    return ((2.0 * u - 1.0) * a).to(torch.float32).view(d_in, d_out)


def uniform_tensor(shape, seed: int, lo=-1.0, hi=1.0, device="cpu", stream: int = 600) -> torch.Tensor:
    """fp32 U(lo, hi) of any shape (test helper for gradients, masks' complements, etc.)."""
    numel = 1
    for s in shape:
        numel *= s
    idx = torch.arange(numel, dtype=torch.int64, device=device)
    u = _uniform24(seed, stream, idx, 24).to(torch.float64) * (1.0 / 16777216.0)
    return (lo + (hi - lo) * u).to(torch.float32).view(*shape)


# ----------------------------------------------------------------------------- workloads

@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    undirected_edges: int          # target count of distinct undirected edges
    dims: tuple                    # (d0, d1, ..., dL); dL = number of classes
    mask_p: float
    precision: str                 # "fp32" | "tf32" | "bf16": arithmetic of the dense update
    seed_base: int
    note: str = ""
    seeds: dict = field(default_factory=dict)

    @property
    def classes(self) -> int:
        return self.dims[-1]

    def seed(self, what: str) -> int:
        order = {"graph": 1000, "features": 2000, "labels": 3000, "mask": 4000, "weights": 5000}
        return order[what] + self.seed_base


CONFIGS = {
    "C1": Workload("C1-tiny", 4096, 32768, (64, 32, 8), 0.5, "fp32", 1,
                   "smoke-sized; the oracle finishes in well under a second"),
    "C2": Workload("C2-dense-neighbourhood", 232965, 57_300_000, (602, 256, 256, 41), 0.66, "tf32", 2,
                   "shape of the densest row of the paper's datasets table (233K nodes, ~115M edges, 602 features, 41 classes)"),
    "C3": Workload("C3-co-purchase-shaped", 2449029, 61_850_000, (100, 256, 256, 47), 0.08, "tf32", 3,
                   "sparse, heavy-tailed, 100 features, 47 classes"),
    "C4": Workload("C4-wide-features", 1_000_000, 15_000_000, (1024, 1024, 1024, 64), 0.5, "bf16", 4,
                   "GEMM-heavy by construction"),
    "C5": Workload("C5-large-citation-shaped", 30_000_000, 240_000_000, (128, 128, 128, 172), 0.01, "tf32", 5,
                   "128 features / 172 classes as in the largest row of the paper's datasets table, node count scaled to one GPU"),
}


def make_weights(wl: Workload, device="cpu"):
    """Glorot-uniform W_l (d_l x d_{l+1}) and zero biases for every layer of a workload."""
    Ws, bs = [], []
    for l in range(len(wl.dims) - 1):
        Ws.append(glorot_uniform(wl.dims[l], wl.dims[l + 1], wl.seed("weights") * 16 + l, device))
        bs.append(torch.zeros(wl.dims[l + 1], dtype=torch.float32, device=device))
    return Ws, bs
