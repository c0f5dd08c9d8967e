"""Shared test plumbing: tolerances, Frobenius error, padded device tensors."""
import numpy as np
import torch

# fp32 path: relative Frobenius error against the fp64 oracle.  Rounding of one fp32 FMA chain of
# length k grows like sqrt(k) * 2^-24 ~ 6e-8 * sqrt(k); the kernels keep chains <= ~1e3 terms
# (two-level accumulation, fp64 final sums), which leaves roughly one decimal digit of margin.
TOL_FP32 = 1e-5
# TF32 / BF16 operands with fp32 accumulation
TOL_LOWP = 5e-3


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def round4(x):
    return (x + 3) // 4 * 4


def padded(t: torch.Tensor, device="cuda", fill=0.0):
    """Host n x d tensor -> device n x round4(d) fp32 tensor whose pad columns hold `fill`."""
    n, d = t.shape
    out = torch.full((n, round4(d)), fill, dtype=torch.float32, device=device)
    out[:, :d] = t.to(device=device, dtype=torch.float32)
    return out


def host(t: torch.Tensor, d=None):
    a = t.detach().cpu().numpy()
    return a if d is None else a[:, :d]


# Adam's scalars are fp32 arguments of the C entry point; the oracle receives the same (fp32-rounded) values
ADAM = dict(lr=float(np.float32(0.01)), beta1=float(np.float32(0.9)), beta2=float(np.float32(0.999)),
            eps=float(np.float32(1e-8)))
