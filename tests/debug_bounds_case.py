"""Body of tests/test_gpu_debug_bounds.py: runs in a process of its own with MIXGCN_LIBRARY=debug, so that the
bounds-checked build of the library is the one loaded.  Not collected by pytest (no test_ prefix)."""
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from helpers import TOL_FP32, rel_fro          # noqa: E402
from oracle import gcn_oracle as orc            # noqa: E402
from paper_2501_01951_b200 import binding as mg, synth   # noqa: E402


def guarded(n, ld):
    """n x ld matrix with one spare row on either side: an index one step outside [0, n) would still land in
    this allocation even if a check let it through."""
    buf = torch.zeros(n + 2, ld, device="cuda")
    return buf, buf[1:n + 1]


def main():
    assert mg.build_info()["debug_bounds"], "MIXGCN_LIBRARY=debug must load the bounds-checked build"
    n, hub = 9000, 6000
    rng = np.random.default_rng(5)
    # node 0 is a hub (long-row segments), nodes 1..6000 have a handful of entries, the rest only their diagonal
    s = np.concatenate([np.zeros(hub, np.int64), rng.integers(1, hub + 1, 3 * hub)])
    d = np.concatenate([np.arange(1, hub + 1), rng.integers(1, hub + 1, 3 * hub)])
    go = orc.graph_build(n, s, d)
    ctx = mg.ctx_create(0)
    g = mg.graph_create(ctx, n, torch.tensor(s, dtype=torch.int32), torch.tensor(d, dtype=torch.int32))
    ex = mg.graph_export(g)
    rowptr, col, val = ex["rowptr"].numpy(), ex["col"].numpy(), ex["val"].numpy()
    deg = np.diff(rowptr)
    assert deg[0] > 512 and (deg == 1).any() and ((deg > 12) & (deg <= 512)).any()
    for w in (12, 128, 300):
        ld = (w + 3) // 4 * 4
        X = synth.uniform_tensor((n, w), 40 + w, -1, 1)
        _, Xd = guarded(n, ld)
        Xd[:, :w] = X.cuda()
        _, Z = guarded(n, ld)
        want = orc.aggregate(go, X.numpy())
        mg.spmm(ctx, g, Xd, Z, w)
        assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
        assert rel_fro(Z[:, :w].cpu().numpy().astype(np.float64), want) <= TOL_FP32        # the checked kernels compute the same thing
        rows = [0, int(np.flatnonzero((deg > 12) & (deg <= 512))[0]), int(np.flatnonzero(deg == 1)[0])]   # segment / group / short-row kernels
        for u in rows:
            for bad in (n, -1):                      # one step outside on either side
                e = int(rowptr[u] + deg[u] // 2)
                old = mg.debug_poke_col(g, e, bad)
                assert old == col[e]
                Z.zero_()
                mg.spmm(ctx, g, Xd, Z, w)
                with_error = None
                try:
                    mg.ctx_poll_status(ctx)
                except mg.MixgcnError as err:
                    with_error = err
                assert with_error is not None and with_error.status == mg.EDEVICE, f"row {u} width {w} index {bad}: not reported"
                assert "column id" in str(with_error) and str(bad) in str(with_error), str(with_error)
                # the bad entry's term is skipped, everything else is computed: row u misses val * X[old column]
                expect = want.copy()
                expect[u] -= float(val[e]) * X.numpy()[old].astype(np.float64)
                got = Z[:, :w].cpu().numpy().astype(np.float64)
                assert rel_fro(got, expect) <= TOL_FP32 and rel_fro(got[u], expect[u]) <= TOL_FP32
                assert mg.debug_poke_col(g, e, old) == bad
                Z.zero_()
                mg.spmm(ctx, g, Xd, Z, w)                                              # the context is still usable
                assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
                assert rel_fro(Z[:, :w].cpu().numpy().astype(np.float64), want) <= TOL_FP32
    g.close(); ctx.close()
    print("debug-bounds case: ok")


if __name__ == "__main__":
    main()
