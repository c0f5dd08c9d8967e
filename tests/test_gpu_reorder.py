"""Node reordering (Section 3.2.2): bandwidth, reverse Cuthill-McKee, stage count, relabelled graphs."""
import numpy as np
import pytest
import torch

from helpers import TOL_FP32, host, padded, rel_fro
from oracle import gcn_oracle as orc
from paper_2501_01951_b200 import synth


@pytest.fixture(scope="module")
def mg():
    from paper_2501_01951_b200 import build
    build.build()
    from paper_2501_01951_b200 import binding
    return binding


def test_pipeline_stage_count_matches_the_oracle(mg):          # host arithmetic: no GPU needed
    for n, b in ((1000, 800), (1000, 0), (1000, 1), (1000, 999), (37, 5), (12345, 6789), (30_000_000, 29_999_000)):
        assert mg.pipeline_stages(n, b) == orc.pipeline_stages(n, b)
    with pytest.raises(mg.MixgcnError):
        mg.pipeline_stages(10, 10)
    with pytest.raises(mg.MixgcnError):
        mg.pipeline_stages(0, 0)


def _graphs():
    rng = np.random.default_rng(11)
    n = 64
    lab = rng.permutation(n)
    yield "scrambled-path", n, lab[:-1], lab[1:]
    yield "random", 500, rng.integers(0, 500, 900), rng.integers(0, 500, 900)
    yield "components", 40, np.array([0, 1, 5, 9, 9]), np.array([1, 2, 6, 10, 11])
    s, d = synth.rmat_graph(4096, 32768, 1001)
    yield "rmat", 4096, s.numpy(), d.numpy()


@pytest.mark.gpu
@pytest.mark.parametrize("case", list(_graphs()), ids=lambda c: c[0])
def test_rcm_and_bandwidth_match_the_oracle(mg, case):
    name, n, s, d = case
    ctx = mg.ctx_create(0)
    go = orc.graph_build(n, s, d)
    gg = mg.graph_create(ctx, n, torch.tensor(s, dtype=torch.int32), torch.tensor(d, dtype=torch.int32))
    assert mg.graph_bandwidth(gg) == orc.bandwidth(go)
    order = mg.graph_rcm(gg)
    want = orc.rcm(go)
    assert np.array_equal(order.numpy().astype(np.int64), want)              # same rule, same ties: identical order
    b = mg.graph_bandwidth(gg, order)
    assert b == orc.bandwidth(go, want)
    if name == "scrambled-path":
        assert b == 1 and mg.pipeline_stages(n, b) == 3
    # relabelled graph: P A_hat P^T, entry for entry
    gp = mg.graph_create_permuted(ctx, gg, order)
    assert (gp.n, gp.nnz, gp.symmetric) == (gg.n, gg.nnz, True)
    assert mg.graph_bandwidth(gp) == b
    pos = np.empty(n, dtype=np.int64); pos[want] = np.arange(n)
    gpo = orc.graph_build(n, pos[np.asarray(s)], pos[np.asarray(d)])
    e = mg.graph_export(gp)
    assert np.array_equal(e["rowptr"].numpy(), gpo.rowptr) and np.array_equal(e["col"].numpy(), gpo.col)
    assert e["val"].numpy().tobytes() == gpo.val32.tobytes()
    # aggregation commutes with the relabelling: (P A P^T)(P X) = P (A X)
    X = synth.uniform_tensor((n, 12), 5, -1, 1)
    Xp = X[torch.tensor(want)]
    Z = torch.zeros(n, 12, device="cuda"); Zp = torch.zeros(n, 12, device="cuda")
    mg.spmm(ctx, gg, padded(X), Z, 12)
    mg.spmm(ctx, gp, padded(Xp), Zp, 12)
    assert rel_fro(host(Zp), host(Z)[want]) <= TOL_FP32
    with pytest.raises(mg.MixgcnError):
        mg.graph_bandwidth(gg, torch.zeros(n, dtype=torch.int32))             # not a permutation
    gp.close(); gg.close(); ctx.close()


@pytest.mark.gpu
def test_rcm_needs_a_symmetric_graph(mg):
    ctx = mg.ctx_create(0)
    gg = mg.graph_create(ctx, 4, torch.tensor([0, 1], dtype=torch.int32), torch.tensor([1, 2], dtype=torch.int32),
                         mg.GRAPH_ADD_SELF_LOOPS)
    with pytest.raises(mg.MixgcnError) as e:
        mg.graph_rcm(gg)
    assert e.value.status == mg.EUNSUPPORTED
    gg.close(); ctx.close()
