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
    # a level-synchronous device search against the oracle's one-node-at-a-time queue: same rule and
    # ties, so the same order although the two share no structure
    assert np.array_equal(order.numpy().astype(np.int64), want)
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


def _grid_edges(rows, cols):
    """A rows x cols grid graph under scrambled labels: a graph that HAS locality for the ordering to find."""
    ids = np.arange(rows * cols).reshape(rows, cols)
    s = np.concatenate([ids[:, :-1].ravel(), ids[:-1, :].ravel()])
    d = np.concatenate([ids[:, 1:].ravel(), ids[1:, :].ravel()])
    lab = np.random.default_rng(21).permutation(rows * cols)
    return rows * cols, lab[s], lab[d]


@pytest.mark.gpu
@pytest.mark.parametrize("kind", ["grid", "rmat"])
def test_pipeline_with_the_stage_count_of_the_reordered_graph(mg, kind):
    """The fine-grain pipeline as Section 3.2.2 composes it: reorder the nodes (RCM), take the stage count
    s = ceil(2n / (n - b)) of Proposition 3.5 from the bandwidth b of the new order, and run the layer in s
    row chunks (aggregation of chunk k+1 overlapping the update of chunk k).  Forward output and every
    gradient must be the oracle's on the permuted inputs."""
    from helpers import round4
    if kind == "grid":
        n, s, d = _grid_edges(40, 50)
    else:
        n = 4096
        ss, dd = synth.rmat_graph(n, 32768, 1001)
        s, d = ss.numpy(), dd.numpy()
    ctx = mg.ctx_create(0)
    g0 = mg.graph_create(ctx, n, torch.tensor(s, dtype=torch.int32), torch.tensor(d, dtype=torch.int32))
    order = mg.graph_rcm(g0)
    b = mg.graph_bandwidth(g0, order)
    stages = mg.pipeline_stages(n, b)
    assert stages == orc.pipeline_stages(n, b) and stages >= 3
    if kind == "grid":
        assert b <= 2 * 50 and stages == 3          # the ordering recovered the grid's band: the smallest stage count
    n_chunks = min(stages, 64)
    gp = mg.graph_create_permuted(ctx, g0, order)
    assert mg.graph_bandwidth(gp) == b
    # the oracle sees the relabelled edge list and the permuted inputs
    o = order.numpy().astype(np.int64)
    pos = np.empty(n, dtype=np.int64); pos[o] = np.arange(n)
    go = orc.graph_build(n, pos[np.asarray(s)], pos[np.asarray(d)])
    d_in, d_out = 48, 40
    X = synth.uniform_tensor((n, d_in), 31, -1, 1)[torch.tensor(o)]
    W = synth.glorot_uniform(d_in, d_out, 32)
    bias = synth.uniform_tensor((d_out,), 33, -0.2, 0.2)
    Gout = synth.uniform_tensor((n, d_out), 34, -1, 1)[torch.tensor(o)]
    desc = mg.layer_desc(d_in, d_out, round4(d_in), round4(d_out), round4(d_in), mg.ORDER_AGG_FIRST, mg.PREC_FP32,
                         mg.LAYER_RELU, 1.0, 1.0, n_chunks)
    Xd, Wd, bd = padded(X), W.cuda(), bias.cuda()
    saved = torch.zeros(n, round4(d_in), device="cuda"); Xout = torch.zeros(n, round4(d_out), device="cuda")
    mg.layer_fwd(ctx, gp, desc, Xd, Wd, bd, None, saved, Xout)
    Z = orc.aggregate(go, X.numpy())
    P = orc.update(Z, W.numpy(), bias.numpy())
    assert rel_fro(host(Xout, d_out), orc.activation(P, True)) <= TOL_FP32
    Gd = padded(Gout); Gin = torch.zeros(n, round4(d_in), device="cuda")
    dW = torch.zeros(d_in, d_out, device="cuda"); db = torch.zeros(d_out, device="cuda")
    mg.layer_bwd(ctx, gp, desc, Xd, saved, Xout, None, Wd, Gd, Gin, dW, db)
    _, dWo, dbo, dZo = orc.update_bwd(Z, P, W.numpy(), Gout.numpy(), True, None, 1.0, need_dZ=True)
    assert rel_fro(host(dW), dWo) <= TOL_FP32 and rel_fro(db.cpu().numpy(), dbo) <= TOL_FP32
    assert rel_fro(host(Gin, d_in), orc.aggregate(go, dZo, transposed=True)) <= TOL_FP32
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    gp.close(); g0.close(); ctx.close()
