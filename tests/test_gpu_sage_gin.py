"""GraphSAGE (mean aggregator) and GIN, the two other architectures the paper's evaluation names:
whole training iterations through the C-ABI against the CPU oracle's iterations."""
import numpy as np
import pytest
import torch

from helpers import ADAM, TOL_FP32, TOL_LOWP, host, padded, rel_fro, round4
from oracle import gcn_oracle as orc
from paper_2501_01951_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2501_01951_b200 import build
    build.build()
    from paper_2501_01951_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(mg):
    c = mg.ctx_create(0)
    yield c
    assert mg.ctx_poll_status(c, raise_on_error=False) == 0
    c.close()


def _problem(dims):
    wl = synth.CONFIGS["C1"]
    s, d = synth.rmat_graph(wl.n, wl.undirected_edges, wl.seed("graph"))
    X = synth.normal_features(wl.n, dims[0], wl.seed("features"))
    y = synth.uniform_labels(wl.n, dims[-1], wl.seed("labels"))
    m = synth.bernoulli_mask(wl.n, 0.3, wl.seed("mask"))
    return wl.n, s, d, X, y, m


@pytest.mark.parametrize("dims", [(64, 32, 16, 8), (30, 18, 7)])
def test_sage_training_epochs_match_oracle(mg, ctx, dims):
    from paper_2501_01951_b200.sage_gin import SageTrainer
    n, s, d, X, y, m = _problem(dims)
    L = len(dims) - 1
    go = orc.graph_build(n, s.numpy(), d.numpy(), orc.SYMMETRISE, norm="row")
    gg = mg.graph_create(ctx, n, s, d, mg.GRAPH_SYMMETRISE | mg.GRAPH_NORM_ROW)
    Ws = [synth.glorot_uniform(dims[i], dims[i + 1], 500 + i) for i in range(L)]
    Wn = [synth.glorot_uniform(dims[i], dims[i + 1], 520 + i) for i in range(L)]
    bs = [synth.uniform_tensor((dims[i + 1],), 540 + i, -0.1, 0.1) for i in range(L)]
    tr = SageTrainer(ctx, gg, dims, mg.PREC_FP32)
    tr.set_params(Ws, Wn, bs)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    ref = orc.sage_epoch(go, X.numpy(), [w.numpy() for w in Ws], [w.numpy() for w in Wn], [b.numpy() for b in bs],
                         y.numpy(), m.numpy(), None, 1, **ADAM)
    tr.forward()
    assert rel_fro(host(tr.logits, dims[-1]), ref["logits"]) <= TOL_FP32
    tr.compute_loss(); tr.backward(); tr.step(1, **ADAM)
    assert abs(tr.loss.item() - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    assert tr.n_correct.item() == ref["n_correct"]
    for l in range(L):
        gcat = tr.grads[l].cpu().numpy()
        d_l, ld_l = dims[l], round4(dims[l])
        assert rel_fro(gcat[:d_l], ref["grads"][l]) <= TOL_FP32                      # W_self
        assert rel_fro(gcat[ld_l:ld_l + d_l], ref["grads"][L + l]) <= TOL_FP32       # W_neigh
        assert rel_fro(tr.grads[L + l].cpu().numpy(), ref["grads"][2 * L + l]) <= TOL_FP32
        big = np.abs(ref["grads"][l]) > 1e-4 * np.abs(ref["grads"][l]).max()
        dgpu = tr.params[l].cpu().numpy()[:d_l].astype(np.float64) - Ws[l].numpy()
        assert rel_fro(dgpu[big], (ref["params"][l] - Ws[l].numpy())[big]) <= 1e-3  # the Adam step
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


@pytest.mark.parametrize("dims,hidden,gin_eps", [((64, 32, 16, 8), 24, 0.0), ((30, 18, 7), 11, 0.25)])
def test_gin_training_epochs_match_oracle(mg, ctx, dims, hidden, gin_eps):
    from paper_2501_01951_b200.sage_gin import GinTrainer
    n, s, d, X, y, m = _problem(dims)
    L = len(dims) - 1
    go = orc.graph_build(n, s.numpy(), d.numpy(), orc.SYMMETRISE, norm="none")
    gg = mg.graph_create(ctx, n, s, d, mg.GRAPH_SYMMETRISE | mg.GRAPH_NORM_NONE)
    # sums over hundreds of neighbours: keep the weights small so that the logits stay O(1)
    W1 = [synth.glorot_uniform(dims[i], hidden, 600 + i) * 0.05 for i in range(L)]
    b1 = [synth.uniform_tensor((hidden,), 620 + i, -0.1, 0.1) for i in range(L)]
    W2 = [synth.glorot_uniform(hidden, dims[i + 1], 640 + i) * 0.3 for i in range(L)]
    b2 = [synth.uniform_tensor((dims[i + 1],), 660 + i, -0.1, 0.1) for i in range(L)]
    tr = GinTrainer(ctx, gg, dims, hidden, mg.PREC_FP32, gin_eps=gin_eps)
    tr.set_params(W1, b1, W2, b2)
    tr.set_inputs(padded(X), y.cuda(), m.cuda())
    npl = lambda lst: [t.numpy() for t in lst]
    ref = orc.gin_epoch(go, X.numpy(), npl(W1), npl(b1), npl(W2), npl(b2), y.numpy(), m.numpy(), gin_eps, None, 1, **ADAM)
    tr.forward()
    assert rel_fro(host(tr.logits, dims[-1]), ref["logits"]) <= TOL_FP32
    tr.compute_loss(); tr.backward(); tr.step(1, **ADAM)
    assert abs(tr.loss.item() - ref["loss"]) <= 1e-5 * abs(ref["loss"])
    for i in range(4 * L):
        assert rel_fro(tr.grads[i].cpu().numpy(), ref["grads"][i]) <= 2 * TOL_FP32, f"gradient {i}"
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0


def test_sage_and_gin_run_on_tensor_cores(mg, ctx):
    """TF32 products: logits and loss stay within the reduced-precision tolerance."""
    from paper_2501_01951_b200.sage_gin import GinTrainer, SageTrainer
    dims = (64, 32, 16, 8)
    n, s, d, X, y, m = _problem(dims)
    L = 3
    go = orc.graph_build(n, s.numpy(), d.numpy(), orc.SYMMETRISE, norm="row")
    gg = mg.graph_create(ctx, n, s, d, mg.GRAPH_SYMMETRISE | mg.GRAPH_NORM_ROW)
    Ws = [synth.glorot_uniform(dims[i], dims[i + 1], 500 + i) for i in range(L)]
    Wn = [synth.glorot_uniform(dims[i], dims[i + 1], 520 + i) for i in range(L)]
    bs = [synth.uniform_tensor((dims[i + 1],), 540 + i, -0.1, 0.1) for i in range(L)]
    tr = SageTrainer(ctx, gg, dims, mg.PREC_TF32)
    tr.set_params(Ws, Wn, bs); tr.set_inputs(padded(X), y.cuda(), m.cuda())
    ref = orc.sage_epoch(go, X.numpy(), [w.numpy() for w in Ws], [w.numpy() for w in Wn], [b.numpy() for b in bs],
                         y.numpy(), m.numpy(), None, 1, **ADAM)
    tr.forward()
    assert rel_fro(host(tr.logits, dims[-1]), ref["logits"]) <= TOL_LOWP
    tr.compute_loss(); tr.backward()
    assert abs(tr.loss.item() - ref["loss"]) <= TOL_LOWP * abs(ref["loss"])
    for t_ in tr.grads:
        assert bool(torch.isfinite(t_).all())
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
