"""Bit-packed masks (the bitmap mask buffer of Section 3.2.1): the sign bitmap a forward kernel writes beside its
result, and the same bitmap read as the gate of Eq. 4's backward form instead of the fp32 tensor.  A gate decision
is a bit either way, so everything must agree BIT FOR BIT with the fp32-gate path, which the other parity tests
hold against the oracle; the bitmap itself is checked against numpy."""
import numpy as np
import pytest
import torch

from helpers import TOL_FP32, host, padded, rel_fro, round4
from oracle import gcn_oracle as orc
from paper_2501_01951_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2501_01951_b200 import build
    build.build()
    from paper_2501_01951_b200 import binding
    return binding


@pytest.fixture()
def ctx(mg):
    c = mg.ctx_create(0)
    yield c
    c.close()


def pack(positive):
    """numpy bool (n x d) -> uint32 words (n x ceil(d/32)), bit j & 31 of word j >> 5."""
    n, d = positive.shape
    words = (d + 31) // 32
    padded_bits = np.zeros((n, words * 32), dtype=np.uint8)
    padded_bits[:, :d] = positive
    return np.packbits(padded_bits.reshape(n, words, 32), axis=2, bitorder="little").view(np.uint32).reshape(n, words)


def words_of(t):
    return t.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("M,N,K", [(300, 47, 64), (1000, 256, 100), (777, 172, 128), (5000, 600, 520), (4100, 1024, 512)])
@pytest.mark.parametrize("prec", ["fp32", "tf32", "bf16"])
def test_product_writes_the_sign_bitmap_and_reads_a_bitmap_gate(mg, ctx, M, N, K, prec):
    P = mg.PRECISIONS[prec]
    A = synth.uniform_tensor((M, K), 700 + M, -1, 1)
    B = synth.uniform_tensor((K, N), 701 + N, -1, 1)
    bias = synth.uniform_tensor((N,), 702, -1, 1)
    Ad, Bd = padded(A), B.cuda().contiguous()
    words = (N + 31) // 32
    # forward form: bias + ReLU, sign bitmap beside the result (spare word per row must survive)
    C1 = torch.zeros(M, round4(N), device="cuda")
    bits = torch.full((M, words + 1), -1, dtype=torch.int32, device="cuda")
    mg.gemm(ctx, P, False, False, M, N, K, Ad, Bd, C1, epi=mg.make_epilogue(bias=bias.cuda(), relu=True, sign_bits=bits[:, :words]))
    C0 = torch.zeros_like(C1)
    mg.gemm(ctx, P, False, False, M, N, K, Ad, Bd, C0, epi=mg.make_epilogue(bias=bias.cuda(), relu=True))
    assert torch.equal(C0, C1)
    assert np.array_equal(words_of(bits[:, :words].contiguous()), pack(host(C1, N) > 0))
    assert torch.all(bits[:, words] == -1)
    # with a dropout mask the bitmap is that of the final values
    drop = (synth.uniform_tensor((M, N), 703, 0, 1) < 0.7).to(torch.uint8).cuda().contiguous()
    C2 = torch.zeros_like(C1); bits2 = torch.zeros(M, words, dtype=torch.int32, device="cuda")
    mg.gemm(ctx, P, False, False, M, N, K, Ad, Bd, C2,
            epi=mg.make_epilogue(bias=bias.cuda(), relu=True, drop_mask=drop, keep_scale=1 / 0.7, sign_bits=bits2))
    assert np.array_equal(words_of(bits2), pack(host(C2, N) > 0))
    # backward form: the gate read from the bitmap against the gate read from the fp32 tensor
    G0 = torch.zeros_like(C1); G1 = torch.zeros_like(C1)
    mg.gemm(ctx, P, False, False, M, N, K, Ad, Bd, G0, epi=mg.make_epilogue(gate=C1, gate_scale=1.25))
    mg.gemm(ctx, P, False, False, M, N, K, Ad, Bd, G1, epi=mg.make_epilogue(gate_bits=bits[:, :words], gate_scale=1.25))
    assert torch.equal(G0, G1)
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    with pytest.raises(mg.MixgcnError):      # the weight-gradient form takes no bit-packed mask
        mg.gemm(ctx, P, True, False, K, N, M, Ad, padded(synth.uniform_tensor((M, N), 1, -1, 1)), torch.zeros(K, round4(N), device="cuda"),
                epi=mg.make_epilogue(sign_bits=bits2))


@pytest.mark.parametrize("w", [4, 12, 47, 128, 172, 300])
def test_aggregation_with_bitmap_gate_and_sign_bitmap(mg, ctx, w):
    n = 4096
    s, d = synth.rmat_graph(n, 32768, 1001)
    go = orc.graph_build(n, s.numpy(), d.numpy())
    gg = mg.graph_create(ctx, n, s, d)
    Y = synth.uniform_tensor((n, w), 710 + w, -1, 1)
    act = synth.uniform_tensor((n, w), 711 + w, -1, 1)               # the activation whose sign is the gate
    bias = synth.uniform_tensor((w,), 712, -0.3, 0.3)
    words = (w + 31) // 32
    gate_words = torch.tensor(pack(act.numpy() > 0).view(np.int32), device="cuda")
    Z0 = torch.zeros(n, round4(w), device="cuda"); Z1 = torch.zeros_like(Z0)
    mg.spmm(ctx, gg, padded(Y), Z0, w, epi=mg.make_epilogue(gate=padded(act), gate_scale=2.0))
    mg.spmm(ctx, gg, padded(Y), Z1, w, epi=mg.make_epilogue(gate_bits=gate_words, gate_scale=2.0))
    assert torch.equal(Z0, Z1)
    want = orc.aggregate(go, Y.numpy()) * (act.numpy() > 0) * 2.0
    assert rel_fro(host(Z1, w), want) <= TOL_FP32
    bits = torch.full((n, words + 1), -1, dtype=torch.int32, device="cuda")
    Z2 = torch.zeros_like(Z0)
    mg.spmm(ctx, gg, padded(Y), Z2, w, epi=mg.make_epilogue(bias=bias.cuda(), relu=True, sign_bits=bits[:, :words]))
    assert np.array_equal(words_of(bits[:, :words].contiguous()), pack(host(Z2, w) > 0)) and torch.all(bits[:, words] == -1)
    assert rel_fro(host(Z2, w), orc.activation(orc.aggregate(go, Y.numpy()) + bias.numpy().astype(np.float64), True)) <= TOL_FP32
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    gg.close()


@pytest.mark.parametrize("precision", ["fp32", "tf32", "bf16"])
@pytest.mark.parametrize("order", ["auto", "agg", "upd"])
@pytest.mark.parametrize("dropout", [False, True])
def test_training_iteration_with_sign_bitmaps_is_bitwise_the_one_without(mg, ctx, precision, order, dropout):
    from paper_2501_01951_b200.train import GcnTrainer
    wl = synth.CONFIGS["C1"]
    s, d = synth.rmat_graph(wl.n, wl.undirected_edges, wl.seed("graph"))
    X = synth.normal_features(wl.n, wl.dims[0], wl.seed("features"))
    y = synth.uniform_labels(wl.n, wl.classes, wl.seed("labels"))
    m = synth.bernoulli_mask(wl.n, wl.mask_p, wl.seed("mask"))
    Ws, bs = synth.make_weights(wl)
    gg = mg.graph_create(ctx, wl.n, s, d)
    o = {"auto": mg.ORDER_AUTO, "agg": mg.ORDER_AGG_FIRST, "upd": mg.ORDER_UPD_FIRST}[order]
    masks = None
    if dropout:
        masks = [(synth.uniform_tensor((wl.n, wl.dims[l + 1]), 720 + l, 0, 1) < 0.8).to(torch.uint8).cuda().contiguous()
                 for l in range(len(wl.dims) - 2)]
    runs = []
    for bitmaps in (True, False):
        tr = GcnTrainer(ctx, gg, wl.dims, mg.PRECISIONS[precision], order=o, row_sparse=0, sign_bitmaps=bitmaps,
                        keep_scale=1 / 0.8 if dropout else 1.0)
        tr.set_params(Ws, bs)
        tr.set_inputs(padded(X), y.cuda(), m.cuda(), drop_masks=masks)
        tr.forward()
        if bitmaps:
            assert any(t is not None for t in tr.xbits) == (order != "upd")
            for l in range(1, tr.L):
                if tr.xbits[l] is None:
                    continue                        # produced by an aggregation: the trainer keeps the fp32 gate there
                assert np.array_equal(words_of(tr.xbits[l]), pack(host(tr.X[l], wl.dims[l]) > 0)), f"bitmap of X[{l}]"
        tr.compute_loss(); tr.backward()
        runs.append([t.clone() for t in tr.dW + tr.db] + [tr.loss.clone()])
        assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    gg.close()
