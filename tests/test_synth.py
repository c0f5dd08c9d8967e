"""The seeded input generators: determinism, chunk independence, basic distribution sanity."""
import numpy as np
import torch

from paper_2501_01951_b200 import synth


def test_rmat_is_deterministic_and_well_formed():
    s1, d1 = synth.rmat_graph(4096, 32768, 1001)
    s2, d2 = synth.rmat_graph(4096, 32768, 1001)
    assert torch.equal(s1, s2) and torch.equal(d1, d2)
    assert s1.dtype == torch.int32 and len(s1) >= 32768 and len(s1) < 32768 + 4096 * 2
    assert torch.all(s1 < d1) and int(d1.max()) < 4096 and int(s1.min()) >= 0
    keys = s1.long() * 4096 + d1.long()
    assert len(torch.unique(keys)) == len(keys)
    s3, _ = synth.rmat_graph(4096, 32768, 1002)
    assert not torch.equal(s1[:100], s3[:100])
    deg = torch.bincount(torch.cat([s1, d1]).long(), minlength=4096)
    assert deg.max() > 20 * deg.float().mean()          # heavy tail


def test_candidates_do_not_depend_on_chunking():
    u, v = synth.rmat_candidates(5, 0, 1000, 12)
    u2, v2 = synth.rmat_candidates(5, 400, 300, 12)
    assert torch.equal(u[400:700], u2) and torch.equal(v[400:700], v2)


def test_scramble_is_a_bijection():
    for s in (1, 5, 12, 18):
        x = torch.arange(1 << s, dtype=torch.int64)
        y = synth._scramble_ids(x, s, 77)
        assert len(torch.unique(y)) == 1 << s and int(y.max()) < (1 << s) and int(y.min()) >= 0


def test_features_labels_masks_weights():
    X = synth.normal_features(3000, 20, 9, ld=24)
    assert X.shape == (3000, 24) and torch.all(X[:, 20:] == 0)
    assert abs(float(X[:, :20].mean())) < 0.02 and abs(float(X[:, :20].std()) - 1) < 0.02
    Xc = synth.normal_features(3000, 20, 9, ld=24, rows_per_chunk=777)
    assert torch.equal(X, Xc)
    y = synth.uniform_labels(10000, 41, 3)
    assert y.dtype == torch.int32 and int(y.min()) == 0 and int(y.max()) == 40
    m = synth.bernoulli_mask(100000, 0.08, 4)
    assert m.dtype == torch.uint8 and abs(float(m.float().mean()) - 0.08) < 0.005
    W = synth.glorot_uniform(100, 256, 5)
    a = (6 / 356) ** 0.5
    assert W.shape == (100, 256) and float(W.abs().max()) <= a and float(W.abs().max()) > 0.99 * a
    Ws, bs = synth.make_weights(synth.CONFIGS["C1"])
    assert [tuple(w.shape) for w in Ws] == [(64, 32), (32, 8)] and all(float(b.abs().sum()) == 0 for b in bs)
