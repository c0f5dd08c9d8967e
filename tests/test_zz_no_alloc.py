"""The allocation-free loss entry point against the regular one.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has
already run every other test.  It must pass alone in a fresh process and after the other tests."""
import numpy as np
import pytest
import torch

from oracle import gcn_oracle as orc
from paper_2501_01951_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mg():
    from paper_2501_01951_b200 import build
    build.build()
    from paper_2501_01951_b200 import binding
    return binding


def _outputs(n, ld, dev):
    return dict(loss=torch.full((1,), -1.0, device=dev), G=torch.full((n, ld), 5.0, device=dev),
                pred=torch.full((n,), -1, dtype=torch.int32, device=dev),
                nc=torch.full((1,), -1, dtype=torch.int64, device=dev))


def test_noalloc_loss_matches_the_regular_entry_point_twice(mg):
    """Two calls in a row (different inputs, so stale scratch contents would show) against
    mixgcn_loss_softmax_xent: same kernels, so the loss agrees to 1e-6 relative (the partial sums are
    grouped differently), the gradient and the integer outputs exactly.  Each call is also held to the
    CPU oracle within the fp32 tolerance."""
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = mg.ctx_create(0)
    for call, (n, Cc, p) in enumerate([(5000, 41, 0.5), (3333, 172, 0.1)]):
        ld = (Cc + 3) // 4 * 4
        P = torch.zeros(n, ld, device=dev)
        P[:, :Cc] = synth.uniform_tensor((n, Cc), 900 + call, -5, 5).to(dev)
        y = synth.uniform_labels(n, Cc, 901 + call).to(dev)
        m = synth.bernoulli_mask(n, p, 902 + call).to(dev)
        a, b = _outputs(n, ld, dev), _outputs(n, ld, dev)
        st = torch.full((1,), -1, dtype=torch.int32, device=dev)
        mg.loss_softmax_xent(ctx, P, y, m, a["loss"], a["G"], a["pred"], a["nc"], C_=Cc)
        mg.loss_softmax_xent_noalloc(P, y, m, b["loss"], b["G"], b["pred"], b["nc"], st, C_=Cc)
        torch.cuda.synchronize()
        assert abs(a["loss"].item() - b["loss"].item()) <= 1e-6 * abs(a["loss"].item())
        assert torch.equal(a["G"], b["G"]) and torch.equal(a["pred"], b["pred"]) and torch.equal(a["nc"], b["nc"])
        assert st.item() == 0
        # and against the CPU oracle, like the regular entry point's own parity test
        lo, G, pred, nc, _ = orc.loss(P[:, :Cc].cpu().numpy(), y.cpu().numpy(), m.cpu().numpy())
        assert abs(b["loss"].item() - lo) <= 1e-6 * max(1.0, abs(lo))
        Gb = b["G"][:, :Cc].cpu().numpy().astype(np.float64)
        assert np.linalg.norm(Gb - G) <= 1e-5 * np.linalg.norm(G)
        assert np.array_equal(b["pred"].cpu().numpy(), pred) and b["nc"].item() == nc
    # device-visible errors come back through the caller's status word, and the next call starts clean
    n, Cc = 64, 5
    P = torch.zeros(n, 8, device=dev); y = torch.zeros(n, dtype=torch.int32, device=dev)
    out = _outputs(n, 8, dev); st = torch.zeros(1, dtype=torch.int32, device=dev)
    mg.loss_softmax_xent_noalloc(P, y, torch.zeros(n, dtype=torch.uint8, device=dev), out["loss"], out["G"], None, None, st, C_=Cc)
    assert st.item() == 1 and out["loss"].item() == 0
    mg.loss_softmax_xent_noalloc(P, y, torch.ones(n, dtype=torch.uint8, device=dev), out["loss"], out["G"], None, None, st, C_=Cc)
    assert st.item() == 0 and abs(out["loss"].item() - 1.6094379) < 1e-5
    assert mg.ctx_poll_status(ctx, raise_on_error=False) == 0
    ctx.close()


def test_noalloc_loss_rejects_sizes_beyond_its_scratch(mg):
    dev = torch.device("cuda", 0)
    P = torch.zeros(8, 4, device=dev); y = torch.zeros(8, dtype=torch.int32, device=dev)
    m = torch.ones(8, dtype=torch.uint8, device=dev); loss = torch.full((1,), 7.0, device=dev)
    rc = mg.lib.mixgcn_loss_softmax_xent_noalloc(mg.C.c_int64(33_554_433), mg.C.c_int32(4), mg.C.c_void_p(P.data_ptr()),
                                                 mg.C.c_int64(4), mg.C.c_void_p(y.data_ptr()), mg.C.c_void_p(m.data_ptr()),
                                                 mg.C.c_void_p(loss.data_ptr()), None, None, None, None, None)
    assert rc == mg.EUNSUPPORTED and b"exceeds" in mg.lib.mixgcn_last_error()
    torch.cuda.synchronize()
    assert loss.item() == 7.0                       # nothing was launched
