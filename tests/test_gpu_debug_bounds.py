"""The bounds-checked debug build: an index outside its range is recorded in the status word and the access
skipped -- the kernel finishes, the rest of the result is right and the context stays usable."""
import os
import subprocess
import sys

import pytest
import torch

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.gpu
def test_release_build_has_no_debug_hook():
    from paper_2501_01951_b200 import build
    build.build()
    from paper_2501_01951_b200 import binding as mg
    assert mg.build_info() == {"debug_bounds": False}
    ctx = mg.ctx_create(0)
    g = mg.graph_create(ctx, 4, torch.tensor([0, 1], dtype=torch.int32), torch.tensor([1, 2], dtype=torch.int32))
    with pytest.raises(mg.MixgcnError) as e:
        mg.debug_poke_col(g, 0, 0)
    assert e.value.status == mg.EUNSUPPORTED
    g.close(); ctx.close()


@pytest.mark.gpu
def test_bad_column_id_is_reported_and_skipped_in_the_debug_build():
    from paper_2501_01951_b200 import build
    build.build(debug=True)
    env = dict(os.environ, MIXGCN_LIBRARY="debug")
    r = subprocess.run([sys.executable, os.path.join(HERE, "debug_bounds_case.py")], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "debug-bounds case: ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
