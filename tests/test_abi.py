"""CPU-side checks of the C-ABI: the library loads, exports every symbol the header declares,
its host-only logic (ordering rule) is right, and it fails loudly without a GPU."""
import ctypes as C
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mg():
    from paper_2501_01951_b200 import build
    build.build()
    from paper_2501_01951_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(mg):
    header = open(os.path.join(ROOT, "include", "mixgcn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(mixgcn_[a-z0-9_]+)\s*\(", header))
    assert declared == set(mg.SYMBOLS)
    for name in declared:
        assert getattr(mg.lib, name) is not None


def test_status_strings(mg):
    names = [mg.lib.mixgcn_status_string(i).decode() for i in range(8)]
    assert len(set(names)) == 8 and names[0] == "ok"
    assert mg.lib.mixgcn_status_string(99).decode() == "unknown status"


def test_struct_layouts_match_the_header(mg, tmp_path):
    """sizeof and every field's offset as a C compiler lays the header's structs out, against the ctypes mirror."""
    import subprocess
    checks = []
    for cname, cls in (("mixgcn_epilogue", mg.Epilogue), ("mixgcn_layer_desc", mg.LayerDesc)):
        checks.append(f'printf("{cname} %zu\\n", sizeof({cname}));')
        for field, _ in cls._fields_:
            checks.append(f'printf("{cname}.{field} %zu\\n", offsetof({cname}, {field}));')
    src = tmp_path / "layout.c"
    src.write_text('#include <stddef.h>\n#include <stdio.h>\n#include "mixgcn.h"\nint main(void) {\n' + "\n".join(checks) + "\nreturn 0; }\n")
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = dict(line.split() for line in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    for cname, cls in (("mixgcn_epilogue", mg.Epilogue), ("mixgcn_layer_desc", mg.LayerDesc)):
        assert int(out[cname]) == C.sizeof(cls), cname
        for field, _ in cls._fields_:
            assert int(out[f"{cname}.{field}"]) == getattr(cls, field).offset, f"{cname}.{field}"
    assert C.sizeof(mg.Epilogue) == 112 and C.sizeof(mg.LayerDesc) == 184      # an ABI change is a deliberate edit here too


@pytest.mark.parametrize("d_in,d_out,first,want", [
    # cost(agg-first) = c*d_in, c = 1 for a first layer else 2; cost(upd-first) = 2*d_out; ties -> agg-first
    (64, 32, True, "agg"), (32, 8, False, "upd"), (602, 256, True, "upd"), (256, 256, False, "agg"),
    (256, 41, False, "upd"), (100, 256, True, "agg"), (1024, 1024, True, "agg"), (1024, 64, False, "upd"),
    (128, 128, False, "agg"), (128, 172, False, "agg"), (512, 256, True, "agg"), (513, 256, True, "upd"),
])
def test_ordering_rule_from_the_flop_model(mg, d_in, d_out, first, want):
    d = mg.layer_desc(d_in, d_out, 4, 4, 4, flags=mg.LAYER_FIRST if first else 0)
    order, cols = mg.layer_plan(d)
    assert order == (mg.ORDER_AGG_FIRST if want == "agg" else mg.ORDER_UPD_FIRST)
    assert cols == (d_in if want == "agg" else d_out)
    d.order = mg.ORDER_UPD_FIRST
    assert mg.layer_plan(d) == (mg.ORDER_UPD_FIRST, d_out)


def test_plan_rejects_bad_descriptors(mg):
    with pytest.raises(mg.MixgcnError) as e:
        mg.layer_plan(mg.layer_desc(0, 4, 4, 4, 4))
    assert e.value.status == mg.EINVAL


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_gpu_fails_loudly(mg):
    with pytest.raises(mg.MixgcnError):
        mg.ctx_create(0)


def test_null_arguments_are_rejected_without_a_device(mg):
    assert mg.lib.mixgcn_ctx_create(None, 0) == mg.EINVAL
    assert mg.lib.mixgcn_graph_info(None, None, None, None, None) == mg.EINVAL
    assert mg.lib.mixgcn_ctx_destroy(None) == mg.OK and mg.lib.mixgcn_graph_destroy(None) == mg.OK
    assert b"null" in mg.lib.mixgcn_last_error()


def test_hot_aggregation_kernels_compile_without_register_spills(tmp_path):
    """The aggregation kernels that carry the epochs run under a register cap (four CTAs of 256 threads per SM);
    a spill there costs several per cent of an epoch, and nothing else would notice it: ask the assembler."""
    import subprocess
    from paper_2501_01951_b200 import build as b
    cmd = [b.NVCC, *b.ARCH, *b.CFLAGS, "-Xptxas", "-v", "-c", "spmm.cu", "-o", str(tmp_path / "spmm.o")]
    r = subprocess.run(cmd, capture_output=True, text=True, cwd=b.CSRC)
    assert r.returncode == 0, r.stderr[-2000:]
    log = r.stdout + r.stderr
    entries = re.findall(r"Compiling entry function '(\S+)'.*?\n.*?\n\s+\d+ bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", log)
    assert len(entries) > 50
    # every instance of the group kernel but those with the loss epilogue (third template argument 1), the short-row
    # kernel and the plain combination kernel
    hot = [(name, int(st), int(ld)) for name, st, ld in entries
           if re.search(r"spmm_group_kernelILi\d+ELi\d+ELi[023]E", name) or "spmm_short_kernel" in name or "spmm_combine_kernelILb0" in name]
    assert len(hot) >= 30
    spilled = [(name, st, ld) for name, st, ld in hot if st or ld]
    assert not spilled, spilled
