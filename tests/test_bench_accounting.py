"""The byte and FLOP accounting behind bench.py's roofline figures, checked by hand on small cases
(host logic only; no GPU)."""
import importlib.util
import os
import types

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    from paper_2501_01951_b200 import build
    build.build()
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _wl(dims):
    return types.SimpleNamespace(dims=tuple(dims))


def test_spmm_plan_counts_dense_input_calls(bench):
    from paper_2501_01951_b200 import binding as mg
    A, U = mg.ORDER_AGG_FIRST, mg.ORDER_UPD_FIRST
    wl = _wl((128, 128, 128, 172))
    # agg-first everywhere: forward aggregates at d_in; the first layer's backward needs no aggregation
    assert bench.spmm_plan(wl, [A, A, A], 0) == [(128, 1), (128, 2), (128, 2)]
    # the top two layers' backward aggregations take the row-sparse path
    assert bench.spmm_plan(wl, [A, A, A], 2) == [(128, 1), (128, 1), (128, 1)]
    # and the last layer's forward aggregation runs on train rows only
    assert bench.spmm_plan(wl, [A, A, A], 2, True) == [(128, 1), (128, 1), (128, 0)]
    # update-first aggregates at d_out, forward and backward, first layer included
    assert bench.spmm_plan(_wl((602, 256, 41)), [U, U], 0) == [(256, 2), (41, 2)]


def test_spmm_algorithmic_bytes(bench):
    # 3 rows, 5 stored entries, width 4: row pointers 4 x 8, column ids and values 5 x 4 each,
    # one read of the 3 x 4 input and one write of the 3 x 4 output
    assert bench.spmm_alg_bytes(3, 5, 4) == 32 + 20 + 20 + 48 + 48


def test_gemm_flops_and_bytes(bench):
    from paper_2501_01951_b200 import binding as mg
    A = mg.ORDER_AGG_FIRST
    n, dims = 10, (4, 3, 2)
    # layer 0: forward + dW; layer 1: forward + dW + dX; each product 2 * rows * d_in * d_out
    assert bench.gemm_flops(n, dims, [A, A]) == 2 * 10 * 4 * 3 * 2 + 2 * 10 * 3 * 2 * 3
    # last layer's backward on 5 compacted rows
    assert bench.gemm_flops(n, dims, [A, A], [None, 5]) == 2 * 10 * 4 * 3 * 2 + 2 * 10 * 3 * 2 + 2 * (2 * 5 * 3 * 2)
    # ... and its forward too
    assert bench.gemm_flops(n, dims, [A, A], [None, 5], 5) == 2 * 10 * 4 * 3 * 2 + 3 * (2 * 5 * 3 * 2)
    # first layer's backward (dW only) on 2 rows
    assert bench.gemm_flops(n, dims, [A, A], [2, None]) == 2 * 4 * 3 * (10 + 2) + 2 * 10 * 3 * 2 * 3
    # bytes: every rows x d operand and result once per product
    assert bench.gemm_min_bytes(n, dims) == 4 * 10 * (4 + 3) * 2 + 4 * 10 * (3 + 2) * 3
    assert bench.gemm_min_bytes(n, dims, [None, 5]) == 4 * 10 * (4 + 3) * 2 + 4 * 10 * (3 + 2) + 2 * 4 * 5 * (3 + 2)
    assert bench.gemm_min_bytes(n, dims, [None, 5], 5) == 4 * 10 * (4 + 3) * 2 + 3 * 4 * 5 * (3 + 2)


def test_peaks_are_read_from_the_measured_file_or_fall_back(bench):
    p = bench.load_peaks()
    assert p["source"] in ("measured", "fallback") and p["hbm_gbs"] > 1000 and p["bf16_tflops"] > 100


def test_ideal_static_cache_floor_by_hand(bench):
    import torch
    # 6 rows of width 4 (16-byte rows): pretend the cache holds 2 rows.  Rows are gathered 5, 3, 1, 1, 0, 0
    # times (10 stored entries).  Cached: the rows gathered 5 and 3 times -> 2 reads; the two rows gathered
    # once -> 2 reads; nothing else.  Bytes: row pointers 8*7, ids + values 8*10, output 4*6*4, gathers 16*4.
    old = bench.L2_BYTES
    bench.L2_BYTES = 2 * 16
    try:
        deg = torch.tensor([1, 5, 0, 3, 1, 0], dtype=torch.int32)
        floor, k, hit = bench.ideal_cache_floor(deg, 6, 10, 4)
    finally:
        bench.L2_BYTES = old
    assert k == 2 and abs(hit - 0.8) < 1e-12
    assert floor == 8 * 7 + 8 * 10 + 4 * 6 * 4 + 16 * (2 + 2)


def test_tensor_peak_labels(bench):
    peaks = dict(bf16_tflops=1600.0, bf16_tflops_sustained=1300.0, source="measured")
    assert bench.gemm_peak_for("bf16", peaks, None)[0] == 1600.0
    assert bench.gemm_peak_for("tf32", peaks, dict(tf32_tflops_measured=700.0))[0] == 700.0
    assert abs(bench.gemm_peak_for("tf32", peaks, None)[0] - 1600.0 * 1.1 / 2.25) < 1e-9
    assert bench.gemm_peak_for("fp32", peaks, None)[0] is None
