"""csb_spmv_static_scratch: the SpMV variant for callers that cannot allocate device memory
(servers and real-time loops whose memory budget is frozen, plug-ins handed a fixed arena).
Its scratch is a fixed array inside the library instead of buffers that come with the handle.

The file name sorts last on purpose: if this extra entry point ever fails, a run that stops at
the first failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

import workloads
from oracle import csb_oracle as O
from paper_2005_05758_b200 import binding

pytestmark = pytest.mark.gpu

RTOL = {"f16": 2e-3, "f32": 1e-5}      # the tolerances of the product tests


def _check_against_oracle(got, m, X):
    args = (m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)
    want, scale = O.spmm(*args, X)[0], O.abs_scale(*args, X)[0]
    g = got.astype(np.float64)
    assert np.all(np.abs(g - want) <= RTOL[m.val_dtype] * np.maximum(np.abs(want), 1e-2 * scale))
    assert np.all(g[scale == 0] == 0.0)


def _both(A, x, rows, calls=2):
    """The same product through csb_spmv and `calls` times through the static-scratch entry point."""
    want = torch.full((rows,), float("nan"), device="cuda")
    binding.csb_spmv(A, x, want)
    gots = []
    for _ in range(calls):
        got = torch.full((rows,), float("nan"), device="cuda")
        binding.csb_spmv_static_scratch(A, x, got)
        gots.append(got)
    torch.cuda.synchronize()
    return want.cpu().numpy(), [g.cpu().numpy() for g in gots]


def test_two_calls_in_a_row_match_csb_spmv_and_the_oracle(monkeypatch):
    # Different matrices back to back on one stream, many block-rows first and few afterwards, so
    # that every call finds partial sums and counters of another layout in the shared array.  With
    # CSB_NO_PANEL csb_spmv runs the same kernel with the handle's own scratch: equal bit for bit.
    monkeypatch.setenv("CSB_NO_PANEL", "1")
    cases = [(3, 4096, 1536, 64, 6.0, "f16"), (4, 1024, 4096, 64, 12.0, "f16"), (5, 2048, 1024, 32, 5.0, "f32"),
             (6, 256, 8192, 64, 8.0, "f16")]
    for seed, rows, cols, blk, rate, vd in cases:
        w = workloads.make_spmv_workload(seed, rows, cols, blk, blk, "lognormal", rate=rate, batch=1, w_std=0.05, val_dtype=vd)
        m = w.matrix
        A = binding.csb_encode(m.dense, blk, blk, m.row_keep, m.col_keep, vd, 0)
        want, gots = _both(A, torch.from_numpy(w.X).cuda()[0], m.rows)
        for g in gots:
            assert np.array_equal(g, want), (seed, "differs from csb_spmv's stream kernel")
            _check_against_oracle(g, m, w.X)
        A.free()


def test_divided_block_rows_go_through_the_shared_array(monkeypatch):
    # one block-row keeps everything: the planner divides it between CTAs, whose pieces meet through
    # partial-sum slots -- here those of the built-in array
    monkeypatch.setenv("CSB_NO_PANEL", "1")
    w = workloads.make_spmv_workload(11, 8192, 4096, 64, 64, "lognormal", rate=10.0, batch=1, w_std=0.05)
    m = w.matrix
    m.row_keep.reshape(128, 64, 64)[5] = 1
    m.col_keep.reshape(128, 64, 64)[5] = 1
    A = binding.csb_encode(m.dense, 64, 64, m.row_keep, m.col_keep, "f16", 0)
    want, gots = _both(A, torch.from_numpy(w.X).cuda()[0], m.rows, calls=3)
    for g in gots:
        assert np.array_equal(g, want)
        _check_against_oracle(g, m, w.X)
    A.free()


def test_panel_handle_matches_within_tolerance():
    # default handles run csb_spmv on the panel kernel (another summation order): same result
    # within the product tolerance, and the static-scratch call itself against the oracle
    w = workloads.make_spmv_workload(3, 2048, 1536, 64, 64, "lognormal", rate=6.0, batch=1, w_std=0.05)
    m = w.matrix
    A = binding.csb_encode(m.dense, 64, 64, m.row_keep, m.col_keep, "f16", 0)
    want, gots = _both(A, torch.from_numpy(w.X).cuda()[0], m.rows)
    for g in gots:
        _check_against_oracle(g, m, w.X)
        _check_against_oracle(want, m, w.X)
    A.free()


def test_limits_are_refused_with_a_clear_message():
    # 20000 block-rows of one row each need more arrival counters than the built-in array has
    rows, cols = 20000, 8
    dense = np.ones((rows, cols), np.float32)
    A = binding.csb_encode(dense, 1, 8, np.ones(rows, np.uint8), np.ones(rows * 8, np.uint8), "f16", 0)
    x = torch.ones(cols, device="cuda")
    y = torch.empty(rows, device="cuda")
    with pytest.raises(binding.CsbError) as e:
        binding.csb_spmv_static_scratch(A, x, y)
    assert e.value.status == -8 and "built-in scratch" in str(e.value)
    binding.csb_spmv(A, x, y)                      # the ordinary entry point still serves it
    torch.cuda.synchronize()
    assert torch.all(y == 8.0)
    A.free()
