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
from paper_2005_05758_b200 import binding

pytestmark = pytest.mark.gpu

RTOL = 2e-3      # the tolerance of the fp16-value product tests


def _matrix(seed, rows, cols, rate):
    w = workloads.make_spmv_workload(seed, rows, cols, 64, 64, "lognormal", rate=rate, batch=1, w_std=0.05)
    m = w.matrix
    return binding.csb_encode(m.dense, 64, 64, m.row_keep, m.col_keep, "f16", 0), torch.from_numpy(w.X).cuda(), m


def test_two_calls_in_a_row_match_csb_spmv():
    # two different matrices back to back on one stream: the second call finds the first one's
    # leftovers in the shared array and must not be disturbed by them
    for seed, rows, cols, rate in ((3, 2048, 1536, 6.0), (4, 1024, 4096, 12.0)):
        A, x, m = _matrix(seed, rows, cols, rate)
        want = torch.full((m.rows,), float("nan"), device="cuda")
        binding.csb_spmv(A, x[0], want)
        for call in range(2):
            got = torch.full((m.rows,), float("nan"), device="cuda")
            binding.csb_spmv_static_scratch(A, x[0], got)
            torch.cuda.synchronize()
            g, w = got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(g))
            scale = max(float(np.sqrt(np.mean(w ** 2))), 1e-30)
            assert np.all(np.abs(g - w) <= RTOL * np.maximum(np.abs(w), 1e-2 * scale)), (seed, call)
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
