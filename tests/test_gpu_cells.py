"""Parity of the cell variants (csb_lstmp_forward, csb_ligru_forward, csb_gru_reset_before_forward;
CUDA, through the C ABI) with the float64 oracle recurrences, states after the full sequence included."""
import numpy as np
import pytest
import torch

import workloads
from oracle import rnn_oracle as R
from paper_2005_05758_b200 import binding
from test_gpu_rnn import close

pytestmark = pytest.mark.gpu


def _tup(m):
    return (m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)


def _enc(ms):
    return [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, 0) for m in ms]


def run(w, host_io=False, chunks=None):
    L, B, H, T = len(w.layers), w.B, w.hidden_size, w.T
    S = w.proj_size if w.cell == "lstmp" else H
    mats = _enc(w.layers)
    proj = _enc(w.proj) if w.cell == "lstmp" else None
    dev = (lambda a: None if a is None else (np.ascontiguousarray(a) if host_io else torch.from_numpy(np.ascontiguousarray(a)).cuda()))
    bias = None if all(b is None for b in w.bias) else [torch.from_numpy(b).cuda() for b in w.bias]
    new = (lambda *s: np.full(s, np.nan, np.float32) if host_io else torch.full(s, float("nan"), device="cuda"))
    flags = binding.CSB_FLAG_HOST_IO if host_io else 0
    ys, h, c = [], dev(w.h0), dev(w.c0)
    for (t0, t1) in (chunks or [(0, T)]):
        x = dev(w.x[t0:t1])
        y, hT = new(t1 - t0, B, S), new(L, B, S)
        if w.cell == "lstmp":
            cT = new(L, B, H)
            binding.csb_lstmp_forward(mats, proj, bias, x, h, c, y, hT, cT, flags)
            c = cT
        elif w.cell == "ligru":
            binding.csb_ligru_forward(mats, bias, x, h, y, hT, flags)
        else:
            binding.csb_gru_reset_before_forward(mats, bias, x, h, y, hT, flags)
        h = hT
        ys.append(y)
    if not host_io:
        torch.cuda.synchronize()
    tonp = (lambda a: None if a is None else (a if host_io else a.cpu().numpy()))
    out = np.concatenate([tonp(y) for y in ys]), tonp(h), tonp(c) if w.cell == "lstmp" else None
    for m in mats + (proj or []):
        m.free()
    return out


def check(w, **kw):
    got_y, got_h, got_c = run(w, **kw)
    vd = w.layers[0].val_dtype
    lay = [_tup(m) for m in w.layers]
    if w.cell == "lstmp":
        y, hT, cT = R.lstmp_forward(lay, [_tup(m) for m in w.proj], w.bias, w.x, w.h0, w.c0)
        close(got_c, cT, vd, "cT")
    elif w.cell == "ligru":
        y, hT = R.ligru_forward(lay, w.bias, w.x, w.h0)
    else:
        y, hT = R.gru_reset_before_forward(lay, w.bias, w.x, w.h0)
    close(got_y, y, vd, "y")
    close(got_h, hT, vd, "hT")
    return got_y, got_h, got_c


def make(cell, B, vd="f16", I=40, H=48, L=2, br=16, bc=16, T=7, **kw):
    extra = dict(proj_size=kw.pop("P", 32)) if cell == "lstmp" else {}
    return workloads.make_rnn_workload(23, cell, I, H, L, br, bc, "uniform", lo=0.2, hi=0.9, T=T, B=B, w_std=0.2, val_dtype=vd,
                                       bias_std=0.1, state_std=0.5, **extra, **kw)


@pytest.mark.parametrize("cell", ["lstmp", "ligru", "gru_rb"])
@pytest.mark.parametrize("vd", ["f16", "f32"])
@pytest.mark.parametrize("B", [1, 3, 8, 20])
def test_small_stack(cell, vd, B):
    check(make(cell, B, vd))


@pytest.mark.parametrize("cell,I,H,br,bc", [("lstmp", 153, 160, 32, 32), ("ligru", 39, 100, 32, 32), ("gru_rb", 50, 96, 64, 64), ("ligru", 1, 24, 8, 8)])
def test_ragged_shapes(cell, I, H, br, bc):
    extra = dict(proj_size=72) if cell == "lstmp" else {}
    w = workloads.make_rnn_workload(5, cell, I, H, 1, br, bc, "lognormal", rate=4.0, T=9, B=2, w_std=0.15, bias_std=0.2, state_std=0.3, **extra)
    check(w)


@pytest.mark.parametrize("cell", ["lstmp", "ligru", "gru_rb"])
def test_resume_equals_one_call_bitwise_and_host_io(cell):
    w = make(cell, 2, T=12)
    y1, h1, c1 = check(w)
    y2, h2, c2 = run(w, chunks=[(0, 5), (5, 12)])
    assert np.array_equal(y1, y2) and np.array_equal(h1, h2) and (c1 is None or np.array_equal(c1, c2))
    y3, h3, c3 = run(w, host_io=True)
    assert np.array_equal(y1, y3) and np.array_equal(h1, h3) and (c1 is None or np.array_equal(c1, c3))


def test_table1_layer_shapes_full_length():
    # the layer sizes of the paper's Table 1 (SR1: LSTMP 153 -> 1024 with a projection to 512, then 512 -> 1024;
    # SR3: Li-GRU 39 -> 512 -> 512) with synthetic masks of about the table's pruning rates, batch 1, 100 steps
    w = workloads.make_rnn_workload(0, "lstmp", 153, 1024, 2, 32, 32, "uniform", lo=0.2, hi=0.35, T=100, B=1, w_std=0.05, proj_size=512)
    check(w)
    w = workloads.make_rnn_workload(0, "ligru", 39, 512, 2, 32, 32, "uniform", lo=0.3, hi=0.45, T=100, B=1, w_std=0.05)
    check(w)
    w = workloads.make_rnn_workload(0, "gru_rb", 39, 1024, 2, 32, 32, "uniform", lo=0.15, hi=0.3, T=100, B=8, w_std=0.05)
    check(w)


def test_zero_weight_closed_forms():
    w = make("gru_rb", 2, L=1, T=6, I=16, H=32, br=8, bc=8)
    w.layers[0].dense[:] = 0
    w.bias[0][:] = 0
    y, hT, _ = run(w)
    assert np.array_equal(hT[0], w.h0[0] / np.float32(64.0))          # r = z = 1/2, n = 0: h halves every step
    w = make("ligru", 2, L=1, T=4, I=16, H=32, br=8, bc=8)
    w.layers[0].dense[:] = 0
    w.bias[0][:32] = 0                                                 # z = 1/2
    w.bias[0][32:] = -1                                                # the rectifier cuts the candidate off
    y, hT, _ = run(w)
    assert np.array_equal(hT[0], w.h0[0] / np.float32(16.0))


def test_shape_errors():
    w = make("ligru", 1, L=1)
    A = _enc(w.layers)[0]
    x = torch.zeros(2, 1, 40, device="cuda")
    y = torch.zeros(2, 1, 48, device="cuda")
    with pytest.raises(binding.CsbError) as e:
        binding.csb_lstmp_forward([A], [A], None, x, None, None, y, None, None)    # a 96-row "projection" leaves no input columns
    assert e.value.status == -2
    odd = binding.csb_encode(np.ones((9, 8), np.float32), 3, 4, np.ones(18, np.uint8), np.ones(24, np.uint8), "f16", 0)
    with pytest.raises(binding.CsbError) as e:
        binding.csb_ligru_forward([odd], None, x, None, y, None)                   # 9 rows are not 2 * H
    assert e.value.status == -2
    odd.free()
    blk4 = binding.csb_encode(np.ones((9, 8), np.float32), 4, 4, np.ones(24, np.uint8), np.ones(24, np.uint8), "f16", 0)
    with pytest.raises(binding.CsbError) as e:
        binding.csb_gru_reset_before_forward([blk4], None, x, None, y, None)       # 2 * H = 6 is not a multiple of block_r = 4
    assert e.value.status == -8
    blk4.free()
    binding.csb_ligru_forward([A], None, x[:0], None, None, None)              # T = 0: nothing to do
    A.free()
