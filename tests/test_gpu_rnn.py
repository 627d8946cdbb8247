"""Parity of csb_lstm_forward / csb_gru_forward (CUDA, through the C ABI) with the float64
oracle recurrence, including hidden and cell states after the full sequence."""
import numpy as np
import pytest
import torch

import workloads
from oracle import rnn_oracle as R
from paper_2005_05758_b200 import binding

pytestmark = pytest.mark.gpu

RTOL = {"f16": 2e-3, "f32": 1e-5}


FLOOR = {"f16": 1e-2, "f32": 0.1}   # in units of rms(want)


def close(got, want, vd, what):
    """|got - want| <= rtol * max(|want|, floor * rms(want)) element by element: relative error per
    output, with a floor where the exact state is near zero.  fp16 values (rtol 2e-3): floor
    1e-2 * rms.  fp32 values (rtol 1e-5): floor 0.1 * rms -- a state near zero comes out of sums
    that cancel (c = f*c + i*g), so its error is absolute, about one fp32 rounding (6e-8) of a
    pre-activation of size 1, and 1e-5 * 1e-2 * rms (about 1.5e-8) would sit below that single
    rounding.  Also prints the raw maximum relative error over the outputs above the floor."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    floor = FLOOR[vd] * np.sqrt(np.mean(want ** 2)) if want.size else 0.0
    tol = RTOL[vd] * np.maximum(np.abs(want), floor)
    err = np.abs(got - want)
    big = np.abs(want) > floor
    raw = float(np.max(err[big] / np.abs(want[big]))) if big.any() else 0.0
    print("%s: max relative error %.3g over %d outputs above the floor, worst error/tolerance %.3g"
          % (what, raw, int(big.sum()), float(np.max(err / np.maximum(tol, 1e-300))) if err.size else 0.0))
    assert np.all(err <= tol), "%s: worst error/tolerance %.3g" % (what, np.max(err / np.maximum(tol, 1e-300)))


def layers_of(w):
    return [(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype) for m in w.layers]


def run(w, host_io=False, chunks=None):
    """Run the library on workload w; returns y, hT, cT as numpy."""
    L, B, H, T = len(w.layers), w.B, w.hidden_size, w.T
    mats = [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, 0) for m in w.layers]
    dev = (lambda a: None if a is None else (np.ascontiguousarray(a) if host_io else torch.from_numpy(np.ascontiguousarray(a)).cuda()))
    bias = None if all(b is None for b in w.bias) else \
        [torch.from_numpy(b if b is not None else np.zeros(4 * H, np.float32)).cuda() for b in w.bias]
    new = (lambda *s: np.full(s, np.nan, np.float32) if host_io else torch.full(s, float("nan"), device="cuda"))
    flags = binding.CSB_FLAG_HOST_IO if host_io else 0
    ys = []
    h, c = dev(w.h0), dev(w.c0)
    for (t0, t1) in (chunks or [(0, T)]):
        x = dev(w.x[t0:t1])
        y, hT = new(t1 - t0, B, H), new(L, B, H)
        if w.cell == "lstm":
            cT = new(L, B, H)
            binding.csb_lstm_forward(mats, bias, x, h, c, y, hT, cT, flags)
            c = cT
        else:
            cT = None
            binding.csb_gru_forward(mats, bias, x, h, y, hT, flags)
        h = hT
        ys.append(y)
    if not host_io:
        torch.cuda.synchronize()
    tonp = (lambda a: None if a is None else (a if host_io else a.cpu().numpy()))
    out = np.concatenate([tonp(y) for y in ys]), tonp(h), tonp(c) if w.cell == "lstm" else None
    for m in mats:
        m.free()
    return out


def check(w, **kw):
    got_y, got_h, got_c = run(w, **kw)
    vd = w.layers[0].val_dtype
    if w.cell == "lstm":
        y, hT, cT = R.lstm_forward(layers_of(w), w.bias, w.x, w.h0, w.c0)
        close(got_c, cT, vd, "cT")
    else:
        y, hT = R.gru_forward(layers_of(w), w.bias, w.x, w.h0)
    close(got_y, y, vd, "y")
    close(got_h, hT, vd, "hT")
    return got_y, got_h, got_c


@pytest.mark.parametrize("cell", ["lstm", "gru"])
@pytest.mark.parametrize("vd", ["f16", "f32"])
@pytest.mark.parametrize("B", [1, 3, 8])
def test_small_stack(cell, vd, B):
    w = workloads.make_rnn_workload(21, cell, 40, 48, 2, 16, 16, "uniform", lo=0.2, hi=0.9, T=7, B=B, w_std=0.2,
                                    val_dtype=vd, bias_std=0.1, state_std=0.5)
    check(w)


@pytest.mark.parametrize("cell,I,H,br,bc", [("lstm", 153, 160, 32, 32), ("gru", 39, 100, 32, 32), ("gru", 50, 96, 64, 64),
                                            ("lstm", 1, 24, 8, 8), ("lstm", 70, 200, 64, 16)])
def test_ragged_shapes_and_boundary_straddle(cell, I, H, br, bc):
    # input sizes that are not multiples of the block width: blocks straddle the x | h boundary
    w = workloads.make_rnn_workload(5, cell, I, H, 1, br, bc, "lognormal", rate=4.0, T=9, B=2, w_std=0.15,
                                    bias_std=0.2, state_std=0.3)
    check(w)


def test_cfg1_lstm_fp32():
    check(workloads.CONFIGS["cfg1"]())


def test_cfg2_lstm_fp16_100_steps():
    check(workloads.CONFIGS["cfg2"]())


@pytest.mark.parametrize("B", [1, 8])
def test_cfg3_gru_lognormal_full_length(B):
    check(workloads.CONFIGS["cfg3"](B=B))                 # T = 256, as benchmarked


@pytest.mark.parametrize("B", [1, 32])
def test_cfg5_two_layer_full_length(B):
    # the benchmarked workload itself: 512 steps through both layers; hidden and cell states after
    # the full sequence and every output on the way are compared (the float64 oracle takes a few
    # milliseconds per step and layer here)
    check(workloads.CONFIGS["cfg5"](B=B))


def test_resume_equals_one_call_bitwise_and_host_io():
    w = workloads.make_rnn_workload(8, "lstm", 64, 128, 2, 16, 16, "uniform", lo=0.3, hi=0.7, T=12, B=2, w_std=0.1,
                                    bias_std=0.1, state_std=0.2)
    y1, h1, c1 = check(w)
    y2, h2, c2 = run(w, chunks=[(0, 5), (5, 12)])
    assert np.array_equal(y1, y2) and np.array_equal(h1, h2) and np.array_equal(c1, c2)
    y3, h3, c3 = run(w, host_io=True)
    assert np.array_equal(y1, y3) and np.array_equal(h1, h3) and np.array_equal(c1, c3)


@pytest.mark.parametrize("B,I,H,L,br,bc", [(16, 40, 48, 2, 16, 16), (32, 153, 160, 1, 32, 32), (40, 70, 192, 2, 64, 32), (8, 200, 512, 1, 32, 32)])
def test_lstm_large_batch_runs_step_by_step_on_tensor_cores(B, I, H, L, br, bc):
    # batches of 16 and more take the path of one product (tensor cores) + one gate kernel per layer
    # and step; bias, initial states, resumption and host I/O as for the persistent kernel
    w = workloads.make_rnn_workload(31, "lstm", I, H, L, br, bc, "lognormal", rate=4.0, T=6, B=B, w_std=0.15,
                                    bias_std=0.2, state_std=0.4)
    y1, h1, c1 = check(w)
    y2, h2, c2 = run(w, chunks=[(0, 2), (2, 6)])
    assert np.array_equal(y1, y2) and np.array_equal(h1, h2) and np.array_equal(c1, c2)
    y3, h3, c3 = run(w, host_io=True)
    assert np.array_equal(y1, y3) and np.array_equal(h1, h3) and np.array_equal(c1, c3)


def test_lstm_large_batch_both_paths_agree(monkeypatch):
    w = workloads.make_rnn_workload(32, "lstm", 64, 128, 2, 32, 32, "uniform", lo=0.3, hi=0.7, T=5, B=24, w_std=0.1,
                                    bias_std=0.1, state_std=0.2)
    ya, ha, ca = check(w)
    monkeypatch.setenv("CSB_RNN_NO_STEPWISE", "1")       # the persistent kernel, CUDA cores
    yb, hb, cb = check(w)
    assert np.max(np.abs(ya - yb)) < 1e-4


@pytest.mark.parametrize("cell,B,I", [("lstm", 32, 153), ("lstm", 9, 40), ("gru", 16, 70), ("gru", 11, 33)])
def test_step_by_step_packed_inputs_equal_the_fp32_buffers(monkeypatch, cell, B, I):
    # up to 32 product rows the gate kernels write h_t and x_{t+1} straight into the products' packed
    # binary16 (hi, lo) inputs; the same numbers as packing the fp32 buffers in a kernel of its own
    w = workloads.make_rnn_workload(33, cell, I, 512, 2, 32, 32, "lognormal", rate=4.0, T=5, B=B, w_std=0.15,
                                    bias_std=0.2, state_std=0.4)
    ya, ha, ca = check(w)
    monkeypatch.setenv("CSB_RNN_STEP_UNPACKED", "1")
    yb, hb, cb = check(w)
    assert np.array_equal(ya, yb) and np.array_equal(ha, hb)
    if cell == "lstm":
        assert np.array_equal(ca, cb)


@pytest.mark.parametrize("cell,B,I,H,L,br", [("lstm", 32, 153, 512, 2, 32), ("lstm", 16, 40, 48, 2, 16), ("gru", 16, 70, 512, 2, 32),
                                             ("gru", 8, 300, 512, 1, 32), ("lstm", 24, 64, 256, 3, 64)])
def test_one_launch_time_loop_equals_the_launches(monkeypatch, cell, B, I, H, L, br):
    # CSB_RNN_STEP_LOOP=1: all steps of all layers in one cooperative launch of the product kernel
    # (product pass, grid barrier, gates, grid barrier); the same arithmetic in the same order
    w = workloads.make_rnn_workload(34, cell, I, H, L, br, br, "lognormal", rate=4.0, T=9, B=B, w_std=0.15,
                                    bias_std=0.2, state_std=0.4)
    ya, ha, ca = check(w)
    monkeypatch.setenv("CSB_RNN_STEP_LOOP", "1")
    yb, hb, cb = check(w)
    assert np.array_equal(ya, yb) and np.array_equal(ha, hb)
    if cell == "lstm":
        assert np.array_equal(ca, cb)
    yc, hc, cc = run(w, chunks=[(0, 4), (4, 9)])
    assert np.array_equal(ya, yc) and np.array_equal(ha, hc)


@pytest.mark.parametrize("B,I,H,L,br,bc", [(16, 40, 48, 2, 16, 16), (20, 39, 100, 1, 32, 32), (33, 70, 192, 2, 64, 32), (8, 300, 512, 1, 32, 32)])
def test_gru_batch_runs_step_by_step_on_tensor_cores(B, I, H, L, br, bc):
    # GRU from batch 16 (from batch 8 for layers of 100 k weights and more): one product over 2B rows ([u ; 0] and [0 ; h]) keeps the candidate's two parts apart
    w = workloads.make_rnn_workload(41, "gru", I, H, L, br, bc, "lognormal", rate=4.0, T=6, B=B, w_std=0.15,
                                    bias_std=0.2, state_std=0.4)
    y1, h1, _ = check(w)
    y2, h2, _ = run(w, chunks=[(0, 2), (2, 6)])
    assert np.array_equal(y1, y2) and np.array_equal(h1, h2)
    y3, h3, _ = run(w, host_io=True)
    assert np.array_equal(y1, y3) and np.array_equal(h1, h3)


@pytest.mark.parametrize("cell,B", [("gru", 8), ("lstm", 16)])
def test_persistent_kernel_still_serves_these_batches(monkeypatch, cell, B):
    monkeypatch.setenv("CSB_RNN_NO_STEPWISE", "1")
    w = workloads.make_rnn_workload(42, cell, 40, 48, 2, 16, 16, "uniform", lo=0.2, hi=0.9, T=7, B=B, w_std=0.2,
                                    bias_std=0.1, state_std=0.5)
    check(w)


def test_two_streams_in_turn_agree_bitwise():
    # calls on the same matrices share cached device state, so they must not overlap; in turn, with
    # an event between them, two streams give the same bits
    w = workloads.make_rnn_workload(8, "lstm", 64, 128, 2, 16, 16, "uniform", lo=0.3, hi=0.7, T=12, B=2, w_std=0.1,
                                    bias_std=0.1, state_std=0.2)
    mats = [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, 0) for m in w.layers]
    x, h0, c0 = (torch.from_numpy(a).cuda() for a in (w.x, w.h0, w.c0))
    bias = [torch.from_numpy(b).cuda() for b in w.bias]
    outs = []
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    ev = None
    for st in (s1, s2):
        y = torch.full((w.T, w.B, w.hidden_size), float("nan"), device="cuda")
        hT = torch.full((2, w.B, w.hidden_size), float("nan"), device="cuda")
        cT = torch.full((2, w.B, w.hidden_size), float("nan"), device="cuda")
        if ev is not None:
            st.wait_event(ev)
        binding.csb_lstm_forward(mats, bias, x, h0, c0, y, hT, cT, binding.CSB_FLAG_ASYNC, stream=st)
        ev = torch.cuda.Event()
        ev.record(st)
        outs.append((y, hT, cT))
    torch.cuda.synchronize()
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    want, _, _ = R.lstm_forward(layers_of(w), w.bias, w.x, w.h0, w.c0)
    close(outs[1][0].cpu().numpy(), want, "f16", "y")
    for m in mats:
        m.free()


def test_zero_weight_closed_forms():
    w = workloads.make_rnn_workload(2, "gru", 16, 32, 1, 8, 8, "uniform", lo=0.5, hi=0.5, T=6, B=2, w_std=0.1, state_std=1.0)
    w.layers[0].dense[:] = 0
    y, hT, _ = run(w)
    assert np.array_equal(hT[0], w.h0[0] / np.float32(64.0))       # r = z = 1/2, n = 0: h halves every step
    w = workloads.make_rnn_workload(2, "lstm", 16, 32, 1, 8, 8, "uniform", lo=0.5, hi=0.5, T=6, B=2, w_std=0.1)
    w.layers[0].dense[:] = 0
    y, hT, cT = run(w)
    assert not y.any() and not hT.any() and not cT.any()


def test_shape_errors_and_noops():
    w = workloads.make_rnn_workload(2, "lstm", 16, 32, 1, 8, 8, "uniform", lo=0.5, hi=0.5, T=2, B=1, w_std=0.1)
    m = w.layers[0]
    A = binding.csb_encode(m.dense, 8, 8, m.row_keep, m.col_keep, "f16", 0)
    x = torch.zeros(2, 1, 16, device="cuda")
    y = torch.zeros(2, 1, 32, device="cuda")
    with pytest.raises(binding.CsbError) as e:
        binding.csb_gru_forward([A], None, x, None, y, None)          # 128 rows are not 3 * H
    assert e.value.status == -2
    with pytest.raises(binding.CsbError) as e:
        binding.csb_lstm_forward([A, A], None, x, None, None, y, None, None)   # layer 1 input must be H wide
    assert e.value.status == -2
    binding.csb_lstm_forward([A], None, x[:0], None, None, None, None, None)    # T = 0: nothing to do
    A.free()


def test_barrier_gives_up_and_context_survives():
    w = workloads.make_rnn_workload(2, "lstm", 16, 32, 1, 8, 8, "uniform", lo=0.5, hi=0.5, T=4, B=1, w_std=0.1)
    m = w.layers[0]
    A = binding.csb_encode(m.dense, 8, 8, m.row_keep, m.col_keep, "f16", 0)
    x = torch.from_numpy(w.x).cuda()
    y = torch.zeros(4, 1, 32, device="cuda")
    binding.lib.csb_test_barrier_hook(1, 200_000)          # one arrival never comes; give up after 200 us
    try:
        with pytest.raises(binding.CsbError) as e:
            binding.csb_lstm_forward([A], None, x, None, None, y, None, None)
        assert e.value.status == -7
    finally:
        binding.lib.csb_test_barrier_hook(0, 0)
    binding.csb_lstm_forward([A], None, x, None, None, y, None, None)            # same context still works
    torch.cuda.synchronize()
    want, _, _ = R.lstm_forward(layers_of(w), w.bias, w.x)
    close(y.cpu().numpy(), want, "f16", "y after timeout")
    A.free()
