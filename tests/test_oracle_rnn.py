"""Pins for the recurrent oracle (CPU only): an independent library cell,
closed forms for zero weights, and structural invariants."""
import numpy as np
import pytest
import torch

import workloads
from oracle import csb_oracle as O
from oracle import rnn_oracle as R


def _layers(w):
    return [(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype) for m in w.layers]


def _small(cell, L=2, B=3, T=5, I=20, H=24, seed=11, vd="f16", bias_std=0.1, state_std=0.5):
    return workloads.make_rnn_workload(seed, cell, I, H, L, 8, 8, "uniform", lo=0.3, hi=0.8, T=T, B=B,
                                       w_std=0.3, val_dtype=vd, bias_std=bias_std, state_std=state_std)


def _torch_cell(cell, w):
    """torch.nn.LSTM / GRU in float64 holding the masked dense weights."""
    H, I, L = w.hidden_size, w.input_size, len(w.layers)
    G = 4 if cell == "lstm" else 3
    net = (torch.nn.LSTM if cell == "lstm" else torch.nn.GRU)(I, H, num_layers=L).double()
    with torch.no_grad():
        for l, m in enumerate(w.layers):
            Wm = torch.from_numpy(O.masked_dense(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep,
                                                 m.val_dtype))
            in_l = I if l == 0 else H
            getattr(net, "weight_ih_l%d" % l).copy_(Wm[:, :in_l])
            getattr(net, "weight_hh_l%d" % l).copy_(Wm[:, in_l:])
            b = torch.zeros(4 * H, dtype=torch.float64) if w.bias[l] is None else \
                torch.from_numpy(w.bias[l].astype(np.float64))
            bih, bhh = torch.zeros(G * H, dtype=torch.float64), torch.zeros(G * H, dtype=torch.float64)
            if cell == "lstm":
                bih.copy_(b)
            else:                       # b_r, b_z go to the input side; b_in / b_hn stay apart
                bih[:3 * H] = b[:3 * H]
                bhh[2 * H:] = b[3 * H:]
            getattr(net, "bias_ih_l%d" % l).copy_(bih)
            getattr(net, "bias_hh_l%d" % l).copy_(bhh)
    return net


@pytest.mark.parametrize("vd", ["f16", "f32"])
def test_lstm_matches_torch_float64(vd):
    w = _small("lstm", vd=vd)
    y, hT, cT = R.lstm_forward(_layers(w), w.bias, w.x, w.h0, w.c0)
    net = _torch_cell("lstm", w)
    with torch.no_grad():
        ty, (th, tc) = net(torch.from_numpy(w.x).double(),
                           (torch.from_numpy(w.h0).double(), torch.from_numpy(w.c0).double()))
    np.testing.assert_allclose(y, ty.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(hT, th.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(cT, tc.numpy(), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("vd", ["f16", "f32"])
def test_gru_matches_torch_float64(vd):
    w = _small("gru", vd=vd)
    y, hT = R.gru_forward(_layers(w), w.bias, w.x, w.h0)
    net = _torch_cell("gru", w)
    with torch.no_grad():
        ty, th = net(torch.from_numpy(w.x).double(), torch.from_numpy(w.h0).double())
    np.testing.assert_allclose(y, ty.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(hT, th.numpy(), rtol=1e-12, atol=1e-13)


def _zero_weight(w):
    for m in w.layers:
        m.dense[:] = 0
    return w


def test_zero_weight_closed_forms():
    # LSTM, W = 0, b = 0, zero state: every gate pre-activation is 0, c stays 0, h stays 0.
    w = _zero_weight(_small("lstm", L=1, bias_std=0.0, state_std=0.0))
    y, hT, cT = R.lstm_forward(_layers(w), w.bias, w.x)
    assert np.all(y == 0) and np.all(hT == 0) and np.all(cT == 0)
    # LSTM, W = 0, bias only: c_t = s_f * c_{t-1} + s_i * tanh(b_g) is a geometric series.
    w = _zero_weight(_small("lstm", L=1, T=7, bias_std=0.7, state_std=0.0))
    H = w.hidden_size
    b = w.bias[0].astype(np.float64)
    s = lambda a: 1.0 / (1.0 + np.exp(-a))
    si, sf, tg, so = s(b[:H]), s(b[H:2 * H]), np.tanh(b[2 * H:3 * H]), s(b[3 * H:])
    y, hT, cT = R.lstm_forward(_layers(w), w.bias, w.x)
    c_closed = si * tg * (1 - sf ** 7) / (1 - sf)
    np.testing.assert_allclose(cT[0], np.broadcast_to(c_closed, cT[0].shape), rtol=1e-12)
    np.testing.assert_allclose(hT[0], np.broadcast_to(so * np.tanh(c_closed), hT[0].shape), rtol=1e-12)
    # GRU, W = 0, b = 0: r = z = 1/2, n = 0, so h_t = h_0 / 2^t exactly.
    w = _zero_weight(_small("gru", L=1, T=6, bias_std=0.0, state_std=1.0))
    y, hT = R.gru_forward(_layers(w), w.bias, w.x, w.h0)
    assert np.array_equal(hT[0], w.h0[0].astype(np.float64) / 64.0)
    assert np.array_equal(y[2], w.h0[0].astype(np.float64) / 8.0)


@pytest.mark.parametrize("cell", ["lstm", "gru"])
def test_resume_batch_independence_and_stacking(cell):
    w = _small(cell, L=2, B=3, T=6)
    lay = _layers(w)
    if cell == "lstm":
        y, hT, cT = R.lstm_forward(lay, w.bias, w.x, w.h0, w.c0)
        y1, h1, c1 = R.lstm_forward(lay, w.bias, w.x[:2], w.h0, w.c0)
        y2, h2, c2 = R.lstm_forward(lay, w.bias, w.x[2:], h1, c1)
        assert np.array_equal(c2, cT)
        yb, hb, _ = R.lstm_forward(lay, w.bias, w.x[:, 1:2], w.h0[:, 1:2], w.c0[:, 1:2])
        ya, _, _ = R.lstm_forward(lay[:1], w.bias[:1], w.x, w.h0[:1], w.c0[:1])
        yc, hc, _ = R.lstm_forward(lay[1:], w.bias[1:], ya, w.h0[1:], w.c0[1:])
    else:
        y, hT = R.gru_forward(lay, w.bias, w.x, w.h0)
        y1, h1 = R.gru_forward(lay, w.bias, w.x[:2], w.h0)
        y2, h2 = R.gru_forward(lay, w.bias, w.x[2:], h1)
        yb, hb = R.gru_forward(lay, w.bias, w.x[:, 1:2], w.h0[:, 1:2])
        ya, _ = R.gru_forward(lay[:1], w.bias[:1], w.x, w.h0[:1])
        yc, hc = R.gru_forward(lay[1:], w.bias[1:], ya, w.h0[1:])
    assert np.array_equal(np.concatenate([y1, y2]), y) and np.array_equal(h2, hT)
    np.testing.assert_allclose(yb[:, 0], y[:, 1], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(hb[:, 0], hT[:, 1], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(yc, y, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(hc[0], hT[1], rtol=1e-13, atol=1e-15)


def test_gate_order_and_sign_sensitivity():
    # A mistake in gate order or in the (1 - z) / z roles must not survive the torch pin:
    # make sure the pin is sensitive, by planting the mistake on the oracle's side.
    w = _small("gru", L=1, T=3)
    y, _ = R.gru_forward(_layers(w), w.bias, w.x, w.h0)
    m = w.layers[0]
    H = w.hidden_size
    swapped = m.dense.copy()
    swapped[:H], swapped[H:2 * H] = m.dense[H:2 * H], m.dense[:H]
    lay = [(swapped, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)]
    y_bad, _ = R.gru_forward(lay, w.bias, w.x, w.h0)
    assert np.max(np.abs(y - y_bad)) > 1e-3
    assert np.allclose(R.sigmoid(np.array([-800.0, 0.0, 800.0])), [0.0, 0.5, 1.0])
