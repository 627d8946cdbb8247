"""Pins for the cell variants of the recurrent oracle (CPU only): LSTMP against an independent
library cell, Li-GRU and the reset-before GRU against scalar hand loops written from the cited
definitions, closed forms for zero weights, and the special case in which the two GRU variants
coincide."""
import math

import numpy as np
import pytest
import torch

import workloads
from oracle import csb_oracle as O
from oracle import rnn_oracle as R


def _tup(m):
    return (m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)


def _masked(m):
    return O.masked_dense(*_tup(m))


def _small(cell, L=2, B=3, T=5, I=20, H=24, seed=13, vd="f16", bias_std=0.2, state_std=0.5, **kw):
    return workloads.make_rnn_workload(seed, cell, I, H, L, 8, 8, "uniform", lo=0.3, hi=0.8, T=T, B=B, w_std=0.3,
                                       val_dtype=vd, bias_std=bias_std, state_std=state_std, **kw)


@pytest.mark.parametrize("vd", ["f16", "f32"])
def test_lstmp_matches_torch_proj_size_float64(vd):
    w = _small("lstmp", vd=vd, proj_size=16)
    H, P, I, L = w.hidden_size, w.proj_size, w.input_size, len(w.layers)
    y, hT, cT = R.lstmp_forward([_tup(m) for m in w.layers], [_tup(m) for m in w.proj], w.bias, w.x, w.h0, w.c0)
    net = torch.nn.LSTM(I, H, num_layers=L, proj_size=P).double()
    with torch.no_grad():
        for l in range(L):
            Wm, Wp = torch.from_numpy(_masked(w.layers[l])), torch.from_numpy(_masked(w.proj[l]))
            in_l = I if l == 0 else P
            getattr(net, "weight_ih_l%d" % l).copy_(Wm[:, :in_l])
            getattr(net, "weight_hh_l%d" % l).copy_(Wm[:, in_l:])
            getattr(net, "weight_hr_l%d" % l).copy_(Wp)
            getattr(net, "bias_ih_l%d" % l).copy_(torch.from_numpy(w.bias[l].astype(np.float64)))
            getattr(net, "bias_hh_l%d" % l).zero_()
        ty, (th, tc) = net(torch.from_numpy(w.x).double(), (torch.from_numpy(w.h0).double(), torch.from_numpy(w.c0).double()))
    assert y.shape == (w.T, w.B, P) and hT.shape == (L, w.B, P) and cT.shape == (L, w.B, H)
    np.testing.assert_allclose(y, ty.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(hT, th.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(cT, tc.numpy(), rtol=1e-12, atol=1e-13)


def test_lstmp_with_identity_projection_is_the_lstm():
    # P = H and W_p = I: the projected state is h itself
    w = _small("lstm", L=1, I=16, H=16)
    m = w.layers[0]
    eye = workloads.MatrixSpec(np.eye(16, dtype=np.float32), 8, 8, np.ones(4 * 8, np.uint8), np.ones(4 * 8, np.uint8), "f32")
    y0, h0, c0 = R.lstm_forward([_tup(m)], w.bias, w.x, w.h0, w.c0)
    y1, h1, c1 = R.lstmp_forward([_tup(m)], [_tup(eye)], w.bias, w.x, w.h0, w.c0)
    np.testing.assert_allclose(y1, y0, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(c1, c0, rtol=1e-14, atol=1e-15)


def _sig(a):
    return 1.0 / (1.0 + math.exp(-a))


def _hand_ligru(W, b, xs, h, I, H):
    """Scalar loops, one batch column: z = s(W_z.[x;h] + b_z), c = relu(W_c.[x;h] + b_c), h = z h + (1 - z) c."""
    out = []
    for x in xs:
        v = list(x) + list(h)
        a = [sum(W[r][k] * v[k] for k in range(I + H)) + b[r] for r in range(2 * H)]
        h = [_sig(a[j]) * h[j] + (1.0 - _sig(a[j])) * max(a[H + j], 0.0) for j in range(H)]
        out.append(h)
    return out


def test_ligru_matches_scalar_hand_loop():
    w = _small("ligru", L=1, B=2, T=4, I=5, H=8, bias_std=0.5)
    y, hT = R.ligru_forward([_tup(w.layers[0])], w.bias, w.x, w.h0)
    Wm = _masked(w.layers[0]).tolist()
    for b in range(w.B):
        want = _hand_ligru(Wm, w.bias[0].astype(np.float64).tolist(), w.x[:, b].astype(np.float64).tolist(),
                           w.h0[0, b].astype(np.float64).tolist(), 5, 8)
        np.testing.assert_allclose(y[:, b], np.array(want), rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(hT[0], y[-1], rtol=0, atol=0)
    assert (y[:, :, :] >= np.minimum(0.0, w.h0[0].min())).all()      # a convex mix of h and a rectified value


def test_ligru_zero_weight_closed_form():
    # W = 0: z = s(b_z) and cand = relu(b_c) are constants, so h_t = z^t h_0 + (1 - z^t) relu(b_c)
    w = _small("ligru", L=1, B=2, T=6, I=4, H=8, bias_std=1.0)
    w.layers[0].dense[:] = 0
    y, hT = R.ligru_forward([_tup(w.layers[0])], w.bias, w.x, w.h0)
    b = w.bias[0].astype(np.float64)
    z, cand = 1.0 / (1.0 + np.exp(-b[:8])), np.maximum(b[8:], 0.0)
    assert (b[8:] < 0).any() and (b[8:] > 0).any()                   # both sides of the rectifier are exercised
    for t in range(6):
        np.testing.assert_allclose(y[t], z ** (t + 1) * w.h0[0] + (1 - z ** (t + 1)) * cand, rtol=1e-12, atol=1e-13)


def _hand_gru_rb(W, b, xs, h, I, H):
    out = []
    for x in xs:
        v = list(x) + list(h)
        a = [sum(W[r][k] * v[k] for k in range(I + H)) + b[r] for r in range(2 * H)]
        r, z = [_sig(a[j]) for j in range(H)], [_sig(a[H + j]) for j in range(H)]
        v2 = list(x) + [r[j] * h[j] for j in range(H)]
        n = [math.tanh(sum(W[2 * H + j][k] * v2[k] for k in range(I + H)) + b[2 * H + j]) for j in range(H)]
        h = [(1.0 - z[j]) * n[j] + z[j] * h[j] for j in range(H)]
        out.append(h)
    return out


def test_gru_reset_before_matches_scalar_hand_loop():
    w = _small("gru_rb", L=1, B=2, T=4, I=5, H=8, bias_std=0.5)
    y, hT = R.gru_reset_before_forward([_tup(w.layers[0])], w.bias, w.x, w.h0)
    Wm = _masked(w.layers[0]).tolist()
    for b in range(w.B):
        want = _hand_gru_rb(Wm, w.bias[0].astype(np.float64).tolist(), w.x[:, b].astype(np.float64).tolist(),
                            w.h0[0, b].astype(np.float64).tolist(), 5, 8)
        np.testing.assert_allclose(y[:, b], np.array(want), rtol=1e-13, atol=1e-14)
    # the reset gate really sits in front of the product: the reset-after cell gives something else
    y2, _ = R.gru_forward([_tup(w.layers[0])], [np.concatenate([w.bias[0], np.zeros(8, np.float32)])], w.x, w.h0)
    assert np.max(np.abs(y2 - y)) > 1e-3


def test_gru_variants_coincide_without_recurrent_candidate_weights():
    # with no recurrent weights in the candidate rows it does not matter where the reset gate sits:
    # both oracle cells and torch.nn.GRU (reset-after) agree
    w = _small("gru_rb", L=2, B=3, T=5, I=12, H=16)
    for l, m in enumerate(w.layers):
        in_l = 12 if l == 0 else 16
        m.dense[2 * 16:, in_l:] = 0
    lay = [_tup(m) for m in w.layers]
    y, hT = R.gru_reset_before_forward(lay, w.bias, w.x, w.h0)
    b4 = [np.concatenate([b, np.zeros(16, np.float32)]) for b in w.bias]
    y2, hT2 = R.gru_forward(lay, b4, w.x, w.h0)
    np.testing.assert_allclose(y, y2, rtol=1e-13, atol=1e-14)
    net = torch.nn.GRU(12, 16, num_layers=2).double()
    with torch.no_grad():
        for l, m in enumerate(w.layers):
            Wm = torch.from_numpy(_masked(m))
            in_l = 12 if l == 0 else 16
            getattr(net, "weight_ih_l%d" % l).copy_(Wm[:, :in_l])
            getattr(net, "weight_hh_l%d" % l).copy_(Wm[:, in_l:])
            getattr(net, "bias_ih_l%d" % l).copy_(torch.from_numpy(w.bias[l].astype(np.float64)))
            getattr(net, "bias_hh_l%d" % l).zero_()
        ty, th = net(torch.from_numpy(w.x).double(), torch.from_numpy(w.h0).double())
    np.testing.assert_allclose(y, ty.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(hT, th.numpy(), rtol=1e-12, atol=1e-13)


def test_gru_reset_before_zero_weight_closed_form():
    # W = 0, b = 0: r = z = 1/2, n = 0, h halves every step
    w = _small("gru_rb", L=1, B=2, T=5, I=4, H=8, bias_std=0.0)
    w.layers[0].dense[:] = 0
    y, hT = R.gru_reset_before_forward([_tup(w.layers[0])], w.bias, w.x, w.h0)
    for t in range(5):
        np.testing.assert_allclose(y[t], w.h0[0] * 0.5 ** (t + 1), rtol=1e-15)


@pytest.mark.parametrize("cell", ["lstmp", "ligru", "gru_rb"])
def test_resume_batch_columns_and_stacking(cell):
    kw = dict(proj_size=16) if cell == "lstmp" else {}
    w = _small(cell, L=2, B=3, T=6, **kw)
    lay = [_tup(m) for m in w.layers]
    prj = [_tup(m) for m in w.proj] if cell == "lstmp" else None

    def run(layers, proj, bias, x, h0, c0):
        if cell == "lstmp":
            return R.lstmp_forward(layers, proj, bias, x, h0, c0)
        if cell == "ligru":
            return R.ligru_forward(layers, bias, x, h0) + (None,)
        return R.gru_reset_before_forward(layers, bias, x, h0) + (None,)

    y, hT, cT = run(lay, prj, w.bias, w.x, w.h0, w.c0)
    # resume
    ya, ha, ca = run(lay, prj, w.bias, w.x[:2], w.h0, w.c0)
    yb, hb, cb = run(lay, prj, w.bias, w.x[2:], ha, ca)
    np.testing.assert_allclose(np.concatenate([ya, yb]), y, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(hb, hT, rtol=1e-13, atol=1e-14)
    # batch columns are independent
    y1, _, _ = run(lay, prj, w.bias, w.x[:, 1:2], w.h0[:, 1:2], None if w.c0 is None else w.c0[:, 1:2])
    np.testing.assert_allclose(y1[:, 0], y[:, 1], rtol=1e-13, atol=1e-14)
    # a stack is its layers run one after the other
    y_l0, _, _ = run(lay[:1], prj[:1] if prj else None, w.bias[:1], w.x, w.h0[:1], None if w.c0 is None else w.c0[:1])
    y_l1, _, _ = run(lay[1:], prj[1:] if prj else None, w.bias[1:], y_l0, w.h0[1:], None if w.c0 is None else w.c0[1:])
    np.testing.assert_allclose(y_l1, y, rtol=1e-13, atol=1e-14)
