"""CPU oracle for the recurrent cells driven by a CSB-pruned weight.

TEST INFRASTRUCTURE ONLY: shares no code with the CUDA library and must not be
reached from any product path.  Arithmetic is float64 throughout.

The paper's Figure 1 (the cell equations) is not legible in the available
text; Section 2.1 names the primitives (matrix-vector products, sigmoid, tanh,
element-wise product and sum, the c/h context link) and cites Hochreiter &
Schmidhuber 1997 and Cho et al. 2014.  Reading taken here:
  * LSTM without peepholes, stacked weight rows ordered i, f, g, o;
  * GRU with stacked rows r, z, n and the reset gate applied AFTER the recurrent
    product, so that a step is ONE product with [x_t ; h_{t-1}] followed by an
    element-wise epilogue (the other variant needs two dependent products);
  * bias is dense and untouched by pruning (Section 3.2); a GRU carries the
    candidate gate's input bias and hidden bias separately.
These are the conventions of torch.nn.LSTM / torch.nn.GRU, which the tests use
as an independent pin, next to closed forms for zero weights.

Pins (tests/test_oracle_rnn.py): torch.nn.LSTM / GRU in float64 loaded with the
masked dense weight; W = 0 closed forms (LSTM state stays 0 without bias, is a
geometric series with bias; GRU halves h each step); resume and batch-column
independence; a stack equals its layers run one after another.
The cell variants of Table 1 (LSTMP, Li-GRU) and the reset-before GRU follow at the end
of the file with their own pins.  Fixed-point arithmetic is not implemented here.
"""
from __future__ import annotations

import numpy as np

from . import csb_oracle


def sigmoid(a):
    """1 / (1 + exp(-a)) evaluated without overflow for large |a|."""
    a = np.asarray(a, dtype=np.float64)
    e = np.exp(-np.abs(a))
    return np.where(a >= 0, 1.0 / (1.0 + e), e / (1.0 + e))


def _masked(layer):
    """layer = (W, BR, BC, row_keep, col_keep, val_dtype) -> float64 masked dense."""
    W, BR, BC, rk, ck, vd = layer
    return csb_oracle.masked_dense(W, BR, BC, rk, ck, vd)


def lstm_forward(layers, bias, x, h0=None, c0=None):
    """Stacked LSTM over a sequence (Section 2.1).

    layers[l] describes W_l of shape [4H, I_l + H]; bias[l] is [4H] or None;
    x is [T, B, I_0]; h0, c0 are [L, B, H] or None (zeros).
    Per layer and step:  z = W_l . [u_t ; h_{t-1}] + b, split into i, f, g, o;
      c_t = sigmoid(f) * c_{t-1} + sigmoid(i) * tanh(g);  h_t = sigmoid(o) * tanh(c_t)
    where u_t is x_t for layer 0 and the h_t of the layer below otherwise.
    Returns y [T, B, H] (top layer's h_t), hT [L, B, H], cT [L, B, H].
    """
    x = np.asarray(x, dtype=np.float64)
    T, B, _ = x.shape
    L = len(layers)
    Wm = [_masked(l) for l in layers]
    H = Wm[0].shape[0] // 4
    h = np.zeros((L, B, H)) if h0 is None else np.array(h0, dtype=np.float64)
    c = np.zeros((L, B, H)) if c0 is None else np.array(c0, dtype=np.float64)
    y = np.zeros((T, B, H))
    for t in range(T):
        u = x[t]
        for l in range(L):
            v = np.concatenate([u, h[l]], axis=1)            # [B, I_l + H]
            z = v @ Wm[l].T
            if bias[l] is not None:
                z = z + np.asarray(bias[l], dtype=np.float64)[None, :]
            i, f, g, o = z[:, 0:H], z[:, H:2 * H], z[:, 2 * H:3 * H], z[:, 3 * H:4 * H]
            c[l] = sigmoid(f) * c[l] + sigmoid(i) * np.tanh(g)
            h[l] = sigmoid(o) * np.tanh(c[l])
            u = h[l]
        y[t] = u
    return y, h, c


def gru_forward(layers, bias, x, h0=None):
    """Stacked GRU, reset applied after the recurrent product.

    layers[l]: W_l of shape [3H, I_l + H], rows r, z, n; bias[l] is [4H] holding
    b_r, b_z, b_in, b_hn (b_r and b_z are the sums of the input and hidden
    biases, which only ever appear added) or None.
      zx = W_l[:, :I_l] . u_t          zh = W_l[:, I_l:] . h_{t-1}
      r = sigmoid(zx_r + zh_r + b_r)   z = sigmoid(zx_z + zh_z + b_z)
      n = tanh(zx_n + b_in + r * (zh_n + b_hn))
      h_t = (1 - z) * n + z * h_{t-1}
    Returns y [T, B, H], hT [L, B, H].
    """
    x = np.asarray(x, dtype=np.float64)
    T, B, _ = x.shape
    L = len(layers)
    Wm = [_masked(l) for l in layers]
    H = Wm[0].shape[0] // 3
    h = np.zeros((L, B, H)) if h0 is None else np.array(h0, dtype=np.float64)
    y = np.zeros((T, B, H))
    for t in range(T):
        u = x[t]
        for l in range(L):
            I_l = u.shape[1]
            zx = u @ Wm[l][:, :I_l].T
            zh = h[l] @ Wm[l][:, I_l:].T
            b = np.zeros(4 * H) if bias[l] is None else np.asarray(bias[l], dtype=np.float64)
            r = sigmoid(zx[:, 0:H] + zh[:, 0:H] + b[0:H])
            z = sigmoid(zx[:, H:2 * H] + zh[:, H:2 * H] + b[H:2 * H])
            n = np.tanh(zx[:, 2 * H:] + b[2 * H:3 * H] + r * (zh[:, 2 * H:] + b[3 * H:]))
            h[l] = (1.0 - z) * n + z * h[l]
            u = h[l]
        y[t] = u
    return y, h


# ---------------------------------------------------------------------------------------
# Cell variants of the paper's Table 1 (LSTMP, Li-GRU) and the reset-before GRU of the
# reference Section 2.1 cites.  The table names the cells and gives their layer sizes
# only; the equations are taken from the cited papers and restated here.  What the table
# fixes: SR1's LSTMP layers (input 153 -> hidden 1024, then input 512 -> hidden 1024,
# 3.25 M and 4.72 M weights, 4 K bias) are consistent with a projection to 512 units and
# no peephole weights: 4 * 1024 * (153 + 512) + 512 * 1024 = 3.25 M.  SR3's Li-GRU layers
# (39 -> 512: 564.2 K weights) are consistent with two gate matrices: 2 * 512 * (39 + 512).
#
# Pins (tests/test_oracle_rnn_variants.py): LSTMP against torch.nn.LSTM(proj_size=...) in
# float64; Li-GRU against a scalar hand loop and a closed form for zero weights; the
# reset-before GRU against a scalar hand loop, against torch.nn.GRU in the special case
# where the two variants coincide (no recurrent weights in the candidate rows), and a
# closed form for zero weights.
# ---------------------------------------------------------------------------------------
def lstmp_forward(layers, proj, bias, x, h0=None, c0=None):
    """Stacked LSTM with a recurrent projection (LSTMP; Table 1, models SR1).

    layers[l]: W_l [4H, I_l + P] (rows i, f, g, o; the last P columns multiply the
    projected state), proj[l]: W_p [P, H], both CSB-pruned; bias[l]: [4H] or None.
      z = W_l . [u_t ; r_{t-1}] + b;   c_t = sigmoid(f) c_{t-1} + sigmoid(i) tanh(g)
      m_t = sigmoid(o) tanh(c_t);      r_t = W_p . m_t          (no bias, no activation)
    The layer's output and recurrent state is r_t (P units); I_l = P above the first layer.
    x [T, B, I_0]; h0 [L, B, P]; c0 [L, B, H].  Returns y [T, B, P], hT [L, B, P], cT [L, B, H].
    """
    x = np.asarray(x, dtype=np.float64)
    T, B, _ = x.shape
    L = len(layers)
    Wm = [_masked(l) for l in layers]
    Wp = [_masked(p) for p in proj]
    H = Wm[0].shape[0] // 4
    P = Wp[0].shape[0]
    r = np.zeros((L, B, P)) if h0 is None else np.array(h0, dtype=np.float64)
    c = np.zeros((L, B, H)) if c0 is None else np.array(c0, dtype=np.float64)
    y = np.zeros((T, B, P))
    for t in range(T):
        u = x[t]
        for l in range(L):
            z = np.concatenate([u, r[l]], axis=1) @ Wm[l].T
            if bias[l] is not None:
                z = z + np.asarray(bias[l], dtype=np.float64)[None, :]
            i, f, g, o = z[:, 0:H], z[:, H:2 * H], z[:, 2 * H:3 * H], z[:, 3 * H:4 * H]
            c[l] = sigmoid(f) * c[l] + sigmoid(i) * np.tanh(g)
            m = sigmoid(o) * np.tanh(c[l])
            r[l] = m @ Wp[l].T
            u = r[l]
        y[t] = u
    return y, r, c


def ligru_forward(layers, bias, x, h0=None):
    """Stacked light GRU (Li-GRU; Table 1, model SR3): no reset gate, rectified candidate.

    layers[l]: W_l [2H, I_l + H], rows z (update gate) then c (candidate); bias[l]: [2H]
    or None.  The batch normalisation the cell applies to its feed-forward products is, at
    inference, a fixed per-unit scale and shift: the scale belongs to the weight rows, the
    shift is the bias here.
      a = W_l . [u_t ; h_{t-1}] + b;   z = sigmoid(a_z);   cand = max(a_c, 0)
      h_t = z h_{t-1} + (1 - z) cand
    Returns y [T, B, H], hT [L, B, H].
    """
    x = np.asarray(x, dtype=np.float64)
    T, B, _ = x.shape
    L = len(layers)
    Wm = [_masked(l) for l in layers]
    H = Wm[0].shape[0] // 2
    h = np.zeros((L, B, H)) if h0 is None else np.array(h0, dtype=np.float64)
    y = np.zeros((T, B, H))
    for t in range(T):
        u = x[t]
        for l in range(L):
            a = np.concatenate([u, h[l]], axis=1) @ Wm[l].T
            if bias[l] is not None:
                a = a + np.asarray(bias[l], dtype=np.float64)[None, :]
            z = sigmoid(a[:, 0:H])
            cand = np.maximum(a[:, H:2 * H], 0.0)
            h[l] = z * h[l] + (1.0 - z) * cand
            u = h[l]
        y[t] = u
    return y, h


def gru_reset_before_forward(layers, bias, x, h0=None):
    """Stacked GRU with the reset gate applied BEFORE the recurrent product of the candidate
    (the form of the GRU reference Section 2.1 cites): two dependent products per step.

    layers[l]: W_l [3H, I_l + H], rows r, z, n; bias[l]: [3H] (b_r, b_z, b_n) or None.
      [a_r ; a_z] = W_l[0:2H] . [u_t ; h_{t-1}] + [b_r ; b_z];  r = sigmoid(a_r);  z = sigmoid(a_z)
      n = tanh(W_l[2H:3H] . [u_t ; r * h_{t-1}] + b_n)
      h_t = (1 - z) n + z h_{t-1}
    Returns y [T, B, H], hT [L, B, H].
    """
    x = np.asarray(x, dtype=np.float64)
    T, B, _ = x.shape
    L = len(layers)
    Wm = [_masked(l) for l in layers]
    H = Wm[0].shape[0] // 3
    h = np.zeros((L, B, H)) if h0 is None else np.array(h0, dtype=np.float64)
    y = np.zeros((T, B, H))
    for t in range(T):
        u = x[t]
        for l in range(L):
            b = np.zeros(3 * H) if bias[l] is None else np.asarray(bias[l], dtype=np.float64)
            a = np.concatenate([u, h[l]], axis=1) @ Wm[l][0:2 * H].T + b[None, 0:2 * H]
            r, z = sigmoid(a[:, 0:H]), sigmoid(a[:, H:2 * H])
            n = np.tanh(np.concatenate([u, r * h[l]], axis=1) @ Wm[l][2 * H:3 * H].T + b[None, 2 * H:3 * H])
            h[l] = (1.0 - z) * n + z * h[l]
            u = h[l]
        y[t] = u
    return y, h
