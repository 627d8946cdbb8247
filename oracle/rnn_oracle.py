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
The reset-before GRU variant and fixed-point arithmetic are not implemented:
parity unpinned for those (nothing here computes them).
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
