"""CPU oracle for the 16-bit fixed-point CSB product.

TEST INFRASTRUCTURE ONLY: shares no code with the CUDA library and must not be reached from any
product path.  Integer arithmetic throughout (numpy int64; Python integers in the brute force).

The paper quantises its CSB-pruned models to 16-bit fixed point for the comparison with prior work
(Section 6.2.2) and its processing elements multiply 16-bit fixed-point numbers (Section 6.3.1).  It
does not say how the binary point is placed, how values are rounded or how wide the accumulators
are.  Reading taken here:
  * a value v with f fraction bits is stored as the integer q = clamp(rint(v * 2^f), -32768, 32767),
    rint rounding halves to the even integer; f is chosen by the caller per weight matrix and per
    input vector (a power-of-two scale, as a fixed-point datapath has); NaN is stored as 0;
  * the product accumulates the exact integer sum of w_q * x_q over the kept cross-points (an
    accumulator wide enough never to overflow: 64 bits here; every 16 x 16-bit product fits 31
    bits), so the result does not depend on the order of summation;
  * the real value of an output is acc * 2^-(f_w + f_x).
Pins (tests/test_oracle_fixed.py): the rounding and saturation rules on hand-picked values, the
hand-written 4 x 6 example (integer weights, f = 0), Python-integer brute force on small matrices,
and the distance to the float64 product, which must stay inside the bound that follows from half a
unit in the last place of every factor.
"""
from __future__ import annotations

import numpy as np

from . import csb_oracle

Q_MIN, Q_MAX = -32768, 32767


def quantize(v, frac_bits):
    """Real values -> 16-bit fixed-point integers with `frac_bits` fraction bits (int64 array)."""
    v = np.asarray(v, dtype=np.float64)
    q = np.rint(np.where(np.isnan(v), 0.0, v) * (2.0 ** frac_bits))
    return np.clip(q, Q_MIN, Q_MAX).astype(np.int64)


def dequantize(q, frac_bits):
    return np.asarray(q, dtype=np.float64) * (2.0 ** -frac_bits)


def masked_quantized(W, BR, BC, row_keep, col_keep, frac_bits):
    """The integer matrix a fixed-point CSB encoding stands for: quantised weights at the kept
    cross-points, zeros elsewhere."""
    W = np.asarray(W, dtype=np.float32)
    mask = csb_oracle.block_mask(W.shape[0], W.shape[1], BR, BC, row_keep, col_keep)
    return np.where(mask, quantize(W, frac_bits), 0)


def spmm_q16(W, BR, BC, row_keep, col_keep, w_frac_bits, Xq):
    """Exact integer accumulators acc[beta, r] = sum_c Wq[r, c] * Xq[beta, c] (int64); Xq holds
    16-bit fixed-point integers.  The real result is acc * 2^-(w_frac_bits + x_frac_bits)."""
    Wq = masked_quantized(W, BR, BC, row_keep, col_keep, w_frac_bits)
    Xq = np.asarray(Xq, dtype=np.int64)
    if Xq.size and (Xq.min() < Q_MIN or Xq.max() > Q_MAX):
        raise ValueError("inputs are not 16-bit")
    return Xq @ Wq.T


def encode_values(W, BR, BC, row_keep, col_keep, frac_bits):
    """Val{} of the fixed-point encoding: the quantised kernel matrices in the order of
    csb_oracle.encode (everything else of the format is the same)."""
    enc = csb_oracle.encode(W, BR, BC, row_keep, col_keep, "f32")
    return quantize(enc["val"], frac_bits).astype(np.int16)
