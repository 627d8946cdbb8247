"""Pins for the fixed-point oracle (CPU only)."""
import json
import os

import numpy as np
import pytest

import workloads
from oracle import csb_oracle as O
from oracle import fixed_oracle as F

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_rounding_and_saturation_by_hand():
    # f = 0: halves go to the even integer; f = 2: steps of a quarter; the range is that of int16
    assert F.quantize([0.5, 1.5, 2.5, -0.5, -1.5, 2.4999, -2.5001], 0).tolist() == [0, 2, 2, 0, -2, 2, -3]
    assert F.quantize([0.125, 0.375, 0.3, -0.3], 2).tolist() == [0, 2, 1, -1]
    assert F.quantize([40000.0, -40000.0, 32767.4, -32768.6, np.inf, -np.inf, np.nan], 0).tolist() == [32767, -32768, 32767, -32768, 32767, -32768, 0]
    assert F.quantize([1.0, -1.0], 15).tolist() == [32767, -32768]          # 1.0 does not fit Q0.15, -1.0 does
    assert F.dequantize([3, -5], 2).tolist() == [0.75, -1.25]


def test_hand_example_with_integer_weights():
    with open(os.path.join(GOLDEN, "hand_4x6.json")) as f:
        g = json.load(f)
    W = np.array([[10 * r + c + 1 for c in range(6)] for r in range(4)], dtype=np.float32)
    acc = F.spmm_q16(W, 2, 3, g["row_keep"], g["col_keep"], 0, np.array([g["x"], g["x_signed"]]))
    assert acc.tolist() == [g["y"], g["y_signed"]]
    # one fraction bit on each side: every factor doubles, the accumulators are four times as large
    acc2 = F.spmm_q16(W, 2, 3, g["row_keep"], g["col_keep"], 1, 2 * np.array([g["x"]]))
    assert acc2.tolist() == [[4 * v for v in g["y"]]]
    assert F.encode_values(W, 2, 3, g["row_keep"], g["col_keep"], 0).tolist() == g["val"]


def test_brute_force_python_integers():
    rng = np.random.default_rng(5)
    R, C, BR, BC = 6, 8, 2, 4
    W = rng.standard_normal((R, C)).astype(np.float32)
    rk = rng.integers(0, 2, 3 * 2 * BR)
    ck = rng.integers(0, 2, 3 * 2 * BC)
    Xq = rng.integers(-32768, 32768, (2, C))
    fw = 13
    got = F.spmm_q16(W, BR, BC, rk, ck, fw, Xq)
    nbc = C // BC
    for beta in range(2):
        for r in range(R):
            acc = 0
            for c in range(C):
                b = (r // BR) * nbc + c // BC
                if rk[b * BR + r % BR] and ck[b * BC + c % BC]:
                    q = int(np.clip(np.rint(float(W[r, c]) * 2 ** fw), -32768, 32767))
                    acc += q * int(Xq[beta, c])
            assert int(got[beta, r]) == acc


def test_distance_to_the_float_product_is_inside_the_quantisation_bound():
    w = workloads.make_spmv_workload(7, 256, 320, 32, 32, "lognormal", rate=6.0, batch=3, w_std=0.05)
    m = w.matrix
    fw, fx = 17, 12                                   # |w| < 0.25 fits 17 fraction bits; |x| < 8 fits 12
    assert np.abs(m.dense).max() < 0.25 and np.abs(w.X).max() < 8
    Xq = F.quantize(w.X, fx)
    acc = F.spmm_q16(m.dense, 32, 32, m.row_keep, m.col_keep, fw, Xq)
    y = F.dequantize(acc, fw + fx)
    Wm = O.masked_dense(m.dense, 32, 32, m.row_keep, m.col_keep, "f32")
    want = w.X.astype(np.float64) @ Wm.T
    # |w_q x_q - w x| <= |w| e_x + |x| e_w + e_w e_x with e = half a unit in the last place
    ew, ex = 2.0 ** -(fw + 1), 2.0 ** -(fx + 1)
    bound = np.abs(w.X).astype(np.float64) @ (np.abs(Wm) > 0).T * ew + ex * np.abs(Wm).sum(axis=1)[None, :] + ew * ex * (Wm != 0).sum(axis=1)[None, :]
    assert np.all(np.abs(y - want) <= bound + 1e-15)
    assert np.max(np.abs(y - want)) > 0               # and the quantisation is really there


def test_rows_kept_nowhere_and_linearity_in_integers():
    w = workloads.make_spmv_workload(8, 64, 64, 16, 16, "uniform", lo=0.0, hi=0.6, batch=2, w_std=0.1)
    m = w.matrix
    Xq = F.quantize(w.X, 10)
    acc = F.spmm_q16(m.dense, 16, 16, m.row_keep, m.col_keep, 14, Xq)
    kept = m.row_keep.reshape(4, 4, 16).any(axis=1).reshape(-1)
    assert np.all(acc[:, ~kept] == 0)
    both = F.spmm_q16(m.dense, 16, 16, m.row_keep, m.col_keep, 14, Xq[0:1] // 2 + Xq[1:2] // 2)
    assert np.array_equal(both[0], F.spmm_q16(m.dense, 16, 16, m.row_keep, m.col_keep, 14, Xq[0:1] // 2)[0]
                          + F.spmm_q16(m.dense, 16, 16, m.row_keep, m.col_keep, 14, Xq[1:2] // 2)[0])
