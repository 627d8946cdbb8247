"""Pins for the CSB oracle: format, mask and product (CPU only).

Each check is something the paper or the mathematics fixes independently of the
oracle's own code path: a hand-derived example, a scalar brute force, a dense
library product, closed forms and invariants.
"""
import itertools
import json
import os

import numpy as np
import pytest

import workloads
from oracle import csb_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _hand():
    with open(os.path.join(GOLDEN, "hand_4x6.json")) as f:
        g = json.load(f)
    W = np.array([[10 * r + c + 1 for c in range(6)] for r in range(4)], dtype=np.float32)
    return g, W


@pytest.mark.parametrize("vd", ["f32", "f16"])
def test_hand_example_arrays(vd):
    g, W = _hand()
    enc = O.encode(W, 2, 3, g["row_keep"], g["col_keep"], vd)
    for k in ("m", "n", "row_idx", "col_idx", "val", "val_off", "ridx_off", "cidx_off"):
        assert enc[k].tolist() == g[k], k
    assert O.nio(enc) == pytest.approx(g["nio"], rel=1e-15)
    y = O.spmm(W, 2, 3, g["row_keep"], g["col_keep"], vd, np.array([g["x"]]))[0]
    assert y.tolist() == g["y"]
    assert O.spmv_from_encoding(enc, g["x"]).tolist() == g["y"]


@pytest.mark.parametrize("vd", ["f32", "f16"])
def test_hand_example_abs_scale(vd):
    # abs_scale sets the floor of every product tolerance, so it gets its own hand-written pin:
    # an input of mixed signs (y differs from the scale), the same scale for W and -W, and the
    # brute-force sum of |w||x| over all mask settings of a small matrix below
    g, W = _hand()
    xs = np.array([g["x_signed"]], dtype=np.float32)
    for sign in (1.0, -1.0):
        args = (sign * W, 2, 3, g["row_keep"], g["col_keep"], vd)
        assert (sign * O.spmm(*args, xs)[0]).tolist() == g["y_signed"]
        assert O.abs_scale(*args, xs)[0].tolist() == g["abs_scale_signed"]
    # two batch rows keep their own scales
    both = np.array([g["x_signed"], g["x"]], dtype=np.float32)
    assert O.abs_scale(W, 2, 3, g["row_keep"], g["col_keep"], vd, both).tolist() == [g["abs_scale_signed"], g["y"]]


def test_abs_scale_brute_force_all_masks():
    rng = np.random.default_rng(11)
    W = rng.integers(-8, 9, (4, 4)).astype(np.float32)
    x = rng.integers(-8, 9, 4).astype(np.float32)
    for bits in range(256):
        rk = [(bits >> k) & 1 for k in range(8)]
        ck = [((bits * 37 + 5) >> k) & 1 for k in range(8)]
        want = _brute_spmv(np.abs(W), 2, 2, rk, ck, np.abs(x))     # scalar loops over |w| * |x|
        assert O.abs_scale(W, 2, 2, rk, ck, "f32", x[None, :])[0].tolist() == want


def _brute_spmv(W, BR, BC, rk, ck, x):
    """Scalar triple loop straight from the definition of the block pattern."""
    R, C = W.shape
    nbc = -(-C // BC)
    y = [0.0] * R
    for r in range(R):
        for c in range(C):
            b = (r // BR) * nbc + (c // BC)
            if rk[b * BR + r % BR] and ck[b * BC + c % BC]:
                y[r] += float(W[r, c]) * float(x[c])
    return y


def test_brute_force_4x4_all_masks():
    rng = np.random.default_rng(7)
    W = rng.integers(-8, 9, (4, 4)).astype(np.float32)       # small integers: sums are exact
    x = rng.integers(-8, 9, 4).astype(np.float32)
    # 2x2 blocks -> 4 blocks, 8 row bits and 8 column bits; sweep all 256 settings of
    # each side against a varying setting of the other.
    for bits in range(256):
        rk = [(bits >> k) & 1 for k in range(8)]
        ck = [((bits * 73 + 41) >> k) & 1 for k in range(8)]
        for a, b in ((rk, ck), (ck, rk)):
            want = _brute_spmv(W, 2, 2, a, b, x)
            got = O.spmm(W, 2, 2, a, b, "f32", x[None, :])[0]
            assert got.tolist() == want
            enc = O.encode(W, 2, 2, a, b, "f32")
            assert O.spmv_from_encoding(enc, x).tolist() == want
            assert np.array_equal(O.decode(enc), O.masked_dense(W, 2, 2, a, b, "f32"))


def test_brute_force_exhaustive_pairs_small():
    # every (row mask, column mask) pair of a 2x4 matrix with 2x2 blocks: 2 blocks,
    # 4 + 4 bits -> 256 pairs, all of them.
    W = np.arange(1, 9, dtype=np.float32).reshape(2, 4)
    x = np.array([1, -2, 3, -4], dtype=np.float32)
    for rb, cb in itertools.product(range(16), range(16)):
        rk = [(rb >> k) & 1 for k in range(4)]
        ck = [(cb >> k) & 1 for k in range(4)]
        assert O.spmm(W, 2, 2, rk, ck, "f32", x[None])[0].tolist() == _brute_spmv(W, 2, 2, rk, ck, x)


def test_all_kept_equals_dense_product():
    rng = np.random.default_rng(1)
    R, C, BR, BC = 50, 39, 16, 8                               # ragged on both sides
    W = rng.standard_normal((R, C)).astype(np.float32)
    X = rng.standard_normal((3, C)).astype(np.float32)
    nbr, nbc = O.grid(R, C, BR, BC)
    rk = np.ones(nbr * nbc * BR, np.uint8)
    ck = np.ones(nbr * nbc * BC, np.uint8)
    got = O.spmm(W, BR, BC, rk, ck, "f32", X)
    want = X.astype(np.float64) @ W.astype(np.float64).T
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)
    enc = O.encode(W, BR, BC, rk, ck, "f32")
    assert int(enc["val_off"][-1]) == R * C                    # edge bits beyond the matrix ignored
    assert O.pruning_rate(enc) == 1.0


def test_edge_bits_beyond_matrix_are_ignored():
    rng = np.random.default_rng(2)
    R, C, BR, BC = 5, 7, 4, 4
    W = rng.standard_normal((R, C)).astype(np.float32)
    nbr, nbc = O.grid(R, C, BR, BC)
    rk = rng.integers(0, 2, nbr * nbc * BR).astype(np.uint8)
    ck = rng.integers(0, 2, nbr * nbc * BC).astype(np.uint8)
    rk2, ck2 = rk.copy().reshape(nbr, nbc, BR), ck.copy().reshape(nbr, nbc, BC)
    rk2[1, :, 1:] ^= 1                                         # rows 5..7 do not exist
    ck2[:, 1, 3:] ^= 1                                         # column 7 does not exist
    e1 = O.encode(W, BR, BC, rk, ck, "f16")
    e2 = O.encode(W, BR, BC, rk2.reshape(-1), ck2.reshape(-1), "f16")
    for k in ("m", "n", "row_idx", "col_idx", "val", "val_off"):
        assert np.array_equal(e1[k], e2[k]), k
    assert np.array_equal(O.block_mask(R, C, BR, BC, rk, ck),
                          O.block_mask(R, C, BR, BC, rk2.reshape(-1), ck2.reshape(-1)))


@pytest.mark.parametrize("cfg,kw", [("cfg1", {}), ("cfg3", {})])
def test_encoding_invariants_on_config_shapes(cfg, kw):
    w = workloads.CONFIGS[cfg](T=1, **kw)
    m = w.layers[0]
    if cfg == "cfg3":                                          # python loops: keep the slice small
        m = workloads.MatrixSpec(m.dense[:256, :320].copy(), 32, 32,
                                 m.row_keep.reshape(96, 48, 32)[:8, :10].reshape(-1).copy(),
                                 m.col_keep.reshape(96, 48, 32)[:8, :10].reshape(-1).copy(), "f16")
    enc = O.encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)
    mm, nn = enc["m"].astype(np.int64), enc["n"].astype(np.int64)
    assert np.array_equal(enc["val_off"], np.concatenate([[0], np.cumsum(mm * nn)]).astype(np.uint64))
    assert np.array_equal(enc["ridx_off"], np.concatenate([[0], np.cumsum(mm)]))
    assert np.array_equal(enc["cidx_off"], np.concatenate([[0], np.cumsum(nn)]))
    assert len(enc["val"]) == int((mm * nn).sum())
    for b in range(len(mm)):
        r = enc["row_idx"][enc["ridx_off"][b]:enc["ridx_off"][b + 1]].astype(int)
        c = enc["col_idx"][enc["cidx_off"][b]:enc["cidx_off"][b + 1]].astype(int)
        assert np.all(np.diff(r) > 0) and np.all(np.diff(c) > 0)
        assert (len(r) == 0 or r[-1] < m.block_r) and (len(c) == 0 or c[-1] < m.block_c)
    Wm = O.masked_dense(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)
    assert np.array_equal(O.decode(enc), Wm)
    x = np.random.default_rng(3).standard_normal(m.cols)
    np.testing.assert_allclose(O.spmv_from_encoding(enc, x), Wm @ x, rtol=1e-12, atol=1e-12)
    if cfg == "cfg1":
        assert O.pruning_rate(enc) == 4.0                      # 8 of 16 rows x 8 of 16 columns
        assert O.nio(enc) == pytest.approx(16 / 64)


def test_nio_matches_paper_order_of_magnitude():
    # Section 6.2.1: index overhead is about 20 % at block size 32.  With ~10x pruning a
    # 32x32 block keeps about 10x10, and (m + n) / (m * n) = 0.2.
    rng = np.random.default_rng(0)
    R = C = 128
    W = rng.standard_normal((R, C)).astype(np.float32)
    rk, ck = workloads.draw_keep_masks(rng, R, C, 32, 32, "exact", count=10)
    enc = O.encode(W, 32, 32, rk, ck, "f16")
    assert O.nio(enc) == pytest.approx(0.2)
    assert O.pruning_rate(enc) == pytest.approx(10.24)


def test_linearity_batch_columns_and_empty_rows():
    w = workloads.make_spmv_workload(5, 96, 80, 32, 16, "lognormal", rate=6.0, batch=4, w_std=0.05)
    m = w.matrix
    args = (m.dense, 32, 16, m.row_keep, m.col_keep, "f16")
    Y = O.spmm(*args, w.X)
    for b in range(4):
        assert np.array_equal(O.spmm(*args, w.X[b:b + 1])[0], Y[b])
    a, c = 0.5, -3.0
    lin = O.spmm(*args, a * w.X[0:1].astype(np.float64) + c * w.X[1:2].astype(np.float64))[0]
    np.testing.assert_allclose(lin, a * Y[0] + c * Y[1], rtol=1e-12, atol=1e-12)
    kept_somewhere = m.row_keep.reshape(3, 5, 32).any(axis=1).reshape(-1)
    cols_any = m.col_keep.reshape(3, 5, 16).any(axis=2)
    assert np.all(Y[:, ~kept_somewhere] == 0.0)
    assert np.all(O.abs_scale(*args, w.X) >= np.abs(Y) - 1e-12)
    assert cols_any.shape == (3, 5)


def test_round_to_storage_is_ieee_binary16():
    v = np.array([1.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 65504.0, 65520.0, 1e-8, -2.0 ** -24 * 0.75],
                 dtype=np.float32)
    got = O.round_to_storage(v, "f16")
    # ties go to the even mantissa; 65520 is the first value that rounds to infinity;
    # below half the smallest subnormal (2^-25) the result is zero.
    assert got.tolist() == [1.0, 1.0, 1.0 + 2.0 ** -9, 65504.0, np.inf, 0.0, -2.0 ** -24]
    assert np.array_equal(O.round_to_storage(v, "f32"), v.astype(np.float64))


def test_c_loop_nest_matches_masked_dense():
    # the second oracle form (plain C loops over the five CSB arrays) against the definition
    from oracle.csb_loops import CsbLoops
    w = workloads.make_spmv_workload(9, 200, 333, 32, 64, "lognormal", rate=5.0, batch=1, w_std=0.05)
    m = w.matrix
    stored = O.round_to_storage(m.dense, "f16").astype(np.float32)
    L = CsbLoops(stored, 32, 64, m.row_keep, m.col_keep)
    want = O.spmm(m.dense, 32, 64, m.row_keep, m.col_keep, "f16", w.X)[0]
    for threads in (1, 3):
        np.testing.assert_allclose(L.spmv(w.X[0], threads), want, rtol=1e-12, atol=1e-13)
    assert L.nnz == int(O.block_mask(200, 333, 32, 64, m.row_keep, m.col_keep).sum())
