"""Host-side encoder of the library against the oracle's plain-loop encoder: bit-exact
arrays (indices, counts, offsets, values).  Runs without a GPU (device = -1)."""
import json
import os

import numpy as np
import pytest

import workloads
from oracle import csb_oracle as O
import paper_2005_05758_b200 as csb
from paper_2005_05758_b200 import binding

KEYS = ("m", "n", "row_idx", "col_idx", "val_off", "ridx_off", "cidx_off")


def _compare(dense, br, bc, rk, ck, vd):
    A = binding.csb_encode(dense, br, bc, rk, ck, vd, device=-1)
    got = A.view()
    want = O.encode(dense, br, bc, rk, ck, vd)
    for k in KEYS:
        assert got[k].dtype == want[k].dtype, k
        assert np.array_equal(got[k], want[k]), k
    # values: compare bit patterns, so that -0.0, inf and NaN payload classes count too
    bits = np.uint16 if vd == "f16" else np.uint32
    assert np.array_equal(got["val"].view(bits), want["val"].view(bits))
    info = A.info()
    assert info["nnz"] == len(want["val"])
    if info["nnz"]:
        assert info["nio"] == pytest.approx(O.nio(want), rel=1e-12)
        assert info["pruning_rate"] == pytest.approx(O.pruning_rate(want), rel=1e-12)
    A.free()
    return got


def test_hand_example():
    with open(os.path.join(os.path.dirname(__file__), "golden", "hand_4x6.json")) as f:
        g = json.load(f)
    W = np.array([[10 * r + c + 1 for c in range(6)] for r in range(4)], dtype=np.float32)
    got = _compare(W, 2, 3, np.array(g["row_keep"], np.uint8), np.array(g["col_keep"], np.uint8), "f32")
    for k in KEYS + ("val",):
        assert got[k].tolist() == g[k], k


@pytest.mark.parametrize("vd", ["f16", "f32"])
@pytest.mark.parametrize("shape", [(4, 4, 2, 2), (50, 39, 16, 8), (96, 70, 32, 32), (33, 300, 7, 256), (5, 7, 4, 4)])
def test_random_masks_bit_exact(shape, vd):
    R, Cc, br, bc = shape
    rng = np.random.default_rng(R * 1000 + Cc)
    W = (rng.standard_normal((R, Cc)) * 0.1).astype(np.float32)
    nblk = -(-R // br) * -(-Cc // bc)
    rk = (rng.random(nblk * br) < 0.5).astype(np.uint8)
    ck = (rng.random(nblk * bc) < 0.4).astype(np.uint8) * 7       # any non-zero byte keeps
    _compare(W, br, bc, rk, ck, vd)


def test_special_values_round_like_ieee():
    vals = np.array([0.0, -0.0, 1.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 65504.0, 65519.99, 65520.0, 1e9, -1e9,
                     2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0001, 6.1e-5, 5.9e-8, np.inf, -np.inf, np.nan, 1e-30,
                     -3.14159, 0.333333, 1234.567, 2.0 ** -14, 2.0 ** -14 * 0.9999], dtype=np.float32)
    W = np.resize(vals, (8, 8)).astype(np.float32)
    ones = np.ones(8, np.uint8)
    for vd in ("f16", "f32"):
        _compare(W, 8, 8, ones, ones, vd)
    # every finite binary16 value survives, and the midpoints between neighbours tie to even
    h = np.arange(0, 0x7c00, dtype=np.uint16).view(np.float16).astype(np.float32)
    mid = (h[:-1].astype(np.float64) + h[1:].astype(np.float64)) / 2
    W2 = np.concatenate([h, mid.astype(np.float32), np.zeros(1, np.float32)]).reshape(248, 256)
    _compare(W2, 248, 256, np.ones(248, np.uint8), np.ones(256, np.uint8), "f16")


def test_empty_and_degenerate_blocks():
    rng = np.random.default_rng(5)
    W = rng.standard_normal((8, 8)).astype(np.float32)
    rk = np.zeros(4 * 4, np.uint8)
    ck = np.ones(4 * 4, np.uint8)
    rk[4:8] = 1                       # block 1 keeps all rows; others keep none
    ck[4:8] = 0                       # ... but block 1 keeps no column
    got = _compare(W, 4, 4, rk, ck, "f16")
    assert got["nnz"] == 0 and got["m"].tolist() == [0, 4, 0, 0] and got["n"].tolist() == [4, 0, 4, 4]


@pytest.mark.parametrize("cfg", ["cfg1", "cfg2"])
def test_config_shapes(cfg):
    w = workloads.CONFIGS[cfg](T=1)
    m = w.layers[0]
    if cfg == "cfg2":                 # the oracle's loops are slow: a ragged corner of the matrix
        full = m
        nbc = 37
        sub_rk = full.row_keep.reshape(128, nbc, 32)[:6, 30:].reshape(-1).copy()
        sub_ck = full.col_keep.reshape(128, nbc, 32)[:6, 30:].reshape(-1).copy()
        m = workloads.MatrixSpec(full.dense[:192, 960:].copy(), 32, 32, sub_rk, sub_ck, "f16")
        assert m.cols == 217          # 6 full block-columns and one 25 wide
    _compare(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)


def test_argument_errors():
    W = np.zeros((4, 4), np.float32)
    k = np.ones(4, np.uint8)
    with pytest.raises(binding.CsbError) as e:
        binding.csb_encode(W, 0, 4, k, k, "f16", device=-1)
    assert e.value.status == -1
    with pytest.raises(binding.CsbError) as e:
        binding.csb_encode(W, 4, 257, k, np.ones(257, np.uint8), "f16", device=-1)
    assert e.value.status == -1
    with pytest.raises(binding.CsbError) as e:
        binding.csb_encode(W, 4, 4, k, k, 9, device=-1)
    assert e.value.status == -3 and "val_dtype" in str(e.value)
    A = binding.csb_encode(W, 4, 4, k, k, "f16", device=-1)
    import ctypes
    assert binding.lib.csb_spmv(A.handle, None, None, None) == -1
    buf = np.zeros(4, np.float32)
    assert binding.lib.csb_spmv(A.handle, buf.ctypes.data, buf.ctypes.data, None) == -8   # host-only handle
    assert binding.lib.csb_encode(None, 4, 4, 4, 4, 4, None, None, 1, -1, None, ctypes.byref(ctypes.c_void_p())) == -1
    assert binding.lib.csb_strerror(-7) == b"bounded device-side wait expired"
