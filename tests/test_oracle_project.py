"""Pins for the projection oracle (Algorithm 1's RowPrune / ColumnPrune), CPU only: a hand-worked
example, counts, the ordering property, ties, limits, invariances and a scalar brute force."""
import json
import os

import numpy as np
import pytest

from oracle import csb_oracle as O
from oracle import project_oracle as P

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_hand_worked_4x4():
    with open(os.path.join(GOLDEN, "project_4x4.json")) as f:
        g = json.load(f)
    rk, ck, Z = P.project(np.array(g["W"], np.float32), g["block_r"], g["block_c"], g["PR"])
    assert rk.tolist() == g["row_keep"] and ck.tolist() == g["col_keep"]
    assert Z.tolist() == g["Z"]
    # the masks describe the same matrix in the encoder's terms
    assert np.array_equal(O.masked_dense(np.array(g["W"], np.float32), 2, 2, rk, ck, "f32"), np.array(g["Z"], float))


def _brute(W, BR, BC, PR):
    """Scalar loops, selection by repeated minimum: nothing shared with the oracle's sorting."""
    R, C = len(W), len(W[0])
    nbr, nbc = -(-R // BR), -(-C // BC)
    p = 1.0 - (1.0 - PR) ** 0.5
    Z = [[float(v) for v in row] for row in W]
    rk = [0] * (nbr * nbc * BR)
    ck = [0] * (nbr * nbc * BC)
    for bj in range(nbc):
        cols = range(bj * BC, min(C, (bj + 1) * BC))
        norm = [sum(Z[r][c] * Z[r][c] for c in cols) for r in range(R)]
        alive = [True] * R
        for _ in range(min(R, int(p * R + 0.5))):
            best = None
            for r in range(R):                      # strictly smaller wins, so among equals the last one is taken
                if alive[r] and (best is None or norm[r] <= norm[best]):
                    best = r
            alive[best] = False
        for r in range(R):
            if alive[r]:
                rk[((r // BR) * nbc + bj) * BR + r % BR] = 1
            else:
                for c in cols:
                    Z[r][c] = 0.0
    for bi in range(nbr):
        rows = range(bi * BR, min(R, (bi + 1) * BR))
        norm = [sum(Z[r][c] * Z[r][c] for r in rows) for c in range(C)]
        alive = [True] * C
        for _ in range(min(C, int(p * C + 0.5))):
            best = None
            for c in range(C):
                if alive[c] and (best is None or norm[c] <= norm[best]):
                    best = c
            alive[best] = False
        for c in range(C):
            if alive[c]:
                ck[(bi * nbc + c // BC) * BC + c % BC] = 1
            else:
                for r in rows:
                    Z[r][c] = 0.0
    return rk, ck, Z


@pytest.mark.parametrize("R,C,BR,BC,PR", [(6, 8, 2, 4, 0.75), (7, 9, 3, 4, 0.6), (8, 8, 4, 4, 0.9375), (5, 5, 5, 5, 0.36), (9, 4, 2, 2, 0.0)])
def test_brute_force(R, C, BR, BC, PR):
    rng = np.random.default_rng(R * 100 + C)
    W = np.round(rng.standard_normal((R, C)) * 4) / 4          # coarse values: ties do occur
    rk, ck, Z = P.project(W, BR, BC, PR)
    brk, bck, bZ = _brute(W.tolist(), BR, BC, PR)
    assert rk.tolist() == brk and ck.tolist() == bck and Z.tolist() == bZ


def test_counts_order_and_overall_rate():
    rng = np.random.default_rng(3)
    R, C, BR, BC, PR = 96, 128, 16, 32, 0.84
    W = rng.standard_normal((R, C))
    rk, ck, Z = P.project(W, BR, BC, PR)
    p = 1 - np.sqrt(1 - PR)
    nbr, nbc = R // BR, C // BC
    rk3, ck3 = rk.reshape(nbr, nbc, BR), ck.reshape(nbr, nbc, BC)
    for bj in range(nbc):                                       # RowPrune: the count, and nothing kept is weaker than anything pruned
        kept = rk3[:, bj, :].reshape(-1).astype(bool)
        assert (~kept).sum() == int(np.floor(p * R + 0.5))
        norms = (W[:, bj * BC:(bj + 1) * BC] ** 2).sum(axis=1)
        assert norms[kept].min() >= norms[~kept].max()
    after_rows = W * np.repeat(rk3.transpose(0, 2, 1).reshape(R, nbc), BC, axis=1)
    for bi in range(nbr):
        kept = ck3[bi].reshape(-1).astype(bool)
        assert (~kept).sum() == int(np.floor(p * C + 0.5))
        norms = (after_rows[bi * BR:(bi + 1) * BR] ** 2).sum(axis=0)
        assert norms[kept].min() >= norms[~kept].max()
    assert abs((Z != 0).mean() - (1 - PR)) < 0.02               # the two prunes together remove about PR
    assert np.array_equal(Z, O.masked_dense(W.astype(np.float32), BR, BC, rk, ck, "f32")) or \
        np.allclose(Z, O.masked_dense(W.astype(np.float32), BR, BC, rk, ck, "f32"), rtol=1e-7)


def test_ties_keep_the_lower_index_and_limits():
    W = np.ones((4, 4))
    rk, ck, Z = P.project(W, 2, 2, 0.75)                        # all norms equal: rows / columns 2, 3 go everywhere
    assert rk.reshape(2, 2, 2).tolist() == [[[1, 1], [1, 1]], [[0, 0], [0, 0]]]
    assert ck.reshape(2, 2, 2)[0].tolist() == [[1, 1], [0, 0]]
    rk, ck, Z = P.project(W, 2, 2, 0.0)
    assert rk.all() and ck.all() and np.array_equal(Z, W)
    rk, ck, Z = P.project(W, 2, 2, 1.0)
    assert not rk.any() and not ck.any() and not Z.any()


def test_scale_invariance_and_block_column_independence():
    rng = np.random.default_rng(5)
    W = rng.standard_normal((12, 12))
    a = P.project(W, 4, 4, 0.7)
    b = P.project(3.0 * W, 4, 4, 0.7)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    W2 = W.copy()
    W2[:, 8:] *= 100.0                                          # RowPrune of block-columns 0 and 1 must not notice
    c = P.project(W2, 4, 4, 0.7)
    assert np.array_equal(a[0].reshape(3, 3, 4)[:, :2], c[0].reshape(3, 3, 4)[:, :2])
