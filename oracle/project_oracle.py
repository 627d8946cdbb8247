"""CPU oracle for the projection of a dense weight onto the CSB pattern.

TEST INFRASTRUCTURE ONLY (see csb_oracle.py): plain, slow, float64, no code
shared with the library.

Algorithm 1 of the paper, the part between its training calls: the matrix is
partitioned into BR x BC blocks; RowPrune acts on every block-column on its own
(the squared l2-norm of every row segment, i.e. of the part of a matrix row that
lies in the block-column, decides which segments go), then ColumnPrune acts on
every block-row of the result in the same way on column segments.  Both prune the
fraction p = 1 - sqrt(1 - PR), so that about PR of the weights are gone after
the two.

Readings where the paper is silent:
  * PR is the fraction of weights removed (a "4x" pruning rate is PR = 0.75);
  * the number of segments pruned in a block-column is round-half-up(p * R)
    (p * C column segments in a block-row);
  * the weakest go first; among equal norms the segment with the HIGHER index is
    pruned first (the lower index is kept);
  * ColumnPrune looks at the matrix after RowPrune (pruned row segments count
    as zeros);
  * a short last block is a short segment (the paper zero-pads, Section 6.2.1).

Pins (tests/test_oracle_project.py): a hand-worked 4x4 example, the number of
pruned segments, "nothing kept is weaker than anything pruned", ties, PR = 0
and PR -> 1, scale invariance, a scalar brute force on small matrices.
"""
from __future__ import annotations

import numpy as np


def prune_fraction(PR):
    """Fraction of segments each of the two prunes removes (Algorithm 1)."""
    return 1.0 - np.sqrt(1.0 - float(PR))


def count_pruned(p, n):
    return min(n, int(np.floor(p * n + 0.5)))


def weakest(norms, k):
    """Indices of the k weakest entries: ascending norm, and among equal norms the
    higher index first."""
    n = len(norms)
    order = np.lexsort((-np.arange(n), np.asarray(norms, dtype=np.float64)))
    return order[:k]


def project(W, BR, BC, PR):
    """Returns (row_keep [nblk * BR] uint8, col_keep [nblk * BC] uint8, Z float64)
    in the layout csb_encode takes; Z is W with the pruned lines zeroed."""
    W = np.asarray(W, dtype=np.float64)
    R, C = W.shape
    nbr, nbc = -(-R // BR), -(-C // BC)
    p = prune_fraction(PR)
    rk = np.zeros((nbr, nbc, BR), np.uint8)
    ck = np.zeros((nbr, nbc, BC), np.uint8)
    Z = W.copy()
    # RowPrune, block-column by block-column
    for bj in range(nbc):
        c0, c1 = bj * BC, min(C, (bj + 1) * BC)
        norms = np.array([np.sum(W[r, c0:c1] ** 2) for r in range(R)])
        gone = set(weakest(norms, count_pruned(p, R)).tolist())
        for r in range(R):
            if r in gone:
                Z[r, c0:c1] = 0.0
            else:
                rk[r // BR, bj, r % BR] = 1
    # ColumnPrune on the result, block-row by block-row
    for bi in range(nbr):
        r0, r1 = bi * BR, min(R, (bi + 1) * BR)
        norms = np.array([np.sum(Z[r0:r1, c] ** 2) for c in range(C)])
        gone = set(weakest(norms, count_pruned(p, C)).tolist())
        for c in range(C):
            if c in gone:
                Z[r0:r1, c] = 0.0
            else:
                ck[bi, c // BC, c % BC] = 1
    return rk.reshape(-1), ck.reshape(-1), Z
