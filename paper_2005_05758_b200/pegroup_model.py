"""Cycle model of the paper's CSB-Engine schedule, to set its utilisation beside this library's balance.

The paper's engine (Section 4.3) is K x L PEGroups of P x Q processing elements.  The block grid
is walked in "block iterations" of K x L blocks, one block per PEGroup (Algorithm 2); a PEGroup
needs ceil(m / P) * ceil(n / Q) passes for an m x n kernel matrix, and an iteration lasts as long
as its slowest PEGroup.  Workload sharing (Sections 4.3.2 and 5.2) lets a PEGroup hand a
rectangular part of its kernel matrix to its right neighbour (horizontal) and to its lower
neighbour (vertical, at most half of the rows) on a torus; the parts are whole multiples of P rows
/ Q columns and the three parts tile the kernel matrix in one of two ways (the constraints CLP 1-6
of Section 5.2.2).  The paper searches the part sizes with an SMT solver, widening the allowed
excess over the average load by P * Q per round; here a greedy descent on the sum of squared loads
stands in for the solver, so the figures are a lower bound of what the paper's compiler reaches.

Efficiency = useful multiply-accumulates / (PEs x cycles), the quantity of the paper's Figure 12
(42 % without sharing, 72 % with sharing in one dimension, 94 % in two, averaged over its ten
trained models on 4 x 4 PEGroups of 4 x 4 PEs).  This is context for the planner's balance
figures, not a target and not part of the product path.

    python -m paper_2005_05758_b200.pegroup_model          # table for the synthetic workloads
"""
from __future__ import annotations

import numpy as np

MODES = ("none", "horizontal", "vertical", "2d")


def _passes(m, n, P, Q):
    return -(-m // P) * -(-n // Q) if m > 0 and n > 0 else 0


class _Iteration:
    """One block iteration: K x L kernel matrices and the parts they hand on."""

    def __init__(self, m, n, P, Q):
        self.m, self.n, self.P, self.Q = m, n, P, Q
        self.K, self.L = m.shape
        self.dnh = np.zeros_like(m)    # columns handed to the right neighbour (all local rows, or the rows left after dmv)
        self.dmv = np.zeros_like(m)    # rows handed to the lower neighbour
        self.form = np.zeros_like(m)   # 0: the horizontal part spans all rows (CLP 3); 1: the vertical part spans all columns (CLP 4)

    def parts(self, k, l):
        """(local, horizontal, vertical) part sizes of block (k, l) as (rows, cols) pairs."""
        m, n, dnh, dmv = int(self.m[k, l]), int(self.n[k, l]), int(self.dnh[k, l]), int(self.dmv[k, l])
        local = (m - dmv, n - dnh)
        if self.form[k, l] == 0:
            return local, (m, dnh), (dmv, n - dnh)
        return local, (m - dmv, dnh), (dmv, n)

    def load(self, k, l):
        """Passes PEGroup (k, l) spends: its local part, what its left neighbour handed right, what its upper neighbour handed down."""
        P, Q = self.P, self.Q
        loc, _, _ = self.parts(k, l)
        _, h_in, _ = self.parts(k, (l - 1) % self.L)
        _, _, v_in = self.parts((k - 1) % self.K, l)
        t = _passes(loc[0], loc[1], P, Q)
        if self.L > 1:
            t += _passes(h_in[0], h_in[1], P, Q)
        if self.K > 1:
            t += _passes(v_in[0], v_in[1], P, Q)
        return t

    def loads(self):
        return np.array([[self.load(k, l) for l in range(self.L)] for k in range(self.K)])

    def balance(self, mode):
        """Greedy descent on the sum of squared loads: any PEGroup may hand one more slab of Q columns
        to the right or P rows down (or take one back, or switch between the two tilings) as long as
        that lowers the sum; work then diffuses over the torus until no single step helps."""
        if mode == "none":
            return
        allow_h = mode in ("horizontal", "2d") and self.L > 1
        allow_v = mode in ("vertical", "2d") and self.K > 1
        for _ in range(2000):
            improved = False
            for k in range(self.K):
                for l in range(self.L):
                    m, n = int(self.m[k, l]), int(self.n[k, l])
                    if not m or not n:
                        continue
                    saved = (int(self.dnh[k, l]), int(self.dmv[k, l]), int(self.form[k, l]))
                    touched = {(k, l), (k, (l + 1) % self.L), ((k + 1) % self.K, l)}
                    before = sum(self.load(a, b) ** 2 for a, b in touched)
                    moves = []
                    for f in (0, 1):
                        if allow_h:
                            moves += [(saved[0] + d, saved[1], f) for d in (self.Q, -self.Q) if 0 <= saved[0] + d <= n]
                        if allow_v:
                            moves += [(saved[0], saved[1] + d, f) for d in (self.P, -self.P) if 0 <= saved[1] + d <= m // 2]
                        if f != saved[2]:
                            moves.append((saved[0], saved[1], f))
                    best = None
                    for mv in moves:
                        self.dnh[k, l], self.dmv[k, l], self.form[k, l] = mv
                        after = sum(self.load(a, b) ** 2 for a, b in touched)
                        if after < before and (best is None or after < best[0]):
                            best = (after, mv)
                    if best is None:
                        self.dnh[k, l], self.dmv[k, l], self.form[k, l] = saved
                    else:
                        self.dnh[k, l], self.dmv[k, l], self.form[k, l] = best[1]
                        improved = True
            if not improved:
                return


def efficiency(m_blocks, n_blocks, K=4, L=4, P=4, Q=4, mode="2d"):
    """PE utilisation of one CSB matrix on K x L PEGroups of P x Q PEs.

    m_blocks, n_blocks: [nbr, nbc] kept rows / kept columns per block.  Returns useful
    multiply-accumulates / (K * L * P * Q * cycles)."""
    if mode not in MODES:
        raise ValueError(mode)
    m_blocks, n_blocks = np.asarray(m_blocks, np.int64), np.asarray(n_blocks, np.int64)
    nbr, nbc = m_blocks.shape
    cycles = 0
    for i in range(0, nbr, K):
        for j in range(0, nbc, L):
            m = np.zeros((K, L), np.int64)
            n = np.zeros((K, L), np.int64)
            bm, bn = m_blocks[i:i + K, j:j + L], n_blocks[i:i + K, j:j + L]
            m[:bm.shape[0], :bm.shape[1]] = bm
            n[:bn.shape[0], :bn.shape[1]] = bn
            it = _Iteration(m, n, P, Q)
            it.balance(mode)
            cycles += int(it.loads().max())
    work = int((m_blocks * n_blocks).sum())
    return work / (K * L * P * Q * cycles) if cycles else 1.0


def block_counts(mat):
    """Kept rows / kept columns per block of a workloads.MatrixSpec, as [nbr, nbc] arrays (edge blocks clipped)."""
    R, C, br, bc = mat.rows, mat.cols, mat.block_r, mat.block_c
    nbr, nbc = -(-R // br), -(-C // bc)
    rk = np.asarray(mat.row_keep).reshape(nbr, nbc, br) != 0
    ck = np.asarray(mat.col_keep).reshape(nbr, nbc, bc) != 0
    rvalid = (np.arange(nbr)[:, None] * br + np.arange(br)[None, :]) < R
    cvalid = (np.arange(nbc)[:, None] * bc + np.arange(bc)[None, :]) < C
    return (rk & rvalid[:, None, :]).sum(axis=2), (ck & cvalid[None, :, :]).sum(axis=2)


def table(cases=None, sample_block_rows=64):
    """Efficiency of the model in its four sharing modes on the synthetic workloads (the first
    `sample_block_rows` block-rows of each matrix, to keep the greedy search short)."""
    import workloads
    cases = cases or [("cfg2 LSTM 4096x1177, 32x32, ~8x", workloads.CONFIGS["cfg2"](T=1).layers[0]),
                      ("cfg3 GRU 3072x1536, 32x32, 16x lognormal", workloads.CONFIGS["cfg3"](T=1).layers[0]),
                      ("cfg4 8192x8192, 64x64, 4x lognormal", workloads.CONFIGS["cfg4"](rate=4.0).matrix),
                      ("cfg4 8192x8192, 64x64, 25x lognormal", workloads.CONFIGS["cfg4"](rate=25.0).matrix),
                      ("cfg4 4x, diagonal blocks 4x denser", workloads.CONFIGS["cfg4"](rate=4.0, diag_boost=4.0, n=4096).matrix),
                      ("cfg5 LSTM layer 8192x4096, 64x64, ~10x uniform", workloads.CONFIGS["cfg5"](T=1).layers[0])]
    rows = []
    for name, mat in cases:
        m, n = block_counts(mat)
        m, n = m[:sample_block_rows], n[:sample_block_rows]
        rows.append((name,) + tuple(efficiency(m, n, mode=mode) for mode in MODES))
    return rows


if __name__ == "__main__":
    print("%-52s %8s %10s %8s %6s" % (("workload (4x4 PEGroups of 4x4 PEs)",) + MODES))
    for r in table():
        print("%-52s %8.3f %10.3f %8.3f %6.3f" % r)
