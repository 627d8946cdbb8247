"""The cycle model of the paper's PEGroup schedule (Sections 4.3 and 5.2): closed cases and the
ordering of the sharing modes."""
import numpy as np

import workloads
from paper_2005_05758_b200 import pegroup_model as M


def test_equal_blocks_that_fill_the_pe_array_are_fully_efficient():
    m = np.full((8, 8), 8)
    n = np.full((8, 8), 12)
    for mode in M.MODES:
        assert M.efficiency(m, n, mode=mode) == 1.0


def test_one_heavy_block_by_hand():
    # 2 x 2 PEGroups of 4 x 4 PEs, one iteration: block (0, 0) is 16 x 16 (16 passes), the others are empty.
    m = np.array([[16, 0], [0, 0]])
    n = np.array([[16, 0], [0, 0]])
    kw = dict(K=2, L=2, P=4, Q=4)
    assert M.efficiency(m, n, mode="none", **kw) == 256 / (64 * 16)              # one group works, three wait
    # horizontal sharing: 8 of the 16 columns go to the right neighbour: 8 passes each
    assert M.efficiency(m, n, mode="horizontal", **kw) == 256 / (64 * 8)
    # two dimensions: the right neighbour takes 8 columns (8 passes), the lower one takes 4 of the 8 passes left
    assert M.efficiency(m, n, mode="2d", **kw) >= 256 / (64 * 8)
    assert M.efficiency(m, n, mode="2d", **kw) <= 1.0


def test_sharing_never_hurts_and_orders_as_in_the_paper():
    w = workloads.make_spmv_workload(3, 1024, 1024, 32, 32, "lognormal", rate=10.0, batch=1, w_std=0.05)
    m, n = M.block_counts(w.matrix)
    e = {mode: M.efficiency(m, n, mode=mode) for mode in M.MODES}
    assert e["none"] <= e["horizontal"] <= e["2d"] + 1e-12 and e["none"] <= e["vertical"] <= e["2d"] + 1e-12
    # the shape of the paper's Figure 12: uneven blocks idle most PEs, sharing in one dimension wins some back, in two more
    assert e["none"] < 0.5 and e["2d"] > 1.5 * e["none"] and max(e["horizontal"], e["vertical"]) < e["2d"] <= 1.0


def test_block_counts_clip_the_edges():
    mat = workloads.MatrixSpec(np.ones((5, 7), np.float32), 4, 4, np.ones(2 * 2 * 4, np.uint8), np.ones(2 * 2 * 4, np.uint8), "f16")
    m, n = M.block_counts(mat)
    assert m.tolist() == [[4, 4], [1, 1]] and n.tolist() == [[4, 3], [4, 3]]
