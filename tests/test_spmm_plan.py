"""The planned layout of the tensor-core batched product, decoded on the CPU with the kernel's
addressing rules: every stored weight must come back exactly once, at its place in the masked
matrix, in the stream of the warp that owns its block-row and block-column."""
import numpy as np
import pytest

import workloads
from oracle import csb_oracle as O
from paper_2005_05758_b200 import binding

STAGE = 2304


def decode(plan, rows, cols, br, bc):
    """Walks every weight stream like the kernel does; returns the matrix and a use count."""
    RG = plan["RG"]
    W = np.zeros((rows, cols), np.float64)
    seen = np.zeros((rows, cols), np.int32)
    stream, table, begin = plan["stream"], plan["chunk_table"], plan["stream_begin"]
    for c, (group, split, tile0, ntiles) in enumerate(plan["cta"]):
        assert ntiles >= 1
        rows_of_warps = plan["warp_row"][c].astype(int)
        assert np.all(np.diff(rows_of_warps) >= 0) and rows_of_warps[0] == 0 and rows_of_warps[-1] < RG
        for wp in range(plan["warps"]):
            rr, sidx = rows_of_warps[wp], c * plan["warps"] + wp
            last_tile = -1
            for ch in range(begin[sidx], begin[sidx + 1]):
                off, nbytes = int(table[ch][0]) * 16, int(table[ch][1])
                assert nbytes <= STAGE and nbytes % 16 == 0
                p = off + 16
                end = p + 16 * int(stream[off:off + 4].view(np.uint32)[0])
                assert end == off + nbytes
                while p < end:
                    tile = int(stream[p:p + 2].view(np.uint16)[0])
                    nk, np2 = int(stream[p + 2]), int(stream[p + 3])
                    mask = int(stream[p + 4:p + 12].view(np.uint64)[0])
                    size = 16 * int(stream[p + 12:p + 14].view(np.uint16)[0])
                    assert 0 <= tile < ntiles and tile >= last_tile and 1 <= nk <= 64 and np2 == (nk + 1) // 2
                    last_tile = tile
                    cidx = stream[p + 16:p + 16 + nk].astype(int)
                    vals = stream[p + 16 + ((nk + 3) & ~3):p + size].view(np.float16)
                    kept_rows = [r for r in range(64) if (mask >> r) & 1]
                    need = len(kept_rows) * np2 * 4 + 16 + ((nk + 3) & ~3)
                    assert need <= size < need + 16
                    G = plan["tile_blocks"]
                    assert np.all(cidx // bc == cidx[0] // bc) and cidx[0] // bc < G   # one block per item
                    bi, bj = group * RG + rr, tile0 + tile * G + int(cidx[0]) // bc
                    for i, r in enumerate(kept_rows):
                        for k in range(nk):
                            R, Cc = bi * br + r, bj * bc + int(cidx[k]) % bc
                            W[R, Cc] = float(vals[i * np2 * 2 + k])
                            seen[R, Cc] += 1
                        if nk % 2:
                            assert vals[i * np2 * 2 + nk] == 0          # the padding half of an odd row
                    p += size
    return W, seen


@pytest.mark.parametrize("shape,batch,sms", [((300, 1177, 32, 32), 8, 148), ((512, 192, 16, 16), 32, 148), ((1024, 1536, 64, 64), 64, 148),
                                              ((1024, 768, 64, 64), 16, 20), ((96, 4096, 32, 128), 33, 148), ((200, 130, 64, 8), 8, 7)])
def test_every_weight_once_in_the_right_stream(shape, batch, sms):
    R, C, br, bc = shape
    w = workloads.make_spmv_workload(R + C, R, C, br, bc, "lognormal", rate=5.0, batch=1, w_std=0.05)
    m = w.matrix
    A = binding.csb_encode(m.dense, br, bc, m.row_keep, m.col_keep, "f16", -1)
    plan = binding.csb_spmm_plan_dump(A, batch, sms)
    A.free()
    assert plan["RG"] in (1, 2, 4) and plan["NT"] == (1 if batch <= 8 else 2 if batch <= 16 else 4)
    assert plan["warps"] == (32 if batch <= 8 else 16)
    nbr, nbc = -(-R // br), -(-C // bc)
    groups = -(-nbr // plan["RG"])
    assert plan["ctas"] == groups * plan["S"]
    # the ranges of a row group tile its block-columns without gaps, in order
    for g in range(groups):
        mine = [c for c in plan["cta"] if c[0] == g]
        assert [c[1] for c in mine] == list(range(plan["S"]))
        assert mine[0][2] == 0 and all(mine[i][2] < mine[i + 1][2] <= mine[i][2] + mine[i][3] * plan["tile_blocks"] for i in range(len(mine) - 1))
        assert mine[-1][2] + mine[-1][3] * plan["tile_blocks"] >= nbc
    W, seen = decode(plan, nbr * br, nbc * bc, br, bc)
    want = O.masked_dense(m.dense, br, bc, m.row_keep, m.col_keep, "f16")
    mask = O.block_mask(R, C, br, bc, m.row_keep, m.col_keep)
    assert np.array_equal(seen[:R, :C], mask.astype(np.int32)) and not seen[R:].any() and not seen[:, C:].any()
    assert np.array_equal(W[:R, :C], want)


def test_uneven_blocks_give_even_work():
    # lognormal block sizes (one block has up to ten times the work of another): the column ranges
    # of a row group and the deal of a row's items to its warps must even that out
    w = workloads.CONFIGS["cfg4"](rate=8.0, B=1, n=4096)
    m = w.matrix
    A = binding.csb_encode(m.dense, 64, 64, m.row_keep, m.col_keep, "f16", -1)
    plan = binding.csb_spmm_plan_dump(A, 32, 148)
    A.free()
    assert plan["S"] > 1 and plan["balance"] > 0.8 and plan["warp_balance"] > 0.5, (plan["balance"], plan["warp_balance"])


def test_fp32_values_are_refused():
    W = np.ones((8, 8), np.float32)
    A = binding.csb_encode(W, 4, 4, np.ones(16, np.uint8), np.ones(16, np.uint8), "f32", -1)
    with pytest.raises(binding.CsbError) as e:
        binding.csb_spmm_plan_dump(A, 8, 148)
    assert e.value.status == -8
    A.free()
