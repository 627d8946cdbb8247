"""Host logic without a GPU: the planned device stream of the bare product is decoded in Python,
with the addressing rules the kernel uses, and must (a) reproduce the masked dense matrix exactly,
every stored weight exactly once, and (b) respect every alignment and size rule the kernel and its
bulk copies rely on, for both schedules (row-owned and partial-sum) and all lane-group widths."""
import os

import numpy as np
import pytest

import workloads
from oracle import csb_oracle as O
from paper_2005_05758_b200 import binding


def decode(plan, rows, cols, block_r, val_dtype, stage_bytes):
    """Walk the stream like the kernel does and scatter every value back to (row, column)."""
    gw = plan["group_width"]
    G = 32 // gw
    rpw = 2 if val_dtype == "f16" else 1
    vt = np.float16 if val_dtype == "f16" else np.float32
    s = plan["stream"]
    dense = np.zeros((rows, cols), np.float64)
    count = np.zeros((rows, cols), np.int32)
    flushes = {}                                            # block-row base -> list of (warp, kind, slot)
    pieces = {}                                             # block-row base -> {bit 2 of the tail} for CTA flushes
    for w in range(plan["warps"]):
        for c in range(plan["warp_begin"][w], plan["warp_begin"][w + 1]):
            off16, nbytes = (int(v) for v in plan["chunk_table"][c])
            kind, off = off16 >> 30, (off16 & 0x3FFFFFFF) * 16
            assert nbytes % 16 == 0 and 16 <= nbytes <= stage_bytes, "chunk must fit one ring stage"
            hdr = s[off:off + 16]
            sub16 = hdr[:8].view(np.uint16)
            zbase, tail = (int(v) for v in hdr[8:16].view(np.uint32))
            assert (tail & 3) == kind, "flush kind in the chunk table and in the chunk agree"
            assert 16 + 16 * int(sub16.sum()) == nbytes and not sub16[G:].any()
            if kind:
                flushes.setdefault(zbase, []).append((w, kind, tail >> 3))
                if kind == 3:
                    pieces.setdefault(zbase, set()).add((tail >> 2) & 1)
            p = off + 16
            for g in range(G):
                end = p + 16 * int(sub16[g])
                while p < end:
                    assert p % 16 == 0
                    nk, mr, RL, S = (int(v) for v in s[p:p + 4])
                    xbase = int(s[p + 4:p + 8].view(np.uint32)[0])
                    izb, magic, size16 = (int(v) for v in s[p + 8:p + 14].view(np.uint16))
                    voff = 16 * int(s[p + 15])
                    assert 1 <= nk <= 64 and 1 <= mr <= gw * rpw and RL == -(-mr // rpw) and S == gw // RL and izb == 0
                    assert magic == -(-1024 // RL) and all((l * magic) >> 10 == l // RL for l in range(32))
                    nwords = nk * RL
                    cidx = s[p + 16:p + 16 + nk].astype(int)
                    ro = p + 16 + ((nk + 3) & ~3)
                    ridx = s[ro:ro + mr].astype(int)
                    assert voff == (16 + ((nk + 3) & ~3) + ((mr + 3) & ~3) + 15) & ~15, "values start on a 16-byte boundary behind the indices"
                    assert 16 * size16 == (voff + 4 * nwords + 15) & ~15
                    words = s[p + voff:p + voff + 4 * nwords].view(vt).reshape(nwords, rpw).astype(np.float64)
                    nq = nk // 4
                    for k in range(nk):
                        for wd in range(RL):
                            # quad-columns are interleaved [q][w][4], the tail columns follow as [k][w]
                            wi = ((k // 4) * RL + wd) * 4 + k % 4 if k < nq * 4 else nq * RL * 4 + (k - nq * 4) * RL + wd
                            for q in range(rpw):
                                r = wd * rpw + q
                                if r < mr:
                                    dense[zbase + ridx[r], xbase + cidx[k]] = words[wi, q]
                                    count[zbase + ridx[r], xbase + cidx[k]] += 1
                                else:
                                    assert words[wi, q] == 0.0, "padding rows are zero"
                    p += 16 * size16
                assert p == end
    return dense, count, flushes, pieces


CASES = [
    # rows, cols, br, bc, law, kw, dtype, ctas, warps, stage
    (256, 320, 32, 32, "lognormal", dict(rate=6.0), "f16", 4, 4, 2048),           # few block-rows: partial sums
    (1024, 512, 64, 64, "uniform", dict(lo=0.3, hi=0.7), "f16", 8, 16, 4096),      # 16 block-rows on 8 CTAs: row-owned
    (300, 1177, 32, 32, "uniform", dict(lo=0.25, hi=0.45), "f16", 148, 16, 4096),  # ragged edge, more CTAs than work
    (512, 192, 16, 16, "exact", dict(count=8), "f32", 6, 8, 3072),
    (96, 640, 32, 128, "lognormal", dict(rate=3.0), "f32", 3, 2, 4096),            # wide blocks: column slices
    (640, 256, 64, 64, "exact", dict(count=64), "f16", 10, 4, 4096),               # all kept: row slices of 64-row blocks
    (1024, 4096, 64, 64, "lognormal", dict(rate=8.0), "f16", 20, 8, 4096),         # one block-row keeps everything: it is divided
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("gw", [0, 8, 16, 32])
def test_stream_decodes_to_the_masked_matrix(case, gw):
    rows, cols, br, bc, law, kw, vd, ctas, warps, stage = case
    w = workloads.make_spmv_workload(3, rows, cols, br, bc, law, batch=1, w_std=0.1, val_dtype=vd, **kw)
    m = w.matrix
    if ctas == 20:                                      # a block-row far heavier than the rest
        nbr, nbc = -(-rows // br), -(-cols // bc)
        m.row_keep.reshape(nbr, nbc, br)[0] = 1
        m.col_keep.reshape(nbr, nbc, bc)[0] = 1
    A = binding.csb_encode(m.dense, br, bc, m.row_keep, m.col_keep, vd, device=-1)
    os.environ.pop("CSB_GROUP_WIDTH", None)
    if gw:
        os.environ["CSB_GROUP_WIDTH"] = str(gw)
    try:
        plan = binding.csb_plan_dump(A, ctas, warps, stage)
    finally:
        os.environ.pop("CSB_GROUP_WIDTH", None)
    assert plan["group_width"] in (8, 16, 32) and (not gw or plan["group_width"] == gw)
    dense, count, flushes, piece_bits = decode(plan, rows, cols, br, vd, stage)
    want = O.masked_dense(m.dense, br, bc, m.row_keep, m.col_keep, vd)
    mask = O.block_mask(rows, cols, br, bc, m.row_keep, m.col_keep)
    assert np.array_equal(count, mask.astype(np.int32)), "every stored weight exactly once, nothing else"
    assert np.array_equal(dense, want)
    # every block-row leaves its warps exactly as planned
    nbr = -(-rows // br)
    assert sorted(flushes) == [bi * br for bi in range(nbr)], "every block-row is flushed, empty ones too"
    for zb, fl in flushes.items():
        if zb not in piece_bits:
            piece_bits[zb] = set()
        kinds = {k for _, k, _ in fl}
        assert len(kinds) == 1
        kind = kinds.pop()
        if kind == 1:                                   # one warp owns the block-row
            assert len(fl) == 1 and not plan["row_owned"]
        elif kind == 2:                                 # partial sums: consecutive slots, one per warp
            slots = sorted(sl for _, _, sl in fl)
            assert len(fl) > 1 and slots == list(range(slots[0], slots[0] + len(fl))) and slots[-1] < plan["slots"]
        else:                                           # CTA runs: whole CTAs report; several CTAs = several pieces
            assert plan["row_owned"]
            wpc = plan["warps_per_cta"]
            ws = sorted(wi for wi, _, _ in fl)
            assert len(ws) % wpc == 0 and len(set(ws)) == len(ws)
            n_pieces = len(ws) // wpc
            by_cta = {}
            for wi, _, sl in fl:
                by_cta.setdefault(wi // wpc, []).append(sl)
            assert len(by_cta) == n_pieces and all(len(v) == wpc and len(set(v)) == 1 for v in by_cta.values())
            tails = sorted(v[0] for v in by_cta.values())
            if n_pieces == 1:
                assert piece_bits[zb] == {0}
            else:                                       # one slot per piece, consecutive, all marked as pieces
                assert piece_bits[zb] == {1} and tails == list(range(tails[0], tails[0] + n_pieces))
                assert tails[-1] < plan["slots"]
    if ctas == 20:
        assert plan["row_owned"] and plan["slots"] >= 2, "this case must exercise divided block-rows"
    A.free()


def test_empty_block_rows_and_buffer_errors():
    rng = np.random.default_rng(1)
    W = rng.standard_normal((128, 64)).astype(np.float32)
    rk = np.ones(4 * 32, np.uint8)
    rk[32:64] = 0                                       # block-row 1 keeps nothing
    A = binding.csb_encode(W, 32, 64, rk, np.ones(4 * 64, np.uint8), "f16", device=-1)
    plan = binding.csb_plan_dump(A, 2, 2, 4096)
    dense, count, flushes, _ = decode(plan, 128, 64, 32, "f16", 4096)
    assert not dense[32:64].any() and 32 in flushes
    info = np.zeros(8, np.int64)
    small = np.zeros(16, np.uint8)
    rc = binding.lib.csb_plan_dump(A.handle, 2, 2, 4096, info.ctypes.data, small.ctypes.data, small.size, None, 0, None, 0)
    assert rc == -1 and b"too small" in binding.lib.csb_last_error()
    assert binding.lib.csb_plan_dump(A.handle, 0, 2, 4096, info.ctypes.data, None, 0, None, 0, None, 0) == -1
    A.free()
