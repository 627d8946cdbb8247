"""Host logic without a GPU: the panel layout that the batch-1 product streams is decoded in
Python with the addressing rules of the kernel (lane -> row and column octet, remainder columns,
gather descriptors, stages) and must (a) give back the masked dense matrix, every stored weight
exactly once, (b) keep every size and alignment rule the kernel and its bulk copies rely on, and
(c) give every output row to exactly one CTA (contiguous row ranges that tile the matrix)."""
import numpy as np
import pytest

import workloads
from oracle import csb_oracle as O
from paper_2005_05758_b200 import binding

HDR = ("n_items", "n_gather", "n_xg", "n_stages", "value_bytes", "ridx_bytes", "row0", "n_rows",
       "warp_off", "items_off", "gather_off", "expect_off", "cidx_off", "ridx_off", "list_off", "n_bundles")


def decode(plan, rows, cols, block_r, warps, stage):
    dense = np.zeros((rows, cols), np.float64)
    count = np.zeros((rows, cols), np.int32)
    ranges = []
    blob = plan["panels"]
    for c, (off16, meta_bytes, value_bytes, n_rows) in enumerate(plan["cta"].astype(np.int64)):
        base = int(off16) * 16
        assert base % 128 == 0 and meta_bytes % 128 == 0 and value_bytes % 16 == 0
        assert meta_bytes <= plan["max_meta"]
        meta = blob[base:base + meta_bytes]
        vals = blob[base + meta_bytes:base + meta_bytes + value_bytes]
        h = dict(zip(HDR, (int(v) for v in meta[:64].view(np.uint32))))
        assert h["value_bytes"] == value_bytes and h["n_rows"] == n_rows <= plan["max_rows"]
        assert h["n_stages"] == -(-value_bytes // stage)
        assert h["n_xg"] % 4 == 0 and h["n_xg"] <= plan["max_xg"]
        for k in ("items_off", "gather_off", "expect_off", "cidx_off", "ridx_off", "list_off"):
            assert h[k] % 16 == 0, k
        row0 = h["row0"]
        ranges.append((row0, row0 + n_rows))
        wb = meta[h["warp_off"]:h["warp_off"] + 2 * (warps + 1)].view(np.uint16).astype(int)
        assert wb[0] == 0 and wb[-1] == h["n_bundles"] and (np.diff(wb) >= 0).all()
        wlist = meta[h["list_off"]:h["list_off"] + 2 * h["n_bundles"]].view(np.uint16).astype(int)
        items = meta[h["items_off"]:h["items_off"] + 16 * h["n_items"]]
        gath = meta[h["gather_off"]:h["gather_off"] + 8 * h["n_gather"]]
        expect = meta[h["expect_off"]:h["expect_off"] + 2 * h["n_stages"]].view(np.uint16).astype(int)
        cidx = meta[h["cidx_off"]:h["cidx_off"] + h["n_xg"]].astype(int)
        ridx = meta[h["ridx_off"]:h["ridx_off"] + h["ridx_bytes"]].astype(int)
        # what the gather leaves in shared memory: for every slot the global column it holds
        xg_col = np.full(h["n_xg"], -1)
        pos = 0
        for g in range(h["n_gather"]):
            xbase, n = (int(v) for v in gath[8 * g:8 * g + 4].view(np.uint16))
            xoff = int(gath[8 * g + 4:8 * g + 8].view(np.uint32)[0])
            assert xoff == pos and xoff % 4 == 0 and n >= 1
            xg_col[xoff:xoff + n] = xbase + cidx[xoff:xoff + n]
            pos = (xoff + n + 3) & ~3
        assert pos == h["n_xg"] and xg_col.max(initial=0) < cols
        touched = np.zeros(h["n_stages"], int)
        spans = []
        seen_desc = 0
        for w in range(warps):
            last_stage = -1
            for e in wlist[wb[w]:wb[w + 1]]:
                logg, first = e >> 14, e & 0x3FFF
                G, GW = 1 << logg, 32 >> logg
                assert first == seen_desc, "descriptors sit in the order the warps take them"
                seen_desc += G
                stages = set()
                real = 0
                for grp in range(G):
                    d = items[16 * (first + grp):16 * (first + grp) + 16]
                    off = int(d[0:4].view(np.uint32)[0]) * 16
                    xoff4, roff = int(d[4:6].view(np.uint16)[0]), int(d[8:10].view(np.uint16)[0])
                    zoff = int(d[6:8].view(np.int16)[0])
                    m, logp = int(d[10]), int(d[11])
                    n = int(d[12:14].view(np.uint16)[0])
                    stages.add(off // stage)
                    P = 1 << logp
                    assert P <= GW
                    if m == 0:                          # a missing member: no rows, no columns, same stage
                        assert n == 0 and grp > 0 and P == GW
                        continue
                    real += 1
                    assert 1 <= m <= GW and 1 <= n and P >= m and P < 2 * m
                    assert (m > 16) == (logg == 0) and (m <= 8) == (logg == 2), "items are bundled by height"
                    nbytes = m * n * 2
                    assert off + nbytes <= value_bytes
                    assert off // stage == (off + nbytes - 1) // stage, "no item straddles a stage"
                    spans.append((off, off + ((nbytes + 15) & ~15)))
                    assert (row0 + zoff) % block_r == 0, "zoff is the block-row's first row relative to the panel's"
                    rr = zoff + ridx[roff:roff + m]
                    assert (np.diff(rr) > 0).all() and rr.min() >= 0 and rr.max() < n_rows
                    cc = xg_col[4 * xoff4:4 * xoff4 + n]
                    assert (cc >= 0).all() and (np.diff(cc) > 0).all(), "kept columns of a block are ascending"
                    v = vals[off:off + nbytes].view(np.float16).astype(np.float64)
                    noct = n >> 3
                    # what the lanes of the group read: lane (sub, r) takes octets sub, sub + S, ... of row r
                    S = GW // P
                    got = np.zeros((m, n))
                    for gl in range(GW):
                        r, sub = gl & (P - 1), gl >> logp
                        if r >= m:
                            continue
                        for o in range(sub, noct, S):
                            q = (o * m + r) * 8
                            got[r, 8 * o:8 * o + 8] = v[q:q + 8]
                    tb, k = noct * m * 8, noct * 8
                    for wdt in (4, 2, 1):
                        if n & wdt:
                            for r in range(m):
                                got[r, k:k + wdt] = v[tb + r * wdt:tb + r * wdt + wdt]
                            tb += m * wdt
                            k += wdt
                    for r in range(m):
                        dense[row0 + rr[r], cc] = got[r]
                        count[row0 + rr[r], cc] += 1
                assert real >= 1 and len(stages) == 1, "a bundle sits in one stage"
                st = stages.pop()
                assert st >= last_stage, "a warp takes its bundles in stream order"
                last_stage = st
                touched[st] += 1
        assert seen_desc == h["n_items"]
        assert np.array_equal(touched, expect), "per-stage bundle counts are what the refill protocol waits for"
        spans.sort()
        pos = 0
        for a, b in spans:                                # items tile the value stream; gaps only up to a stage's end
            assert a == pos or (a > pos and a % stage == 0 and a - pos < stage)
            pos = b
        assert pos == value_bytes
    return dense, count, ranges


CASES = [
    # rows, cols, br, bc, law, kw, ctas, warps, stage
    (256, 320, 32, 32, "lognormal", dict(rate=6.0), 4, 4, 8192),
    (1024, 512, 64, 64, "uniform", dict(lo=0.3, hi=0.7), 8, 16, 16384),
    (300, 1177, 32, 32, "uniform", dict(lo=0.25, hi=0.45), 148, 16, 16384),   # ragged edge, more CTAs than work
    (640, 256, 64, 64, "exact", dict(count=64), 10, 4, 8192),                 # all kept: two items per block
    (1024, 4096, 64, 64, "lognormal", dict(rate=8.0), 20, 8, 16384),
    (96, 640, 32, 128, "lognormal", dict(rate=3.0), 3, 2, 8192),              # wide blocks
    (200, 136, 100, 17, "uniform", dict(lo=0.2, hi=0.9), 5, 3, 8192),         # odd block shape: up to four items per block
]


@pytest.mark.parametrize("case", CASES)
def test_panels_decode_to_the_masked_matrix(case):
    rows, cols, br, bc, law, kw, ctas, warps, stage = case
    w = workloads.make_spmv_workload(5, rows, cols, br, bc, law, batch=1, w_std=0.1, val_dtype="f16", **kw)
    m = w.matrix
    A = binding.csb_encode(m.dense, br, bc, m.row_keep, m.col_keep, "f16", device=-1)
    plan = binding.csb_panel_dump(A, ctas, warps, stage)
    assert 1 <= plan["ctas"] <= ctas
    dense, count, ranges = decode(plan, rows, cols, br, warps, stage)
    want = O.masked_dense(m.dense, br, bc, m.row_keep, m.col_keep, "f16")
    mask = O.block_mask(rows, cols, br, bc, m.row_keep, m.col_keep)
    assert np.array_equal(count, mask.astype(np.int32)), "every stored weight exactly once, nothing else"
    assert np.array_equal(dense, want)
    assert ranges[0][0] == 0 and ranges[-1][1] == rows, "the row ranges tile the matrix"
    assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
    assert 0.0 < plan["balance"] <= 1.0 and 0.0 < plan["warp_balance"] <= 1.0
    A.free()


def test_panels_empty_block_rows_and_refusals():
    rng = np.random.default_rng(1)
    W = rng.standard_normal((128, 64)).astype(np.float32)
    rk = np.ones(4 * 32, np.uint8)
    rk[32:64] = 0                                       # block-row 1 keeps nothing
    A = binding.csb_encode(W, 32, 64, rk, np.ones(4 * 64, np.uint8), "f16", device=-1)
    plan = binding.csb_panel_dump(A, 2, 2, 8192)
    dense, count, ranges = decode(plan, 128, 64, 32, 2, 8192)
    assert not dense[32:64].any() and ranges[0][0] == 0 and ranges[-1][1] == 128
    info = np.zeros(8, np.int64)
    small = np.zeros(16, np.uint8)
    rc = binding.lib.csb_panel_dump(A.handle, 2, 2, 8192, info.ctypes.data, small.ctypes.data, small.size, None, 0)
    assert rc == -1 and b"too small" in binding.lib.csb_last_error()
    assert binding.lib.csb_panel_dump(A.handle, 2, 2, 5000, info.ctypes.data, None, 0, None, 0) == -8   # stage not a power of two
    A.free()
    B = binding.csb_encode(W, 32, 64, rk, np.ones(4 * 64, np.uint8), "f32", device=-1)
    assert binding.lib.csb_panel_dump(B.handle, 2, 2, 8192, info.ctypes.data, None, 0, None, 0) == -8      # fp32 values
    B.free()
    # a matrix that keeps nothing at all still plans: one CTA that writes zeros
    Z = binding.csb_encode(W, 32, 64, np.zeros(4 * 32, np.uint8), np.ones(4 * 64, np.uint8), "f16", device=-1)
    plan = binding.csb_panel_dump(Z, 4, 2, 8192)
    dense, count, ranges = decode(plan, 128, 64, 32, 2, 8192)
    assert plan["ctas"] == 1 and ranges == [(0, 128)] and not count.any()
    Z.free()
