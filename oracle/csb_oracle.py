"""CPU oracle for the CSB matrix, its storage format and its product.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  It shares no code with the library, never
calls it, and must not be used by any product path.  Arithmetic is float64.

Notation (the paper's letters are used inconsistently between Section 3.1.1,
Algorithm 1 and Section 4.3.1, so they are fixed here): the matrix is R x C
(rows = output neurons, columns = input neurons, Section 3.1.2), tiled into
BR x BC blocks; block b = bi * nbc + bj in row-major block order; block b keeps
m_b rows and n_b columns; its survivors form the dense m_b x n_b kernel matrix.

What is pinned and by what (tests/test_oracle_*.py):
  block_mask / masked_dense / spmm : brute force over all 256 mask settings of a
      4x4 matrix with 2x2 blocks; all-kept special case equals a dense product;
      linearity; rows kept nowhere give exact zeros.
  encode / decode / nio            : round trip to the masked dense matrix,
      prefix-sum and ordering invariants, hand-written 4x6 example, NIO closed
      form against the paper's "about 20 % at block size 32" (Section 6.2.1).
  round_to_storage                 : IEEE binary16 facts (ties to even, range).
"""
from __future__ import annotations

import numpy as np


def grid(R, C, BR, BC):
    """Block-grid extents; a short last block is allowed (the paper zero-pads
    a short dimension and splits it evenly, Section 6.2.1)."""
    return -(-R // BR), -(-C // BC)


def block_mask(R, C, BR, BC, row_keep, col_keep):
    """Section 3.1.1: inside block b whole rows and whole columns are zeroed, so
    element (r, c) survives iff its row AND its column are kept in its block.
    row_keep is [nblk * BR], col_keep is [nblk * BC] (non-zero = kept); bits that
    fall beyond the matrix edge are ignored."""
    nbr, nbc = grid(R, C, BR, BC)
    rk = np.asarray(row_keep).reshape(nbr, nbc, BR) != 0
    ck = np.asarray(col_keep).reshape(nbr, nbc, BC) != 0
    mask = np.zeros((R, C), dtype=bool)
    for r in range(R):
        bi, lr = divmod(r, BR)
        # columns kept in each block of this block-row, laid side by side
        cols_kept = ck[bi].reshape(nbc * BC)[:C]
        rows_kept = np.repeat(rk[bi, :, lr], BC)[:C]
        mask[r] = rows_kept & cols_kept
    return mask


def round_to_storage(W, val_dtype):
    """Values are stored either as given (binary32) or rounded to binary16 with
    round-to-nearest-even; overflow gives +-inf as IEEE prescribes."""
    W32 = np.asarray(W, dtype=np.float32)
    if val_dtype == "f32":
        return W32.astype(np.float64)
    if val_dtype == "f16":
        with np.errstate(over="ignore"):
            return W32.astype(np.float16).astype(np.float64)
    raise ValueError(val_dtype)


def masked_dense(W, BR, BC, row_keep, col_keep, val_dtype):
    """The matrix a CSB encoding stands for: stored values at kept cross-points,
    exact zeros elsewhere."""
    R, C = W.shape
    mask = block_mask(R, C, BR, BC, row_keep, col_keep)
    return np.where(mask, round_to_storage(W, val_dtype), 0.0)


def spmm(W, BR, BC, row_keep, col_keep, val_dtype, X):
    """CSB-MVM (Section 4.2): Y[beta] = Wm . X[beta] for every batch row beta.
    X is [batch, C]; returns [batch, R] in float64.  batch = 1 is the SpMV."""
    Wm = masked_dense(W, BR, BC, row_keep, col_keep, val_dtype)
    return np.asarray(X, dtype=np.float64) @ Wm.T


def abs_scale(W, BR, BC, row_keep, col_keep, val_dtype, X):
    """sum_c |Wm[r, c]| * |X[beta, c]|: the size of the terms each output sums,
    i.e. the scale against which a rounding error of that output is judged."""
    Wm = masked_dense(W, BR, BC, row_keep, col_keep, val_dtype)
    return np.abs(np.asarray(X, dtype=np.float64)) @ np.abs(Wm).T


def encode(W, BR, BC, row_keep, col_keep, val_dtype):
    """The CSB storage format of Section 3.1.1, written as plain loops.

    Arrays (the paper's five, plus offsets):
      m[b], n[b]        kept-row / kept-column count of block b (the kernel matrix is m x n)
      row_idx, col_idx  in-block, 0-based, ascending indices of the kept rows / columns,
                        blocks concatenated in row-major block order
      val               kernel matrices of successive blocks concatenated; inside a
                        block the m x n kernel matrix is row-major
      val_off, ridx_off, cidx_off   exclusive prefix sums of m*n, m, n (length nblk + 1).
                        The paper leaves offsets out because its hardware walks the
                        blocks in sequence; random access needs them.
    A block with m = 0 or n = 0 stores no values but still lists the other side's
    indices.  Mask bits beyond the matrix edge are ignored.
    """
    W = np.asarray(W, dtype=np.float32)
    R, C = W.shape
    nbr, nbc = grid(R, C, BR, BC)
    np_val = np.float16 if val_dtype == "f16" else np.float32
    with np.errstate(over="ignore"):
        Wq = W.astype(np_val)
    m, n, row_idx, col_idx, val = [], [], [], [], []
    val_off, ridx_off, cidx_off = [0], [0], [0]
    for bi in range(nbr):
        for bj in range(nbc):
            b = bi * nbc + bj
            rows = [i for i in range(BR) if bi * BR + i < R and row_keep[b * BR + i]]
            cols = [j for j in range(BC) if bj * BC + j < C and col_keep[b * BC + j]]
            m.append(len(rows))
            n.append(len(cols))
            row_idx.extend(rows)
            col_idx.extend(cols)
            for i in rows:
                for j in cols:
                    val.append(Wq[bi * BR + i, bj * BC + j])
            val_off.append(val_off[-1] + len(rows) * len(cols))
            ridx_off.append(ridx_off[-1] + len(rows))
            cidx_off.append(cidx_off[-1] + len(cols))
    if not (1 <= BR <= 256 and 1 <= BC <= 256):
        raise ValueError("block sizes 1..256 only (in-block indices are one byte)")
    idx_t, cnt_t = np.uint8, np.uint16      # a count can reach 256, an index cannot
    return {
        "rows": R, "cols": C, "block_r": BR, "block_c": BC, "nbr": nbr, "nbc": nbc,
        "val_dtype": val_dtype,
        "m": np.array(m, dtype=cnt_t), "n": np.array(n, dtype=cnt_t),
        "row_idx": np.array(row_idx, dtype=idx_t), "col_idx": np.array(col_idx, dtype=idx_t),
        "val": np.array(val, dtype=np_val),
        "val_off": np.array(val_off, dtype=np.uint64),
        "ridx_off": np.array(ridx_off, dtype=np.uint32),
        "cidx_off": np.array(cidx_off, dtype=np.uint32),
    }


def decode(enc):
    """Inverse of encode: scatter every kernel matrix back to its cross-points."""
    R, C, BR, BC, nbc = enc["rows"], enc["cols"], enc["block_r"], enc["block_c"], enc["nbc"]
    out = np.zeros((R, C), dtype=np.float64)
    for b in range(len(enc["m"])):
        bi, bj = divmod(b, nbc)
        rows = enc["row_idx"][enc["ridx_off"][b]:enc["ridx_off"][b + 1]]
        cols = enc["col_idx"][enc["cidx_off"][b]:enc["cidx_off"][b + 1]]
        v = enc["val"][int(enc["val_off"][b]):int(enc["val_off"][b + 1])].astype(np.float64)
        p = 0
        for i in rows:
            for j in cols:
                out[bi * BR + int(i), bj * BC + int(j)] = v[p]
                p += 1
    return out


def spmv_from_encoding(enc, x):
    """CSB-MVM taken block by block as the CSB-Engine does (Section 4.3.1): read
    the kept inputs through ColIdx, multiply by the kernel matrix, accumulate
    into the outputs through RowIdx, block-rows accumulated horizontally."""
    R, BR, BC, nbc = enc["rows"], enc["block_r"], enc["block_c"], enc["nbc"]
    x = np.asarray(x, dtype=np.float64)
    y = np.zeros(R, dtype=np.float64)
    for b in range(len(enc["m"])):
        bi, bj = divmod(b, nbc)
        rows = enc["row_idx"][enc["ridx_off"][b]:enc["ridx_off"][b + 1]]
        cols = enc["col_idx"][enc["cidx_off"][b]:enc["cidx_off"][b + 1]]
        p = int(enc["val_off"][b])
        for i in rows:
            acc = 0.0
            for j in cols:
                acc += float(enc["val"][p]) * x[bj * BC + int(j)]
                p += 1
            y[bi * BR + int(i)] += acc
    return y


def nio(enc):
    """Normalized index overhead (Section 6.2.1): index entries per stored weight,
    sum(m_b + n_b) / sum(m_b * n_b)."""
    m = enc["m"].astype(np.int64)
    n = enc["n"].astype(np.int64)
    nnz = int((m * n).sum())
    return float((m + n).sum()) / nnz if nnz else float("inf")


def pruning_rate(enc):
    """Weight count of the original model over that of the pruned one (Section 1)."""
    nnz = int((enc["m"].astype(np.int64) * enc["n"].astype(np.int64)).sum())
    return enc["rows"] * enc["cols"] / nnz if nnz else float("inf")
