"""Seeded generators for the five synthetic workloads.

The paper evaluates on trained, ADMM-pruned speech / language models (Table 1);
none of those weights or datasets is available, so the generators below take
their layer shapes, block sizes (16/32/64, Section 6.2.1), pruning rates
(3.5x-25x) and the uneven per-block sparsity (Section 4.3.2) and draw synthetic
stand-ins.  Only random draws and shaping happen here: no masking, no product,
no encoding.

Streams: ``numpy.random.Generator(PCG64)`` seeded from ``SeedSequence(seed)``
spawned into three children, in this order: weights, masks, inputs.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np


def block_grid(rows: int, cols: int, br: int, bc: int) -> Tuple[int, int]:
    """Number of block-rows and block-columns (the last ones may be partial)."""
    return -(-rows // br), -(-cols // bc)


def _streams(seed: int, n: int = 3):
    return [np.random.Generator(np.random.PCG64(s)) for s in np.random.SeedSequence(seed).spawn(n)]


@dataclass
class MatrixSpec:
    """A dense weight with its per-block keep masks (inputs of the encoder)."""
    dense: np.ndarray            # float32 [rows, cols], C-contiguous
    block_r: int
    block_c: int
    row_keep: np.ndarray         # uint8 [nblk * block_r], block b = bi * nbc + bj
    col_keep: np.ndarray         # uint8 [nblk * block_c]
    val_dtype: str = "f16"       # storage type of the packed values: "f16" | "f32"

    @property
    def rows(self) -> int:
        return int(self.dense.shape[0])

    @property
    def cols(self) -> int:
        return int(self.dense.shape[1])


def _logical_sizes(rows, cols, br, bc):
    """Per-block count of in-range rows and columns (edge blocks are partial)."""
    nbr, nbc = block_grid(rows, cols, br, bc)
    rs = np.minimum(br, rows - np.arange(nbr) * br)
    cs = np.minimum(bc, cols - np.arange(nbc) * bc)
    return np.repeat(rs, nbc), np.tile(cs, nbr)


def _subset_masks(rng, counts: np.ndarray, sizes: np.ndarray, width: int) -> np.ndarray:
    """For each block pick ``counts[b]`` of its first ``sizes[b]`` lines uniformly."""
    nblk = counts.shape[0]
    keys = rng.random((nblk, width))
    keys[np.arange(width)[None, :] >= sizes[:, None]] = 2.0   # out-of-range lines last
    rank = np.argsort(np.argsort(keys, axis=1, kind="stable"), axis=1, kind="stable")
    return (rank < counts[:, None]).astype(np.uint8).reshape(-1)


def _counts_from_fraction(frac: np.ndarray, sizes: np.ndarray) -> np.ndarray:
    return np.clip(np.rint(frac * sizes), 0, sizes).astype(np.int64)


def draw_keep_masks(rng, rows, cols, br, bc, law: str, *, count=None, lo=None, hi=None,
                    sigma=0.8, rate=None, diag_boost=1.0):
    """Per-block row / column keep masks.

    law = "exact":     every block keeps exactly ``count`` rows and columns.
    law = "uniform":   keep fractions f_r, f_c ~ U(lo, hi) i.i.d. per block.
    law = "lognormal": f = f0 * exp(sigma * z - sigma^2 / 2), z ~ N(0, 1) i.i.d.
                       for rows and columns; f0 bisected so that
                       rows * cols / sum(m_b * n_b) lands within 1 % of ``rate``.
    ``diag_boost`` multiplies the keep fraction of diagonal blocks (the
    diagonal-dense pattern is the worst imbalance the paper reports, Sec. 6.3.2).
    """
    nbr, nbc = block_grid(rows, cols, br, bc)
    nblk = nbr * nbc
    rsz, csz = _logical_sizes(rows, cols, br, bc)
    boost = np.ones(nblk)
    if diag_boost != 1.0:
        bi, bj = np.divmod(np.arange(nblk), nbc)
        boost[bi * nbc // max(nbr, 1) == bj] = diag_boost
    if law == "exact":
        m = np.minimum(count, rsz).astype(np.int64)
        n = np.minimum(count, csz).astype(np.int64)
    elif law == "uniform":
        m = _counts_from_fraction(rng.uniform(lo, hi, nblk) * boost, rsz)
        n = _counts_from_fraction(rng.uniform(lo, hi, nblk) * boost, csz)
    elif law == "lognormal":
        zr, zc = rng.standard_normal(nblk), rng.standard_normal(nblk)
        er = np.exp(sigma * zr - 0.5 * sigma * sigma) * boost
        ec = np.exp(sigma * zc - 0.5 * sigma * sigma) * boost

        def achieved(f0):
            mm = _counts_from_fraction(f0 * er, rsz)
            nn = _counts_from_fraction(f0 * ec, csz)
            return mm, nn, float(rows) * cols / max(int((mm * nn).sum()), 1)

        f_lo, f_hi = 1e-3, 4.0
        for _ in range(60):
            f0 = 0.5 * (f_lo + f_hi)
            m, n, r = achieved(f0)
            if abs(r - rate) <= 0.01 * rate:
                break
            if r > rate:      # too sparse: keep more
                f_lo = f0
            else:
                f_hi = f0
    else:
        raise ValueError(law)
    return _subset_masks(rng, m, rsz, br), _subset_masks(rng, n, csz, bc)


def make_matrix(seed, rows, cols, br, bc, law, *, w_std, val_dtype="f16", **mask_kw) -> MatrixSpec:
    rng_w, rng_m, _ = _streams(seed)
    dense = rng_w.standard_normal((rows, cols), dtype=np.float32) * np.float32(w_std)
    rk, ck = draw_keep_masks(rng_m, rows, cols, br, bc, law, **mask_kw)
    return MatrixSpec(np.ascontiguousarray(dense), br, bc, rk, ck, val_dtype)


@dataclass
class RnnWorkload:
    """One recurrent workload: stacked layers, an input sequence, initial state."""
    cell: str                        # "lstm" | "gru" | "lstmp" | "ligru" | "gru_rb" (reset gate before the product)
    input_size: int
    hidden_size: int
    layers: List[MatrixSpec]         # layer l: [G*H, I_l + S], S = size of the recurrent state (H, or the projection size)
    bias: List[Optional[np.ndarray]]  # per layer float32 (lstm, lstmp, gru: [4*H]; gru_rb: [3*H]; ligru: [2*H]) or None
    x: np.ndarray                    # float32 [T, B, I]
    h0: Optional[np.ndarray]         # float32 [L, B, S] or None (= zeros)
    c0: Optional[np.ndarray]         # float32 [L, B, H] (lstm, lstmp)
    name: str = ""
    proj: Optional[List[MatrixSpec]] = None   # lstmp: per layer the projection [P, H]
    proj_size: int = 0

    @property
    def T(self) -> int:
        return int(self.x.shape[0])

    @property
    def B(self) -> int:
        return int(self.x.shape[1])


@dataclass
class SpmvWorkload:
    matrix: MatrixSpec
    X: np.ndarray                    # float32 [batch, cols]
    name: str = ""


GATES = {"lstm": 4, "lstmp": 4, "gru": 3, "gru_rb": 3, "ligru": 2}
BIAS_ROWS = {"lstm": 4, "lstmp": 4, "gru": 4, "gru_rb": 3, "ligru": 2}


def make_rnn_workload(seed, cell, I, H, n_layers, br, bc, law, *, T, B, w_std, x_law="normal",
                      val_dtype="f16", bias_std=0.0, state_std=0.0, name="", proj_size=0, **mask_kw) -> RnnWorkload:
    G = GATES[cell]
    S = proj_size if cell == "lstmp" else H          # width of the recurrent state
    layers, biases, proj = [], [], []
    _, _, rng_x = _streams(seed)
    for l in range(n_layers):
        in_l = I if l == 0 else S
        layers.append(make_matrix(seed + 1000 * l, G * H, in_l + S, br, bc, law,
                                  w_std=w_std, val_dtype=val_dtype, **mask_kw))
        if cell == "lstmp":
            proj.append(make_matrix(seed + 1000 * l + 500, S, H, br, bc, law, w_std=w_std, val_dtype=val_dtype, **mask_kw))
    if x_law == "normal":
        x = rng_x.standard_normal((T, B, I), dtype=np.float32)
    else:
        x = rng_x.uniform(-1.0, 1.0, (T, B, I)).astype(np.float32)
    for l in range(n_layers):
        biases.append((rng_x.standard_normal(BIAS_ROWS[cell] * H) * bias_std).astype(np.float32) if bias_std > 0 else None)
    h0 = c0 = None
    if state_std > 0:
        h0 = (rng_x.standard_normal((n_layers, B, S)) * state_std).astype(np.float32)
        c0 = (rng_x.standard_normal((n_layers, B, H)) * state_std).astype(np.float32)
    return RnnWorkload(cell, I, H, layers, biases, x, h0, c0 if cell in ("lstm", "lstmp") else None, name,
                       proj if cell == "lstmp" else None, S if cell == "lstmp" else 0)


def make_spmv_workload(seed, rows, cols, br, bc, law, *, batch, w_std, val_dtype="f16", name="",
                       **mask_kw) -> SpmvWorkload:
    mat = make_matrix(seed, rows, cols, br, bc, law, w_std=w_std, val_dtype=val_dtype, **mask_kw)
    _, _, rng_x = _streams(seed)
    X = rng_x.standard_normal((batch, cols), dtype=np.float32)
    return SpmvWorkload(mat, X, name)


def _cfg1(B=1, T=16, **kw):
    return make_rnn_workload(0, "lstm", 64, 128, 1, 16, 16, "exact", count=8, T=T, B=B, w_std=0.1,
                             x_law="uniform", val_dtype="f32", name="cfg1_lstm_64_128_b16_f32", **kw)


def _cfg2(B=1, T=100, **kw):
    return make_rnn_workload(0, "lstm", 153, 1024, 1, 32, 32, "uniform", lo=0.25, hi=0.45, T=T, B=B,
                             w_std=0.05, name="cfg2_lstm_153_1024_b32_f16", **kw)


def _cfg3(B=1, T=256, **kw):
    return make_rnn_workload(0, "gru", 512, 1024, 1, 32, 32, "lognormal", rate=16.0, sigma=0.8, T=T,
                             B=B, w_std=0.05, name="cfg3_gru_512_1024_b32_f16", **kw)


def _cfg4(rate=4.0, B=1, diag_boost=1.0, n=8192, **kw):
    return make_spmv_workload(0, n, n, 64, 64, "lognormal", rate=float(rate), sigma=0.8, batch=B,
                              w_std=0.05, diag_boost=diag_boost,
                              name="cfg4_spmv_%d_b64_f16_r%g" % (n, rate), **kw)


def _cfg5(B=1, T=512, **kw):
    return make_rnn_workload(0, "lstm", 2048, 2048, 2, 64, 64, "uniform", lo=0.216, hi=0.416, T=T,
                             B=B, w_std=0.05, name="cfg5_lstm2_2048_b64_f16", **kw)


#: name -> factory.  Keyword arguments override batch / sequence length / rate.
CONFIGS = {"cfg1": _cfg1, "cfg2": _cfg2, "cfg3": _cfg3, "cfg4": _cfg4, "cfg5": _cfg5}
