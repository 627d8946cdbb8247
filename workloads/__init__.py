"""Seeded synthetic inputs for the CSB-RNN hot path.

This package only draws random numbers and shapes them into dense weights,
per-block keep masks and input sequences.  It contains none of the method's
arithmetic (no masking, no products, no encoding, no recurrences), so both the
CPU oracle and the CUDA library can be fed from it without sharing code.
"""
from .configs import (  # noqa: F401
    CONFIGS,
    MatrixSpec,
    RnnWorkload,
    SpmvWorkload,
    block_grid,
    draw_keep_masks,
    make_matrix,
    make_rnn_workload,
    make_spmv_workload,
)
