"""B200-native CSB sparse products and fused LSTM / GRU time loop (libcsb).

The work is done by hand-written sm_100a kernels behind a C ABI (include/csb.h);
this package only marshals arguments.  There is no CPU fallback: importing
``binding`` fails loudly when the shared library is missing.
"""
from .binding import (  # noqa: F401
    CsbError,
    CsbMatrix,
    gru_forward,
    lib,
    lstm_forward,
    spmm,
    spmv,
)
