"""B200-native CSB sparse products and fused LSTM / GRU time loop (libcsb).

The work is done by hand-written sm_100a kernels behind a C ABI (include/csb.h);
this package only marshals arguments.  There is no CPU fallback: touching any
of the library's functions fails loudly when the shared library is missing.

``paper_2005_05758_b200.build`` compiles the library and is importable before
it exists; everything else is loaded from ``binding`` on first use.
"""
_LAZY = ("CsbError", "CsbMatrix", "lib", "csb_encode", "csb_spmv", "csb_spmm", "csb_lstm_forward",
         "csb_gru_forward", "spmv", "spmm", "lstm_forward", "gru_forward")


def __getattr__(name):
    if name in _LAZY:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
