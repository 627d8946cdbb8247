"""ctypes access to oracle/csb_loops.c (test infrastructure; see that file's header)."""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libcsb_loops.so")


def build(force=False):
    src = os.path.join(_HERE, "csb_loops.c")
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(src):
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, src], check=True)
    return _SO


def _lib():
    lib = C.CDLL(build())
    lib.csb_loops_encode.restype = C.c_void_p
    lib.csb_loops_encode.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
    lib.csb_loops_free.argtypes = [C.c_void_p]
    lib.csb_loops_nnz.argtypes = [C.c_void_p]
    lib.csb_loops_nnz.restype = C.c_int64
    lib.csb_loops_spmv.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
    lib.csb_loops_time_spmv.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int]
    lib.csb_loops_time_spmv.restype = C.c_double
    return lib


class CsbLoops:
    """The plain CSB loop nest on the CPU for one matrix (values as stored: pass them rounded)."""

    def __init__(self, stored, br, bc, row_keep, col_keep):
        self.lib = _lib()
        self.stored = np.ascontiguousarray(stored, dtype=np.float32)
        self.rows, self.cols = self.stored.shape
        rk = np.ascontiguousarray(row_keep, dtype=np.uint8)
        ck = np.ascontiguousarray(col_keep, dtype=np.uint8)
        self.h = self.lib.csb_loops_encode(self.stored.ctypes.data, self.rows, self.cols, br, bc, rk.ctypes.data, ck.ctypes.data)

    @property
    def nnz(self):
        return self.lib.csb_loops_nnz(self.h)

    def spmv(self, x, threads=1):
        x = np.ascontiguousarray(x, dtype=np.float64)
        y = np.empty(self.rows, np.float64)
        self.lib.csb_loops_spmv(self.h, x.ctypes.data, y.ctypes.data, threads)
        return y

    def seconds_per_spmv(self, x, threads=1, reps=5):
        x = np.ascontiguousarray(x, dtype=np.float64)
        y = np.empty(self.rows, np.float64)
        return self.lib.csb_loops_time_spmv(self.h, x.ctypes.data, y.ctypes.data, threads, reps)

    def __del__(self):
        try:
            self.lib.csb_loops_free(self.h)
        except Exception:
            pass
