"""ctypes binding of libcsb: argument marshalling only.

Every function mirrors one entry point of include/csb.h under the same name.
Device buffers are torch CUDA tensors (torch is used for device memory and
streams only); host buffers are numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

# CSB_LIBRARY names another build of the same sources (an instrumented one, see build.py)
_LIB_PATH = os.environ.get("CSB_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcsb.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError("libcsb.so is not built: run `python -m paper_2005_05758_b200.build` "
                      "(there is no CPU fallback)")
lib = C.CDLL(_LIB_PATH)

CSB_F32, CSB_F16 = 0, 1
CSB_FLAG_ASYNC, CSB_FLAG_HOST_IO = 1, 2
CSB_Q16 = 2
_DT = {"f32": CSB_F32, "f16": CSB_F16}


class csb_plan_opts(C.Structure):
    _fields_ = [("ctas", C.c_int), ("warps_per_cta", C.c_int), ("stage_bytes", C.c_int), ("stages", C.c_int)]


class csb_view_t(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("block_r", C.c_int32), ("block_c", C.c_int32),
                ("nbr", C.c_int64), ("nbc", C.c_int64), ("nblk", C.c_int64), ("nnz", C.c_int64),
                ("val_dtype", C.c_int32),
                ("m", C.POINTER(C.c_uint16)), ("n", C.POINTER(C.c_uint16)),
                ("row_idx", C.POINTER(C.c_uint8)), ("col_idx", C.POINTER(C.c_uint8)),
                ("val_off", C.POINTER(C.c_uint64)), ("ridx_off", C.POINTER(C.c_uint32)),
                ("cidx_off", C.POINTER(C.c_uint32)), ("val", C.c_void_p)]


class csb_info_t(C.Structure):
    _fields_ = [("nnz", C.c_int64), ("pruning_rate", C.c_double), ("nio", C.c_double),
                ("algorithmic_bytes", C.c_int64), ("device_stream_bytes", C.c_int64),
                ("plan_ctas", C.c_int32), ("plan_warps", C.c_int32), ("balance", C.c_double),
                ("panel_stream_bytes", C.c_int64), ("panel_ctas", C.c_int32), ("panel_warps", C.c_int32),
                ("panel_balance", C.c_double)]


_P = C.c_void_p
lib.csb_encode.argtypes = [_P, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, _P, _P, C.c_int, C.c_int,
                           C.POINTER(csb_plan_opts), C.POINTER(_P)]
lib.csb_view.argtypes = [_P, C.POINTER(csb_view_t)]
lib.csb_info.argtypes = [_P, C.POINTER(csb_info_t)]
lib.csb_free.argtypes = [_P]
lib.csb_free.restype = None
lib.csb_spmv.argtypes = [_P, _P, _P, _P]
lib.csb_spmv_static_scratch.argtypes = [_P, _P, _P, _P]
lib.csb_spmv_static_scratch.restype = C.c_int
lib.csb_spmm.argtypes = [_P, _P, C.c_int64, C.c_int, _P, C.c_int64, _P]
lib.csb_lstm_forward.argtypes = [C.c_int, C.POINTER(_P), C.POINTER(_P), _P, C.c_int64, C.c_int, _P, _P, _P, _P, _P,
                                 C.c_uint, _P]
lib.csb_gru_forward.argtypes = [C.c_int, C.POINTER(_P), C.POINTER(_P), _P, C.c_int64, C.c_int, _P, _P, _P,
                                C.c_uint, _P]
lib.csb_test_barrier_hook.argtypes = [C.c_uint, C.c_ulonglong]
lib.csb_test_barrier_hook.restype = None
lib.csb_strerror.argtypes = [C.c_int]
lib.csb_strerror.restype = C.c_char_p
lib.csb_last_error.restype = C.c_char_p
for _f in ("csb_encode", "csb_view", "csb_info", "csb_spmv", "csb_spmm", "csb_lstm_forward", "csb_gru_forward"):
    getattr(lib, _f).restype = C.c_int


class CsbError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__("%s (%d): %s" % (lib.csb_strerror(status).decode(), status,
                                         lib.csb_last_error().decode()))


def _check(status: int) -> None:
    if status != 0:
        raise CsbError(status)


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array (None stays NULL)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


class CsbMatrix:
    """Owner of a csb_matrix_t handle."""

    def __init__(self, handle: int):
        self.handle = handle

    def view(self) -> dict:
        v = csb_view_t()
        _check(lib.csb_view(self.handle, C.byref(v)))
        nblk, nnz = v.nblk, v.nnz

        def arr(p, n, dt):
            if n == 0:
                return np.zeros(0, dt)
            return np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_uint8)), shape=(n * np.dtype(dt).itemsize,)).view(dt).copy()

        ro = arr(v.ridx_off, nblk + 1, np.uint32)
        co = arr(v.cidx_off, nblk + 1, np.uint32)
        vdt = {CSB_F16: np.float16, CSB_F32: np.float32, CSB_Q16: np.int16}[v.val_dtype]
        return {"rows": v.rows, "cols": v.cols, "block_r": v.block_r, "block_c": v.block_c, "nbr": v.nbr,
                "nbc": v.nbc, "nnz": nnz, "val_dtype": {CSB_F16: "f16", CSB_F32: "f32", CSB_Q16: "q16"}[v.val_dtype],
                "m": arr(v.m, nblk, np.uint16), "n": arr(v.n, nblk, np.uint16),
                "row_idx": arr(v.row_idx, int(ro[-1]), np.uint8), "col_idx": arr(v.col_idx, int(co[-1]), np.uint8),
                "val_off": arr(v.val_off, nblk + 1, np.uint64), "ridx_off": ro, "cidx_off": co,
                "val": arr(v.val, nnz, vdt)}

    def info(self) -> dict:
        o = csb_info_t()
        _check(lib.csb_info(self.handle, C.byref(o)))
        return {k: getattr(o, k) for k, _ in csb_info_t._fields_}

    def free(self) -> None:
        if self.handle:
            lib.csb_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def csb_encode(dense: np.ndarray, block_r: int, block_c: int, row_keep: np.ndarray, col_keep: np.ndarray,
               val_dtype: str = "f16", device: int = 0, opts: Optional[dict] = None) -> CsbMatrix:
    dense = np.ascontiguousarray(dense, dtype=np.float32)
    rk = np.ascontiguousarray(row_keep, dtype=np.uint8)
    ck = np.ascontiguousarray(col_keep, dtype=np.uint8)
    rows, cols = dense.shape
    nblk = -(-rows // block_r) * -(-cols // block_c) if block_r > 0 and block_c > 0 else 0
    if block_r > 0 and block_c > 0 and (rk.size != nblk * block_r or ck.size != nblk * block_c):
        raise ValueError("keep masks must hold nblk*block_r and nblk*block_c bytes")
    o = csb_plan_opts(**opts) if opts else None
    out = _P()
    _check(lib.csb_encode(dense.ctypes.data, rows, cols, cols, block_r, block_c, rk.ctypes.data, ck.ctypes.data,
                          _DT[val_dtype] if isinstance(val_dtype, str) else val_dtype, device,
                          C.byref(o) if o else None, C.byref(out)))
    return CsbMatrix(out.value)


def csb_plan_dump(A: CsbMatrix, ctas: int, warps_per_cta: int, stage_bytes: int) -> dict:
    """Host-only plan of the bare product, copied out for inspection (see csb.h)."""
    lib.csb_plan_dump.argtypes = [_P, C.c_int, C.c_int, C.c_int, _P, _P, C.c_int64, _P, C.c_int64, _P, C.c_int64]
    lib.csb_plan_dump.restype = C.c_int
    info = np.zeros(8, np.int64)
    _check(lib.csb_plan_dump(A.handle, ctas, warps_per_cta, stage_bytes, info.ctypes.data, None, 0, None, 0, None, 0))
    stream = np.zeros(max(int(info[2]), 1), np.uint8)
    chunks = np.zeros((max(int(info[1]), 1), 2), np.uint32)
    wbeg = np.zeros(int(info[0]) + 1, np.uint32)
    _check(lib.csb_plan_dump(A.handle, ctas, warps_per_cta, stage_bytes, info.ctypes.data, stream.ctypes.data, stream.size,
                             chunks.ctypes.data, chunks.shape[0], wbeg.ctypes.data, wbeg.size))
    keys = ("warps", "chunks", "stream_bytes", "group_width", "row_owned", "ctas", "warps_per_cta", "slots")
    out = {k: int(v) for k, v in zip(keys, info)}
    out.update(stream=stream[: out["stream_bytes"]], chunk_table=chunks[: out["chunks"]], warp_begin=wbeg)
    return out


def csb_encode_q16(dense: np.ndarray, block_r: int, block_c: int, row_keep: np.ndarray, col_keep: np.ndarray, frac_bits: int,
                   device: int = 0) -> CsbMatrix:
    """CSB handle with 16-bit fixed-point values (see csb.h); serves csb_spmm_q16 only."""
    lib.csb_encode_q16.argtypes = [_P, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, _P, _P, C.c_int, C.c_int, C.POINTER(_P)]
    lib.csb_encode_q16.restype = C.c_int
    dense = np.ascontiguousarray(dense, dtype=np.float32)
    rk = np.ascontiguousarray(row_keep, dtype=np.uint8)
    ck = np.ascontiguousarray(col_keep, dtype=np.uint8)
    rows, cols = dense.shape
    out = _P()
    _check(lib.csb_encode_q16(dense.ctypes.data, rows, cols, cols, block_r, block_c, rk.ctypes.data, ck.ctypes.data, frac_bits, device,
                              C.byref(out)))
    return CsbMatrix(out.value)


def csb_spmm_q16(A: CsbMatrix, Xq, acc, stream=None) -> None:
    """acc[b, :] = A_q . Xq[b, :] in integers: Xq torch int16 [batch, cols], acc torch int64 [batch, rows]."""
    lib.csb_spmm_q16.argtypes = [_P, _P, C.c_int64, C.c_int, _P, C.c_int64, _P]
    lib.csb_spmm_q16.restype = C.c_int
    batch = Xq.shape[0]
    _check(lib.csb_spmm_q16(A.handle, _ptr(Xq), Xq.stride(0) if batch else 0, batch, _ptr(acc), acc.stride(0) if batch else 0, _stream(stream)))


def csb_spmm_plan_dump(A: CsbMatrix, batch: int, sm_count: int) -> dict:
    """Host-only plan of the tensor-core batched product, copied out for inspection (see csb.h)."""
    lib.csb_spmm_plan_dump.argtypes = [_P, C.c_int, C.c_int, _P, _P, C.c_int64, _P, C.c_int64, _P, C.c_int64, _P, C.c_int64]
    lib.csb_spmm_plan_dump.restype = C.c_int
    info = np.zeros(8, np.int64)
    _check(lib.csb_spmm_plan_dump(A.handle, batch, sm_count, info.ctypes.data, None, 0, None, 0, None, 0, None, 0))
    n_ctas, n_chunks, n_bytes = (int(v) for v in info[:3])
    NT, warps, tile_blocks = int(info[4]) & 255, (int(info[4]) >> 8) & 255, int(info[4]) >> 16
    stream = np.zeros(max(n_bytes, 1), np.uint8)
    chunks = np.zeros((max(n_chunks, 1), 2), np.uint32)
    begin = np.zeros(n_ctas * warps + 1, np.uint32)
    cta = np.zeros((max(n_ctas, 1), 48), np.uint8)
    _check(lib.csb_spmm_plan_dump(A.handle, batch, sm_count, info.ctypes.data, stream.ctypes.data, stream.size, chunks.ctypes.data,
                                  chunks.shape[0], begin.ctypes.data, begin.size, cta.ctypes.data, cta.shape[0]))
    cta = cta[:n_ctas]
    return {"ctas": n_ctas, "RG": int(info[3]), "NT": NT, "warps": warps, "tile_blocks": tile_blocks, "S": int(info[5]), "warp_balance": info[6] / 1e6,
            "balance": info[7] / 1e6, "stream": stream[:n_bytes], "chunk_table": chunks[:n_chunks], "stream_begin": begin,
            "cta": cta[:, :16].copy().view(np.int32).reshape(n_ctas, 4), "warp_row": cta[:, 16:16 + warps].copy()}


def csb_panel_dump(A: CsbMatrix, ctas: int, warps_per_cta: int, stage_bytes: int) -> dict:
    """Host-only plan of the batch-1 panel layout, copied out for inspection (see csb.h)."""
    lib.csb_panel_dump.argtypes = [_P, C.c_int, C.c_int, C.c_int, _P, _P, C.c_int64, _P, C.c_int64]
    lib.csb_panel_dump.restype = C.c_int
    info = np.zeros(8, np.int64)
    _check(lib.csb_panel_dump(A.handle, ctas, warps_per_cta, stage_bytes, info.ctypes.data, None, 0, None, 0))
    panels = np.zeros(max(int(info[1]), 1), np.uint8)
    cta = np.zeros((max(int(info[0]), 1), 4), np.uint32)
    _check(lib.csb_panel_dump(A.handle, ctas, warps_per_cta, stage_bytes, info.ctypes.data, panels.ctypes.data, panels.size,
                              cta.ctypes.data, cta.shape[0]))
    return {"ctas": int(info[0]), "bytes": int(info[1]), "max_meta": int(info[3]),
            "max_xg": int(info[4]), "max_rows": int(info[5]), "balance": info[6] / 1e6, "warp_balance": info[7] / 1e6,
            "panels": panels[: int(info[1])], "cta": cta[: int(info[0])]}


def csb_project(W, block_r: int, block_c: int, prune_fraction: float, row_keep=None, col_keep=None, workspace=None,
                stream=None):
    """Keep masks of the projection of the device matrix W (torch, float32, 2-D) onto the CSB pattern;
    returns (row_keep, col_keep, workspace) as torch uint8 tensors on W's device (allocated when not given)."""
    import torch
    lib.csb_project_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int, C.c_int]
    lib.csb_project_workspace_bytes.restype = C.c_int64
    lib.csb_project.argtypes = [_P, C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_double, _P, _P, _P, C.c_int64, _P]
    lib.csb_project.restype = C.c_int
    rows, cols = W.shape
    nblk = -(-rows // block_r) * -(-cols // block_c) if block_r > 0 and block_c > 0 else 0
    if row_keep is None:
        row_keep = torch.empty(max(nblk * block_r, 1), dtype=torch.uint8, device=W.device)
    if col_keep is None:
        col_keep = torch.empty(max(nblk * block_c, 1), dtype=torch.uint8, device=W.device)
    if workspace is None:
        workspace = torch.empty(max(int(lib.csb_project_workspace_bytes(rows, cols, block_r, block_c)), 16), dtype=torch.uint8,
                                device=W.device)
    _check(lib.csb_project(_ptr(W), rows, cols, W.stride(0), block_r, block_c, float(prune_fraction), _ptr(row_keep),
                           _ptr(col_keep), _ptr(workspace), workspace.numel(), _stream(stream)))
    return row_keep, col_keep, workspace


def csb_spmv(A: CsbMatrix, x, y, stream=None) -> None:
    _check(lib.csb_spmv(A.handle, _ptr(x), _ptr(y), _stream(stream)))


def csb_spmv_static_scratch(A: CsbMatrix, x, y, stream=None) -> None:
    """csb_spmv for callers that may not allocate device memory: the kernel's scratch is a fixed
    array inside the library (4 MiB per GPU), shared by all handles -- do not overlap calls."""
    _check(lib.csb_spmv_static_scratch(A.handle, _ptr(x), _ptr(y), _stream(stream)))


def csb_spmm(A: CsbMatrix, X, Y, stream=None) -> None:
    batch = X.shape[0]
    _check(lib.csb_spmm(A.handle, _ptr(X), X.stride(0) if batch else 0, batch, _ptr(Y),
                        Y.stride(0) if batch else 0, _stream(stream)))


def _ptr_array(items: Sequence, n: int):
    arr = (_P * n)()
    for i in range(n):
        arr[i] = _ptr(items[i]) if not isinstance(items[i], CsbMatrix) else items[i].handle
    return arr


def csb_lstm_forward(W: Sequence[CsbMatrix], bias, x, h0, c0, y, hT, cT, flags: int = 0, stream=None) -> None:
    L = len(W)
    T, B = (x.shape[0], x.shape[1])
    b = _ptr_array(bias, L) if bias is not None else None
    _check(lib.csb_lstm_forward(L, _ptr_array(W, L), b, _ptr(x), T, B, _ptr(h0), _ptr(c0), _ptr(y), _ptr(hT),
                                _ptr(cT), flags, _stream(stream)))


def csb_gru_forward(W: Sequence[CsbMatrix], bias, x, h0, y, hT, flags: int = 0, stream=None) -> None:
    L = len(W)
    T, B = (x.shape[0], x.shape[1])
    b = _ptr_array(bias, L) if bias is not None else None
    _check(lib.csb_gru_forward(L, _ptr_array(W, L), b, _ptr(x), T, B, _ptr(h0), _ptr(y), _ptr(hT), flags,
                               _stream(stream)))


def csb_lstmp_forward(W: Sequence[CsbMatrix], Wp: Sequence[CsbMatrix], bias, x, h0, c0, y, hT, cT, flags: int = 0, stream=None) -> None:
    L = len(W)
    lib.csb_lstmp_forward.argtypes = [C.c_int, C.POINTER(_P), C.POINTER(_P), C.POINTER(_P), _P, C.c_int64, C.c_int, _P, _P, _P, _P, _P, C.c_uint, _P]
    lib.csb_lstmp_forward.restype = C.c_int
    b = _ptr_array(bias, L) if bias is not None else None
    _check(lib.csb_lstmp_forward(L, _ptr_array(W, L), _ptr_array(Wp, L), b, _ptr(x), x.shape[0], x.shape[1], _ptr(h0), _ptr(c0), _ptr(y),
                                 _ptr(hT), _ptr(cT), flags, _stream(stream)))


def _gru_like(fn, W, bias, x, h0, y, hT, flags, stream):
    L = len(W)
    fn.argtypes = [C.c_int, C.POINTER(_P), C.POINTER(_P), _P, C.c_int64, C.c_int, _P, _P, _P, C.c_uint, _P]
    fn.restype = C.c_int
    b = _ptr_array(bias, L) if bias is not None else None
    _check(fn(L, _ptr_array(W, L), b, _ptr(x), x.shape[0], x.shape[1], _ptr(h0), _ptr(y), _ptr(hT), flags, _stream(stream)))


def csb_ligru_forward(W: Sequence[CsbMatrix], bias, x, h0, y, hT, flags: int = 0, stream=None) -> None:
    _gru_like(lib.csb_ligru_forward, W, bias, x, h0, y, hT, flags, stream)


def csb_gru_reset_before_forward(W: Sequence[CsbMatrix], bias, x, h0, y, hT, flags: int = 0, stream=None) -> None:
    _gru_like(lib.csb_gru_reset_before_forward, W, bias, x, h0, y, hT, flags, stream)


# shorter aliases
spmv, spmm, lstm_forward, gru_forward = csb_spmv, csb_spmm, csb_lstm_forward, csb_gru_forward
