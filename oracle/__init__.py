"""CPU oracle for the aggregation primitive: ctypes front end of ``ap_oracle.c``.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this package; it exists so
that the tests, the smoke check and the benchmark's CPU-baseline leg have an independent,
obviously correct statement of what the CUDA library computes (Algorithm 1 of the paper with
the operators of Eq. 1 / Eq. 2 and Table 1 restricted to copy / scalar multiply and sum / mean,
plus the transpose and backward pass the paper leaves implicit).

All arrays are NumPy arrays on the host.  Inputs keep the storage types of the library's ABI
(int64 row pointers, int32 indices, fp32 features and weights); every accumulation is fp64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

OP_SUM = 0
OP_MEAN = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ap_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libap_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``ap_oracle.c`` with gcc into ``libap_oracle.so`` next to it."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", _LIB_PATH, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB_PATH)
        p = ctypes.c_void_p
        i64, i32 = ctypes.c_int64, ctypes.c_int32
        lib.oracle_ap_forward.argtypes = [i64, p, p, p, p, i32, ctypes.c_int, ctypes.c_int, p, i64,
                                          p, p]
        lib.oracle_ap_forward.restype = ctypes.c_int
        lib.oracle_transpose.argtypes = [i64, i64, p, p, p, p, p, p, p]
        lib.oracle_transpose.restype = ctypes.c_int
        lib.oracle_ap_backward.argtypes = [i64, p, p, p, p, p, i32, ctypes.c_int, ctypes.c_int, p,
                                           i64, p, p]
        lib.oracle_ap_backward.restype = ctypes.c_int
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the parallel loop over destination vertices will use."""
    return int(_load().oracle_num_threads())


def set_num_threads(t: int) -> None:
    _load().oracle_set_num_threads(int(t))


def _arr(a, dtype, name):
    if a is None:
        return None
    a = np.asarray(a)
    if a.dtype != dtype:
        raise TypeError(f"{name}: expected {np.dtype(dtype)}, got {a.dtype}")
    return np.ascontiguousarray(a)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def ap_forward(rowptr, colidx, edge_w, H, op, rows=None, self_loops=False):
    """Forward AP of Algorithm 1.  Returns ``(ref, mag)``: fp64 arrays of shape (rows, F).

    ``ref[v] = s_v * sum_k w_k H[colidx[k]]`` over the CSR row of ``v``; ``mag`` is the same
    sum over absolute values, the quantity the fp32 error bound is stated against.
    ``rows`` selects destination vertices (all when None).  ``self_loops`` adds ``H[v]`` to the
    sum and 1 to the mean's divisor (the GCN aggregator of Section 5.1).
    """
    rowptr = _arr(rowptr, np.int64, "rowptr")
    colidx = _arr(colidx, np.int32, "colidx")
    edge_w = _arr(edge_w, np.float32, "edge_w")
    H = _arr(H, np.float32, "H")
    n = rowptr.shape[0] - 1
    if H.ndim != 2 or H.shape[0] != n:
        raise ValueError("H must be (n, F)")
    F = H.shape[1]
    rows_a = None if rows is None else _arr(np.asarray(rows, dtype=np.int64), np.int64, "rows")
    count = n if rows_a is None else rows_a.shape[0]
    ref = np.empty((count, F), dtype=np.float64)
    mag = np.empty((count, F), dtype=np.float64)
    rc = _load().oracle_ap_forward(n, _ptr(rowptr), _ptr(colidx), _ptr(edge_w), _ptr(H), F,
                                   int(op), int(bool(self_loops)), _ptr(rows_a), count,
                                   _ptr(ref), _ptr(mag))
    if rc != 0:
        raise ValueError(f"oracle_ap_forward: invalid argument (code {rc})")
    return ref, mag


def transpose(rowptr, colidx, edge_w=None):
    """Stable counting sort of the edges by source vertex.

    Returns ``(colptr int64[n+1], rowidx_T int32[nnz], w_T fp32[nnz] | None, perm int64[nnz])``.
    """
    rowptr = _arr(rowptr, np.int64, "rowptr")
    colidx = _arr(colidx, np.int32, "colidx")
    edge_w = _arr(edge_w, np.float32, "edge_w")
    n = rowptr.shape[0] - 1
    nnz = colidx.shape[0]
    if int(rowptr[n]) != nnz or int(rowptr[0]) != 0:
        raise ValueError("rowptr does not describe colidx")
    colptr = np.empty(n + 1, dtype=np.int64)
    rowidx_T = np.empty(nnz, dtype=np.int32)
    perm = np.empty(nnz, dtype=np.int64)
    w_T = None if edge_w is None else np.empty(nnz, dtype=np.float32)
    rc = _load().oracle_transpose(n, nnz, _ptr(rowptr), _ptr(colidx), _ptr(edge_w),
                                  _ptr(colptr), _ptr(rowidx_T), _ptr(w_T), _ptr(perm))
    if rc != 0:
        raise ValueError(f"oracle_transpose failed (code {rc})")
    return colptr, rowidx_T, w_T, perm


def ap_backward(rowptr, colptr, rowidx_T, w_T, dOut, op, cols=None, self_loops=False):
    """Backward AP ``dH = A^T dOut`` over the CSC.  Returns ``(ref, mag)`` like ap_forward.

    ``rowptr`` is the CSR row pointer: the mean's divisor is the in-degree of the destination
    (plus 1 with ``self_loops``, which also adds the vertex's own ``dOut`` row, scaled alike).
    """
    rowptr = _arr(rowptr, np.int64, "rowptr")
    colptr = _arr(colptr, np.int64, "colptr")
    rowidx_T = _arr(rowidx_T, np.int32, "rowidx_T")
    w_T = _arr(w_T, np.float32, "w_T")
    dOut = _arr(dOut, np.float32, "dOut")
    n = rowptr.shape[0] - 1
    if dOut.ndim != 2 or dOut.shape[0] != n:
        raise ValueError("dOut must be (n, F)")
    F = dOut.shape[1]
    cols_a = None if cols is None else _arr(np.asarray(cols, dtype=np.int64), np.int64, "cols")
    count = n if cols_a is None else cols_a.shape[0]
    ref = np.empty((count, F), dtype=np.float64)
    mag = np.empty((count, F), dtype=np.float64)
    rc = _load().oracle_ap_backward(n, _ptr(rowptr), _ptr(colptr), _ptr(rowidx_T), _ptr(w_T),
                                    _ptr(dOut), F, int(op), int(bool(self_loops)),
                                    _ptr(cols_a), count, _ptr(ref), _ptr(mag))
    if rc != 0:
        raise ValueError(f"oracle_ap_backward: invalid argument (code {rc})")
    return ref, mag


def error_bound(mag):
    """Per-element fp32 tolerance: 1e-5 * sum|terms| + 1e-7."""
    return 1e-5 * mag + 1e-7
