"""CPU oracle for the aggregation primitive: ctypes front end of ``ap_oracle.c``.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this package; it exists so
that the tests, the smoke check and the benchmark's CPU-baseline leg have an independent,
obviously correct statement of what the CUDA library computes: Algorithm 1 of the paper with
the operators of Eq. 1 / Eq. 2 and Table 1 (``ap_oracle.c``: copy / scalar multiply with sum /
mean, plus the transpose and backward pass the paper leaves implicit; ``ap_general_oracle.c``:
every operator pair of Table 1 with full edge features, their gradients, the gradient with
respect to scalar edge weights, and vertex relabelling).

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
# operators of Table 1 of the paper
BIN_COPY_LHS, BIN_COPY_RHS, BIN_ADD, BIN_SUB, BIN_MUL, BIN_DIV = range(6)
RED_SUM, RED_MAX, RED_MIN = range(3)

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, "ap_oracle.c"), os.path.join(_HERE, "ap_general_oracle.c")]
_LIB_PATH = os.path.join(_HERE, "libap_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle's C files with gcc into ``libap_oracle.so`` next to them."""
    if (not force and os.path.exists(_LIB_PATH)
            and all(os.path.getmtime(_LIB_PATH) >= os.path.getmtime(s) for s in _SRCS)):
        return _LIB_PATH
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-Wall",
           "-Wextra", "-o", _LIB_PATH, *_SRCS, "-lm"]
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
        lib.oracle_general_forward.argtypes = [i64, p, p, p, p, i32, i32, ctypes.c_int,
                                               ctypes.c_int, p, p, p]
        lib.oracle_general_forward.restype = ctypes.c_int
        lib.oracle_general_backward.argtypes = [i64, p, p, p, p, i32, i32, ctypes.c_int,
                                                ctypes.c_int, p, p, p, p, p, p]
        lib.oracle_general_backward.restype = ctypes.c_int
        lib.oracle_edge_weight_grad.argtypes = [i64, p, p, p, p, i32, ctypes.c_int, ctypes.c_int,
                                                p, p]
        lib.oracle_edge_weight_grad.restype = ctypes.c_int
        lib.oracle_order_by_degree.argtypes = [i64, p, p]
        lib.oracle_order_by_degree.restype = ctypes.c_int
        lib.oracle_relabel.argtypes = [i64, p, p, p, p, p, p, p, p]
        lib.oracle_relabel.restype = ctypes.c_int
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


def _edge_features(fE, nnz, F, name="fE"):
    if fE is None:
        return None, 1
    fE = _arr(fE, np.float32, name)
    if fE.ndim == 1:
        fE = fE.reshape(-1, 1)
    if fE.shape[0] != nnz or fE.shape[1] not in (1, F):
        raise ValueError(f"{name} must be (nnz, F) or (nnz, 1)")
    return fE, fE.shape[1]


def general_forward(rowptr, colidx, fV, fE, binary, reduce, F=None):
    """General AP of Eq. 1 / Eq. 2 with the operators of Table 1.

    ``out[v][j] = reduce over the CSR row of v of  binary(fV[colidx[k]][j], fE[k][j])``.
    ``fV`` is (n, F) or None (copyrhs); ``fE`` is (nnz, F), (nnz, 1) (broadcast) or None (copylhs).
    Returns ``(ref, mag, arg)``: fp64 (n, F) values, the sum of message magnitudes (sum) or
    |ref| (max/min), and for max/min the int64 (n, F) edge position of the extremum (lowest
    position among equals, -1 for an empty row; all -1 for sum).
    """
    rowptr = _arr(rowptr, np.int64, "rowptr")
    colidx = _arr(colidx, np.int32, "colidx")
    n, nnz = rowptr.shape[0] - 1, colidx.shape[0]
    fV = _arr(fV, np.float32, "fV")
    if fV is not None:
        F = fV.shape[1]
    elif F is None:
        F = np.asarray(fE).shape[1]
    fE, cols = _edge_features(fE, nnz, F)
    ref = np.empty((n, F), dtype=np.float64)
    mag = np.empty((n, F), dtype=np.float64)
    arg = np.empty((n, F), dtype=np.int64)
    rc = _load().oracle_general_forward(n, _ptr(rowptr), _ptr(colidx), _ptr(fV), _ptr(fE), cols, F,
                                        int(binary), int(reduce), _ptr(ref), _ptr(mag), _ptr(arg))
    if rc != 0:
        raise ValueError(f"oracle_general_forward: invalid argument (code {rc})")
    return ref, mag, arg


def general_backward(rowptr, colidx, fV, fE, binary, reduce, arg, dO, want_dV=True, want_dE=True):
    """Gradients of ``<general_forward(fV, fE), dO>`` with respect to fV and fE.

    Returns ``(dV, magV, dE, magE)``; a pair is None when not wanted (dE also for copylhs).
    ``arg`` is general_forward's third result (needed for max/min).
    """
    rowptr = _arr(rowptr, np.int64, "rowptr")
    colidx = _arr(colidx, np.int32, "colidx")
    n, nnz = rowptr.shape[0] - 1, colidx.shape[0]
    dO = _arr(dO, np.float32, "dO")
    F = dO.shape[1]
    fV = _arr(fV, np.float32, "fV")
    fE, cols = _edge_features(fE, nnz, F)
    arg = None if arg is None else _arr(arg, np.int64, "arg")
    want_dE = want_dE and binary != BIN_COPY_LHS
    dV = magV = dE = magE = None
    if want_dV:
        dV, magV = np.empty((n, F)), np.empty((n, F))
    if want_dE:
        dE, magE = np.empty((nnz, cols)), np.empty((nnz, cols))
    rc = _load().oracle_general_backward(n, _ptr(rowptr), _ptr(colidx), _ptr(fV), _ptr(fE), cols,
                                         F, int(binary), int(reduce), _ptr(arg), _ptr(dO),
                                         _ptr(dV), _ptr(magV), _ptr(dE), _ptr(magE))
    if rc != 0:
        raise ValueError(f"oracle_general_backward: invalid argument (code {rc})")
    return dV, magV, dE, magE


def edge_weight_grad(rowptr, colidx, H, dOut, op, self_loops=False):
    """``dW[k] = s_v <H[u_k], dOut[v_k]>`` for every CSR position k: the gradient of
    ``<ap_forward(H; w), dOut>`` with respect to the scalar edge weights.  Returns (dW, mag)."""
    rowptr = _arr(rowptr, np.int64, "rowptr")
    colidx = _arr(colidx, np.int32, "colidx")
    H = _arr(H, np.float32, "H")
    dOut = _arr(dOut, np.float32, "dOut")
    n, nnz, F = rowptr.shape[0] - 1, colidx.shape[0], H.shape[1]
    if H.shape != dOut.shape or H.shape[0] != n:
        raise ValueError("H and dOut must both be (n, F)")
    dW, mag = np.empty(nnz), np.empty(nnz)
    rc = _load().oracle_edge_weight_grad(n, _ptr(rowptr), _ptr(colidx), _ptr(H), _ptr(dOut), F,
                                         int(op), int(bool(self_loops)), _ptr(dW), _ptr(mag))
    if rc != 0:
        raise ValueError(f"oracle_edge_weight_grad: invalid argument (code {rc})")
    return dW, mag


def order_by_degree(degree):
    """new_of_old (int32) of the hub-first order: largest degree first, ties by ascending id."""
    degree = _arr(np.asarray(degree, dtype=np.int64), np.int64, "degree")
    out = np.empty(degree.shape[0], dtype=np.int32)
    rc = _load().oracle_order_by_degree(degree.shape[0], _ptr(degree), _ptr(out))
    if rc != 0:
        raise ValueError(f"oracle_order_by_degree failed (code {rc})")
    return out


def relabel(rowptr, colidx, edge_w, new_of_old):
    """The CSR of the graph with vertex v renamed new_of_old[v], rows sorted by new source id.

    Returns ``(rowptr2 int64, colidx2 int32, edge_w2 | None, pos2 int64)``; ``pos2[k']`` is the
    old CSR position of new position ``k'``.
    """
    rowptr = _arr(rowptr, np.int64, "rowptr")
    colidx = _arr(colidx, np.int32, "colidx")
    edge_w = _arr(edge_w, np.float32, "edge_w")
    new_of_old = _arr(new_of_old, np.int32, "new_of_old")
    n, nnz = rowptr.shape[0] - 1, colidx.shape[0]
    if new_of_old.shape[0] != n:
        raise ValueError("new_of_old must have n entries")
    rowptr2 = np.empty(n + 1, dtype=np.int64)
    colidx2 = np.empty(nnz, dtype=np.int32)
    pos2 = np.empty(nnz, dtype=np.int64)
    w2 = None if edge_w is None else np.empty(nnz, dtype=np.float32)
    rc = _load().oracle_relabel(n, _ptr(rowptr), _ptr(colidx), _ptr(edge_w), _ptr(new_of_old),
                                _ptr(rowptr2), _ptr(colidx2), _ptr(w2), _ptr(pos2))
    if rc != 0:
        raise ValueError(f"oracle_relabel failed (code {rc}): new_of_old must be a permutation")
    return rowptr2, colidx2, w2, pos2
