"""ctypes binding of libdgagg.so: argument marshalling only.

Every function here has the name and the meaning of the C entry point it forwards to
(``include/dg.h``); torch tensors are passed as raw device pointers and the current torch
stream as the stream handle.  Nothing is computed in Python, and there is no fallback: if the
shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

DG_OK = 0
DG_ERR_INVALID_ARG = 1
DG_ERR_UNSUPPORTED = 2
DG_ERR_CUDA = 3
DG_ERR_NOT_TRANSPOSED = 4
DG_ERR_WORKSPACE = 5
DG_ERR_INVALID_GRAPH = 6
DG_OP_SUM = 0
DG_OP_MEAN = 1
DG_BIN_COPY_LHS, DG_BIN_COPY_RHS, DG_BIN_ADD, DG_BIN_SUB, DG_BIN_MUL, DG_BIN_DIV = range(6)
DG_RED_SUM, DG_RED_MAX, DG_RED_MIN = range(3)
DG_ORDER_GIVEN, DG_ORDER_OUT_DEGREE, DG_ORDER_IN_DEGREE = range(3)

EXPORTS = [
    "dg_graph_create", "dg_graph_destroy", "dg_graph_validate", "dg_graph_transpose_workspace",
    "dg_graph_transpose", "dg_graph_transpose_static", "dg_graph_update_weights", "dg_graph_get_csc", "dg_aggregate_fwd", "dg_aggregate_bwd",
    "dg_aggregate_fwd_bf16", "dg_aggregate_bwd_bf16",
    "dg_ap_fwd", "dg_ap_bwd", "dg_aggregate_edge_grad",
    "dg_graph_reorder_workspace", "dg_graph_reorder", "dg_graph_get_order", "dg_permute_rows",
    "dg_aggregate_host_workspace", "dg_aggregate_host", "dg_graph_set_param",
    "dg_graph_get_param", "dg_probe_gather", "dg_probe_gather_smem", "dg_kernel_launch_count", "dg_last_error", "dg_version",
]

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdgagg.so")
_lib = None


class DgError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"libdgagg status {status}: {message}")
        self.status = status


def lib() -> ctypes.CDLL:
    """The loaded shared library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2104_06700_b200.build`; "
                "there is no CPU or PyTorch fallback for the aggregation kernels")
        L = ctypes.CDLL(LIB_PATH)
        p, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
        pp = ctypes.POINTER(ctypes.c_void_p)
        L.dg_graph_create.argtypes = [i64, i64, p, p, p, pp]
        L.dg_graph_destroy.argtypes = [p]
        L.dg_graph_validate.argtypes = [p, p]
        L.dg_graph_transpose_workspace.argtypes = [p, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.dg_graph_transpose.argtypes = [p, p, sz, p, sz, p]
        L.dg_graph_transpose_static.argtypes = [p, p, sz, p]
        L.dg_graph_update_weights.argtypes = [p, p]
        L.dg_graph_get_csc.argtypes = [p, pp, pp, pp, pp]
        L.dg_aggregate_fwd.argtypes = [p, p, i32, ctypes.c_int, p, p]
        L.dg_aggregate_bwd.argtypes = [p, p, i32, ctypes.c_int, p, p]
        L.dg_aggregate_fwd_bf16.argtypes = [p, p, i32, ctypes.c_int, p, p]
        L.dg_aggregate_bwd_bf16.argtypes = [p, p, i32, ctypes.c_int, p, p]
        L.dg_ap_fwd.argtypes = [p, p, p, i32, i32, ctypes.c_int, ctypes.c_int, p, p, p]
        L.dg_ap_bwd.argtypes = [p, p, p, p, i32, i32, ctypes.c_int, ctypes.c_int, p, p, p, p]
        L.dg_aggregate_edge_grad.argtypes = [p, p, p, i32, ctypes.c_int, p, p]
        L.dg_graph_reorder_workspace.argtypes = [p, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.dg_graph_reorder.argtypes = [p, ctypes.c_int, p, p, sz, p, sz, p, pp]
        L.dg_graph_get_order.argtypes = [p, pp, pp, pp, pp, pp]
        L.dg_permute_rows.argtypes = [p, i64, i32, p, p, ctypes.c_int, p]
        L.dg_aggregate_host_workspace.argtypes = [p, i32]
        L.dg_aggregate_host_workspace.restype = sz
        L.dg_aggregate_host.argtypes = [p, p, p, i32, ctypes.c_int, p, p, p, sz, p]
        L.dg_graph_set_param.argtypes = [p, ctypes.c_char_p, i64]
        L.dg_graph_get_param.argtypes = [p, ctypes.c_char_p, ctypes.POINTER(i64)]
        L.dg_probe_gather.argtypes = [p, i64, i32, p, i64, p, p]
        L.dg_probe_gather_smem.argtypes = [i32, i32, p, i64, p, i32, p]
        L.dg_kernel_launch_count.restype = i64
        L.dg_last_error.restype = ctypes.c_char_p
        L.dg_version.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ("dg_aggregate_host_workspace", "dg_kernel_launch_count",
                            "dg_last_error", "dg_version"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(status: int) -> None:
    if status != DG_OK:
        raise DgError(status, lib().dg_last_error().decode())


def _dev_ptr(t: Optional[torch.Tensor], dtype, name: str):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def dg_version() -> str:
    return lib().dg_version().decode()


def dg_last_error() -> str:
    return lib().dg_last_error().decode()


def dg_kernel_launch_count() -> int:
    return int(lib().dg_kernel_launch_count())


def dg_probe_gather(table: torch.Tensor, idx: torch.Tensor, sink: torch.Tensor, stream=None) -> None:
    """Wraps ``dg_probe_gather``: table (rows, row_floats) fp32, idx int32, sink fp32."""
    _check(lib().dg_probe_gather(_dev_ptr(table, torch.float32, "table"), table.shape[0],
                                 table.shape[1], _dev_ptr(idx, torch.int32, "idx"), idx.numel(),
                                 _dev_ptr(sink, torch.float32, "sink"), _stream(stream)))


def dg_probe_gather_smem(row_floats: int, stage_rows: int, idx: torch.Tensor, sink: torch.Tensor,
                         remote: bool = False, stream=None) -> None:
    """Wraps ``dg_probe_gather_smem``: idx int32 in [0, stage_rows), sink fp32."""
    _check(lib().dg_probe_gather_smem(int(row_floats), int(stage_rows),
                                      _dev_ptr(idx, torch.int32, "idx"), idx.numel(),
                                      _dev_ptr(sink, torch.float32, "sink"), int(bool(remote)),
                                      _stream(stream)))


def dg_graph_create(n: int, nnz: int, rowptr: torch.Tensor, colidx: torch.Tensor,
                    edge_w: Optional[torch.Tensor]) -> "Graph":
    """Wraps ``dg_graph_create``; the returned object keeps the borrowed tensors alive."""
    return Graph(n, nnz, rowptr, colidx, edge_w)


def dg_permute_rows(new_of_old: torch.Tensor, x: torch.Tensor, to_old: bool = False,
                    out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Wraps ``dg_permute_rows``: out[new_of_old[v]] = x[v], or out[v] = x[new_of_old[v]]."""
    if out is None:
        out = torch.empty_like(x)
    _check(lib().dg_permute_rows(_dev_ptr(new_of_old, torch.int32, "new_of_old"), x.shape[0],
                                 x.shape[1], _dev_ptr(x, torch.float32, "x"),
                                 _dev_ptr(out, torch.float32, "out"), int(bool(to_old)),
                                 _stream(stream)))
    return out


class Graph:
    """Owner of one ``dg_graph_t`` and of the torch buffers the handle borrows."""

    def __init__(self, n, nnz, rowptr, colidx, edge_w, _adopt=None):
        self._h = ctypes.c_void_p()
        self.n, self.nnz = int(n), int(nnz)
        self.rowptr, self.colidx, self.edge_w = rowptr, colidx, edge_w
        self._csc = None
        self._storage = None
        if _adopt is not None:          # a handle the library made (dg_graph_reorder)
            self._h, self._storage = _adopt
            return
        with torch.cuda.device(rowptr.device):
            _check(lib().dg_graph_create(
                self.n, self.nnz, _dev_ptr(rowptr, torch.int64, "rowptr"),
                _dev_ptr(colidx, torch.int32, "colidx"),
                _dev_ptr(edge_w, torch.float32, "edge_w"), ctypes.byref(self._h)))

    @property
    def device(self):
        return self.rowptr.device

    def dg_graph_destroy(self) -> None:
        if self._h:
            lib().dg_graph_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.dg_graph_destroy()
        except Exception:
            pass

    def dg_graph_validate(self, stream=None) -> None:
        _check(lib().dg_graph_validate(self._h, _stream(stream)))

    def dg_graph_transpose_workspace(self):
        a, b = ctypes.c_size_t(), ctypes.c_size_t()
        _check(lib().dg_graph_transpose_workspace(self._h, ctypes.byref(a), ctypes.byref(b)))
        return int(a.value), int(b.value)

    def dg_graph_transpose(self, csc_storage: Optional[torch.Tensor] = None,
                           scratch: Optional[torch.Tensor] = None, stream=None) -> None:
        """Builds the CSC.  Buffers are torch uint8 tensors; they are allocated here when not
        given (the scratch is released when the call returns, the stream keeps ordering)."""
        need_csc, need_scratch = self.dg_graph_transpose_workspace()
        if csc_storage is None:
            csc_storage = torch.empty(need_csc, dtype=torch.uint8, device=self.device)
        if scratch is None:
            scratch = torch.empty(need_scratch, dtype=torch.uint8, device=self.device)
        _check(lib().dg_graph_transpose(
            self._h, ctypes.c_void_p(csc_storage.data_ptr()), csc_storage.numel(),
            ctypes.c_void_p(scratch.data_ptr()), scratch.numel(), _stream(stream)))
        self._csc = csc_storage
        scratch.record_stream(torch.cuda.current_stream() if stream is None else stream)

    def dg_graph_transpose_static(self, csc_storage: Optional[torch.Tensor] = None,
                                  stream=None) -> None:
        """Builds the CSC with the scratch that is built into the library (small graphs only;
        larger ones raise DgError with status DG_ERR_UNSUPPORTED).  Only the output storage is
        a torch tensor; the call itself allocates nothing when that tensor is passed in."""
        need_csc, _ = self.dg_graph_transpose_workspace()
        if csc_storage is None:
            csc_storage = torch.empty(need_csc, dtype=torch.uint8, device=self.device)
        _check(lib().dg_graph_transpose_static(
            self._h, ctypes.c_void_p(csc_storage.data_ptr()), csc_storage.numel(),
            _stream(stream)))
        self._csc = csc_storage

    def dg_graph_update_weights(self, stream=None) -> None:
        _check(lib().dg_graph_update_weights(self._h, _stream(stream)))

    def dg_graph_reorder_workspace(self):
        a, b = ctypes.c_size_t(), ctypes.c_size_t()
        _check(lib().dg_graph_reorder_workspace(self._h, ctypes.byref(a), ctypes.byref(b)))
        return int(a.value), int(b.value)

    def dg_graph_reorder(self, order: int, given_new_of_old: Optional[torch.Tensor] = None,
                         stream=None) -> "Graph":
        """Returns a new Graph over the renamed CSR (its arrays are views into a storage tensor
        the new object keeps alive); ``new.new_of_old`` and ``new.pos`` give the permutations."""
        need_storage, need_scratch = self.dg_graph_reorder_workspace()
        storage = torch.empty(need_storage, dtype=torch.uint8, device=self.device)
        scratch = torch.empty(need_scratch, dtype=torch.uint8, device=self.device)
        h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib().dg_graph_reorder(
                self._h, int(order), _dev_ptr(given_new_of_old, torch.int32, "given_new_of_old"),
                ctypes.c_void_p(storage.data_ptr()), storage.numel(),
                ctypes.c_void_p(scratch.data_ptr()), scratch.numel(), _stream(stream),
                ctypes.byref(h)))
        ptrs = [ctypes.c_void_p() for _ in range(5)]
        _check(lib().dg_graph_get_order(h, *[ctypes.byref(p) for p in ptrs]))
        base = storage.data_ptr()

        def view(p, dtype, count):
            if not p.value:
                return None
            off = p.value - base
            size = torch.empty(0, dtype=dtype).element_size() * count
            return storage[off:off + size].view(dtype)

        new = Graph(self.n, self.nnz, view(ptrs[1], torch.int64, self.n + 1),
                    view(ptrs[2], torch.int32, self.nnz), view(ptrs[3], torch.float32, self.nnz),
                    _adopt=(h, storage))
        new.new_of_old = view(ptrs[0], torch.int32, self.n)
        new.pos = view(ptrs[4], torch.int32, self.nnz)
        return new

    def dg_graph_get_csc(self):
        """(colptr int64[n+1], rowidx_T int32[nnz], w_T fp32[nnz] | None, perm int32[nnz]) as
        torch views into the CSC storage."""
        ptrs = [ctypes.c_void_p() for _ in range(4)]
        _check(lib().dg_graph_get_csc(self._h, *[ctypes.byref(p) for p in ptrs]))
        base = self._csc.data_ptr()

        def view(p, dtype, count):
            if not p.value:
                return None
            off = p.value - base
            size = torch.empty(0, dtype=dtype).element_size() * count
            return self._csc[off:off + size].view(dtype)

        return (view(ptrs[0], torch.int64, self.n + 1), view(ptrs[1], torch.int32, self.nnz),
                view(ptrs[2], torch.float32, self.nnz), view(ptrs[3], torch.int32, self.nnz))

    def dg_aggregate_fwd(self, H: torch.Tensor, op: int, out: Optional[torch.Tensor] = None,
                         stream=None) -> torch.Tensor:
        F = H.shape[1]
        if out is None:
            out = torch.empty_like(H)
        _check(lib().dg_aggregate_fwd(self._h, _dev_ptr(H, torch.float32, "H"), F, int(op),
                                      _dev_ptr(out, torch.float32, "out"), _stream(stream)))
        return out

    def dg_aggregate_bwd(self, dOut: torch.Tensor, op: int, dH: Optional[torch.Tensor] = None,
                         stream=None) -> torch.Tensor:
        F = dOut.shape[1]
        if dH is None:
            dH = torch.empty_like(dOut)
        _check(lib().dg_aggregate_bwd(self._h, _dev_ptr(dOut, torch.float32, "dOut"), F, int(op),
                                      _dev_ptr(dH, torch.float32, "dH"), _stream(stream)))
        return dH

    def dg_aggregate_fwd_bf16(self, H: torch.Tensor, op: int, out: Optional[torch.Tensor] = None,
                              stream=None) -> torch.Tensor:
        """H is a torch.bfloat16 matrix; the result is fp32."""
        F = H.shape[1]
        if out is None:
            out = torch.empty(H.shape, dtype=torch.float32, device=H.device)
        _check(lib().dg_aggregate_fwd_bf16(self._h, _dev_ptr(H, torch.bfloat16, "H"), F, int(op),
                                           _dev_ptr(out, torch.float32, "out"), _stream(stream)))
        return out

    def dg_aggregate_bwd_bf16(self, dOut: torch.Tensor, op: int,
                              dH: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        F = dOut.shape[1]
        if dH is None:
            dH = torch.empty(dOut.shape, dtype=torch.float32, device=dOut.device)
        _check(lib().dg_aggregate_bwd_bf16(self._h, _dev_ptr(dOut, torch.bfloat16, "dOut"), F,
                                           int(op), _dev_ptr(dH, torch.float32, "dH"),
                                           _stream(stream)))
        return dH

    def _edge_cols(self, fE, F):
        if fE is None:
            return 1
        if fE.dim() != 2 or fE.shape[0] != self.nnz or fE.shape[1] not in (1, F):
            raise ValueError("fE must be (nnz, F) or (nnz, 1)")
        return fE.shape[1]

    def dg_ap_fwd(self, fV: Optional[torch.Tensor], fE: Optional[torch.Tensor], binary: int,
                  reduce: int, F: Optional[int] = None, fO: Optional[torch.Tensor] = None,
                  want_arg: bool = True, arg: Optional[torch.Tensor] = None, stream=None):
        """General AP.  Returns (fO, arg); arg is an int32 (n, F) tensor for max / min when
        ``want_arg`` (allocated here unless given), else None."""
        if F is None:
            F = fV.shape[1] if fV is not None else fE.shape[1]
        cols = self._edge_cols(fE, F)
        if fO is None:
            fO = torch.empty((self.n, F), dtype=torch.float32, device=self.device)
        if reduce == DG_RED_SUM or not want_arg:
            arg = None
        elif arg is None:
            arg = torch.empty((self.n, F), dtype=torch.int32, device=self.device)
        _check(lib().dg_ap_fwd(self._h, _dev_ptr(fV, torch.float32, "fV"),
                               _dev_ptr(fE, torch.float32, "fE"), cols, F, int(binary), int(reduce),
                               _dev_ptr(fO, torch.float32, "fO"), _dev_ptr(arg, torch.int32, "arg"),
                               _stream(stream)))
        return fO, arg

    def dg_ap_bwd(self, dO: torch.Tensor, fV: Optional[torch.Tensor], fE: Optional[torch.Tensor],
                  binary: int, reduce: int, arg: Optional[torch.Tensor] = None, want_dV: bool = True,
                  want_dE: bool = True, stream=None):
        """Gradients of the general AP.  Returns (dV | None, dE | None)."""
        F = dO.shape[1]
        cols = self._edge_cols(fE, F)
        dV = torch.empty((self.n, F), dtype=torch.float32, device=self.device) if want_dV else None
        dE = None
        if want_dE and binary != DG_BIN_COPY_LHS:
            dE = torch.empty((self.nnz, cols), dtype=torch.float32, device=self.device)
        _check(lib().dg_ap_bwd(self._h, _dev_ptr(dO, torch.float32, "dO"),
                               _dev_ptr(fV, torch.float32, "fV"), _dev_ptr(fE, torch.float32, "fE"),
                               cols, F, int(binary), int(reduce), _dev_ptr(arg, torch.int32, "arg"),
                               _dev_ptr(dV, torch.float32, "dV"), _dev_ptr(dE, torch.float32, "dE"),
                               _stream(stream)))
        return dV, dE

    def dg_aggregate_edge_grad(self, H: torch.Tensor, dOut: torch.Tensor, op: int,
                               dW: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        F = H.shape[1]
        if dOut.shape != H.shape:
            raise ValueError("H and dOut must have the same shape")
        if dW is None:
            dW = torch.empty(self.nnz, dtype=torch.float32, device=self.device)
        _check(lib().dg_aggregate_edge_grad(self._h, _dev_ptr(H, torch.float32, "H"),
                                            _dev_ptr(dOut, torch.float32, "dOut"), F, int(op),
                                            _dev_ptr(dW, torch.float32, "dW"), _stream(stream)))
        return dW

    def dg_aggregate_host_workspace(self, F: int) -> int:
        return int(lib().dg_aggregate_host_workspace(self._h, int(F)))

    def dg_aggregate_host(self, H_host: torch.Tensor, dOut_host: Optional[torch.Tensor], op: int,
                          out_host: torch.Tensor, dH_host: Optional[torch.Tensor],
                          device_ws: torch.Tensor, stream=None) -> None:
        """Host-memory (ideally pinned) feature matrices in, host results out; the copies and
        both kernels are enqueued by the library on the stream."""
        for t in (H_host, dOut_host, out_host, dH_host):
            if t is not None and (t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous()):
                raise ValueError("host matrices must be contiguous fp32 CPU tensors")
        hp = lambda t: None if t is None else ctypes.c_void_p(t.data_ptr())
        _check(lib().dg_aggregate_host(
            self._h, hp(H_host), hp(dOut_host), H_host.shape[1], int(op), hp(out_host),
            hp(dH_host), ctypes.c_void_p(device_ws.data_ptr()), device_ws.numel(),
            _stream(stream)))

    def dg_graph_set_param(self, name: str, value: int) -> None:
        _check(lib().dg_graph_set_param(self._h, name.encode(), int(value)))

    def dg_graph_get_param(self, name: str) -> int:
        v = ctypes.c_int64()
        _check(lib().dg_graph_get_param(self._h, name.encode(), ctypes.byref(v)))
        return int(v.value)
