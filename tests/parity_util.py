"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the same
seeded inputs and compare element by element (fp32: |gpu - ref| <= 1e-5 * sum|terms| + 1e-7;
integers and copied weights: bit-exact)."""
import numpy as np
import torch

import oracle
from paper_2104_06700_b200 import binding

TOL_REL = 1e-5
TOL_ABS = 1e-7


def to_np(t):
    return None if t is None else t.detach().cpu().numpy()


def assert_within_bound(gpu, ref, mag, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    bound = TOL_REL * mag + TOL_ABS
    err = np.abs(gpu - ref)
    worst = float((err / bound).max()) if err.size else 0.0
    assert np.all(err <= bound), f"{what}: max |err|/bound = {worst:.3g}"
    return worst


def make_graph(sg, device="cuda"):
    rowptr, colidx = sg.rowptr.to(device), sg.colidx.to(device)
    w = None if sg.edge_w is None else sg.edge_w.to(device)
    return binding.dg_graph_create(sg.n, sg.nnz, rowptr, colidx, w)


def check_transpose(g, rowptr_h, colidx_h, w_h):
    """Full bit-exact comparison of the GPU CSC with the oracle's stable counting sort."""
    g.dg_graph_transpose()
    torch.cuda.synchronize()
    colptr, rowidx_T, w_T, perm = g.dg_graph_get_csc()
    o_colptr, o_rowidx, o_w, o_perm = oracle.transpose(rowptr_h, colidx_h, w_h)
    assert np.array_equal(to_np(colptr), o_colptr), "colptr"
    assert np.array_equal(to_np(perm).astype(np.int64), o_perm), "perm"
    assert np.array_equal(to_np(rowidx_T), o_rowidx), "rowidx_T"
    if w_h is None:
        assert w_T is None
    else:
        assert to_np(w_T).tobytes() == o_w.tobytes(), "w_T"
    return o_colptr, o_rowidx, o_w


def check_fwd_bwd(g, sg_host, H, G, op, csc_host, rows=None, self_loops=False):
    """Forward on H and backward on G against the oracle; rows=None compares every element.
    `self_loops` must be the handle's "self_loops" attribute (set before the transpose)."""
    rowptr_h, colidx_h, w_h = sg_host
    assert g.dg_graph_get_param("self_loops") == int(self_loops)
    o_colptr, o_rowidx, o_w = csc_host
    out = g.dg_aggregate_fwd(H, op)
    dH = g.dg_aggregate_bwd(G, op)
    torch.cuda.synchronize()
    Hh, Gh = to_np(H), to_np(G)
    if rows is None:
        ref, mag = oracle.ap_forward(rowptr_h, colidx_h, w_h, Hh, op, self_loops=self_loops)
        a = assert_within_bound(to_np(out), ref, mag, "fwd")
        ref, mag = oracle.ap_backward(rowptr_h, o_colptr, o_rowidx, o_w, Gh, op,
                                      self_loops=self_loops)
        b = assert_within_bound(to_np(dH), ref, mag, "bwd")
    else:
        idx = torch.as_tensor(rows, device=out.device)
        ref, mag = oracle.ap_forward(rowptr_h, colidx_h, w_h, Hh, op, rows=rows,
                                     self_loops=self_loops)
        a = assert_within_bound(to_np(out[idx]), ref, mag, "fwd (sampled rows)")
        ref, mag = oracle.ap_backward(rowptr_h, o_colptr, o_rowidx, o_w, Gh, op, cols=rows,
                                      self_loops=self_loops)
        b = assert_within_bound(to_np(dH[idx]), ref, mag, "bwd (sampled rows)")
    return a, b
