"""GPU parity where the fp32 error bound is tightest: non-negative inputs and very long rows.

Every layer of GraphSAGE after the first aggregates activations that went through a ReLU
(Section 5.1 of the paper: Models and Parameters), so all terms of a sum share one sign and the
rounding errors of a long fp32 chain no longer cancel against a zero-mean sum.  These cases
compare the CUDA library with the fp64 oracle under the same bound as everywhere else,
|gpu - ref| <= 1e-5 * sum|terms| + 1e-7 per element, on |N(0,1)| features: the tiny workload, the
scale-0.02 workloads in full, and a two-way star whose hub has more than two million in-edges
(forward: one row of that length) and as many out-edges (backward: one column of that length).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_06700_b200 import binding, synth
from parity_util import assert_within_bound, check_fwd_bwd, check_transpose, make_graph, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"


def host_csr(sg):
    return (to_np(sg.rowptr), to_np(sg.colidx), to_np(sg.edge_w))


@pytest.mark.parametrize("F", [8, 128, 602])
@pytest.mark.parametrize("weighted", [True, False])
def test_tiny_nonnegative_features(F, weighted):
    sg = synth.make("tiny", weighted=weighted)
    g = make_graph(sg)
    csc = check_transpose(g, *host_csr(sg))
    H = synth.features(sg.n, F, 300 + F, DEV, nonneg=True)
    G = synth.features(sg.n, F, 400 + F, DEV, nonneg=True)
    for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
        check_fwd_bwd(g, host_csr(sg), H, G, op, csc)


@pytest.mark.parametrize("name,scale,widths,ops", [
    ("reddit_like", 0.02, (602, 8), (binding.DG_OP_MEAN, binding.DG_OP_SUM)),
    ("products_like", 0.02, (100, 128), (binding.DG_OP_SUM, binding.DG_OP_MEAN)),
    ("proteins_like", 0.02, (8, 64, 256), (binding.DG_OP_SUM,)),
    ("papers_like", 0.002, (128,), (binding.DG_OP_SUM,)),
])
def test_scaled_workloads_nonnegative_features(name, scale, widths, ops):
    sg = synth.make(name, device=DEV, scale=scale)
    g = make_graph(sg)
    csc = check_transpose(g, *host_csr(sg))
    for F in widths:
        H = synth.features(sg.n, F, 33, DEV, nonneg=True)
        G = synth.features(sg.n, F, 34, DEV, nonneg=True)
        for op in ops:
            a, b = check_fwd_bwd(g, host_csr(sg), H, G, op, csc)
            assert a <= 1.0 and b <= 1.0


def two_way_star(leaves, weighted, device=DEV):
    """Vertex 0 receives an edge from each of `leaves` other vertices and sends one to each:
    CSR row 0 and CSC column 0 both hold `leaves` entries, every other row and column one."""
    n = leaves + 1
    rowptr = torch.empty(n + 1, dtype=torch.int64, device=device)
    rowptr[0] = 0
    rowptr[1:] = leaves + torch.arange(0, n, dtype=torch.int64, device=device)
    colidx = torch.zeros(2 * leaves, dtype=torch.int32, device=device)
    colidx[:leaves] = torch.arange(1, n, dtype=torch.int32, device=device)
    w = None
    if weighted:
        gen = torch.Generator(device=device)
        gen.manual_seed(5)
        w = torch.rand(2 * leaves, generator=gen, device=device, dtype=torch.float32)
    return n, rowptr, colidx, w


@pytest.mark.parametrize("F", [8, 128, 602])
@pytest.mark.parametrize("weighted", [False, True])
def test_star_with_two_million_edges_nonnegative(F, weighted):
    """One row (forward) and one column (backward) of 2,100,000 same-sign terms, sum and mean:
    the block-per-row path must keep its fp32 chains short whatever the row length."""
    leaves = 2_100_000
    n, rowptr, colidx, w = two_way_star(leaves, weighted)
    g = binding.dg_graph_create(n, 2 * leaves, rowptr, colidx, w)
    g.dg_graph_transpose()
    colptr, rowidx_T, w_T, _ = g.dg_graph_get_csc()
    assert int(colptr[1]) == leaves and int(rowptr[1]) == leaves
    H = synth.features(n, F, 51, DEV, nonneg=True)
    G = synth.features(n, F, 52, DEV, nonneg=True)
    rows = np.concatenate([[0], np.arange(1, n, 2999)])
    ridx = torch.as_tensor(rows, device=DEV)
    rp, ci, wh = to_np(rowptr), to_np(colidx), to_np(w)
    cp, rt, wt = to_np(colptr), to_np(rowidx_T), to_np(w_T)
    Hh, Gh = to_np(H), to_np(G)
    for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
        out = g.dg_aggregate_fwd(H, op)
        ref, mag = oracle.ap_forward(rp, ci, wh, Hh, op, rows=rows)
        worst = assert_within_bound(to_np(out[ridx]), ref, mag, "fwd star")
        assert worst <= 1.0
        del out
        dH = g.dg_aggregate_bwd(G, op)
        ref, mag = oracle.ap_backward(rp, cp, rt, wt, Gh, op, cols=rows)
        worst = assert_within_bound(to_np(dH[ridx]), ref, mag, "bwd star")
        assert worst <= 1.0
        del dH
