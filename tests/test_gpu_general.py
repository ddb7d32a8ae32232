"""GPU parity of the general aggregation primitive (every operator pair of Table 1 of the paper,
full or scalar edge features), of its gradients, and of the edge-weight gradient, against the
CPU oracle, element by element.

Bars: max / min outputs and their arg indices are bit-exact (both sides form the message as one
fp32 operation and resolve ties to the lowest edge position); sums are within
1e-5 * sum|terms| + 1e-7 per element, `sum|terms|` from the oracle.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2104_06700_b200 import binding, synth
from parity_util import assert_within_bound, make_graph, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"
BINARIES = list(range(6))
REDUCERS = list(range(3))
NAMES = {0: "copylhs", 1: "copyrhs", 2: "add", 3: "sub", 4: "mul", 5: "div"}


def edge_features(nnz, cols, seed, device=DEV):
    """U(0.5, 2) edge features: safe divisors."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    return torch.rand((nnz, cols), generator=gen, device=device, dtype=torch.float32) * 1.5 + 0.5


def run_case(sg, F, cols, binary, reduce, seed=0, tie_heavy=False, heavy_threshold=None,
             params=None, min_launches=0):
    g = make_graph(sg)
    g.dg_graph_transpose()
    if heavy_threshold is not None:
        g.dg_graph_set_param("heavy_threshold", heavy_threshold)
    for name, value in (params or {}).items():
        g.dg_graph_set_param(name, value)
    rp, ci = to_np(sg.rowptr), to_np(sg.colidx)
    X = synth.features(sg.n, F, 500 + seed, DEV)
    Y = edge_features(sg.nnz, cols, 600 + seed)
    if tie_heavy:      # few distinct values: many equal messages, so ties decide the arg
        X = torch.round(X)
        Y = torch.round(Y * 2) / 2 + 0.5
    G = synth.features(sg.n, F, 700 + seed, DEV)
    fV = None if binary == binding.DG_BIN_COPY_RHS else X
    fE = None if binary == binding.DG_BIN_COPY_LHS else Y
    before = binding.dg_kernel_launch_count()
    out, arg = g.dg_ap_fwd(fV, fE, binary, reduce, F=F)
    torch.cuda.synchronize()
    assert binding.dg_kernel_launch_count() - before >= min_launches
    ref, mag, oarg = oracle.general_forward(rp, ci, to_np(fV), to_np(fE), binary, reduce, F=F)
    if reduce == binding.DG_RED_SUM:
        assert arg is None
        assert_within_bound(to_np(out), ref, mag, f"fwd {NAMES[binary]}/sum")
    else:
        assert np.array_equal(to_np(out).astype(np.float64), ref), f"fwd {NAMES[binary]} max/min"
        assert np.array_equal(to_np(arg).astype(np.int64), oarg), "arg"
    before = binding.dg_kernel_launch_count()
    dV, dE = g.dg_ap_bwd(G, fV, fE, binary, reduce, arg=arg)
    torch.cuda.synchronize()
    if binary != binding.DG_BIN_COPY_RHS and "source_blocks" in (params or {}):
        assert binding.dg_kernel_launch_count() - before >= min_launches
    odV, omV, odE, omE = oracle.general_backward(rp, ci, to_np(fV), to_np(fE), binary, reduce,
                                                 oarg, to_np(G))
    assert_within_bound(to_np(dV), odV, omV, f"dV {NAMES[binary]}")
    if binary == binding.DG_BIN_COPY_LHS:
        assert dE is None
    else:
        assert_within_bound(to_np(dE), odE, omE, f"dE {NAMES[binary]}")


@pytest.fixture(scope="module")
def tiny():
    return synth.make("tiny")


@pytest.mark.parametrize("binary,reduce", list(itertools.product(BINARIES, REDUCERS)))
@pytest.mark.parametrize("cols_full", [True, False])
def test_every_operator_pair_on_tiny(tiny, binary, reduce, cols_full):
    F = 64
    run_case(tiny, F, F if cols_full else 1, binary, reduce, seed=binary * 3 + reduce)


@pytest.mark.parametrize("F", [1, 3, 8, 33, 100, 130])
@pytest.mark.parametrize("binary,reduce", [(4, 0), (2, 1), (5, 2), (0, 1), (1, 0)])
def test_feature_widths(tiny, F, binary, reduce):
    run_case(tiny, F, F, binary, reduce, seed=F)
    run_case(tiny, F, 1, binary, reduce, seed=F + 1)


@pytest.mark.parametrize("binary,reduce", [(0, 1), (0, 2), (2, 1), (4, 2), (1, 1)])
def test_ties_go_to_the_lowest_edge_position(tiny, binary, reduce):
    run_case(tiny, 16, 16, binary, reduce, seed=3, tie_heavy=True)
    run_case(tiny, 40, 1, binary, reduce, seed=4, tie_heavy=True)


@pytest.mark.parametrize("name,scale,F", [("reddit_like", 0.01, 48), ("products_like", 0.01, 100),
                                          ("papers_like", 0.001, 128)])
def test_scaled_workloads(name, scale, F):
    """Thousands of rows of very different lengths (heavy rows, empty rows), in full."""
    sg = synth.make(name, device=DEV, scale=scale)
    for binary, reduce, cols in ((4, 0, F), (4, 0, 1), (0, 1, 1), (3, 2, F), (5, 0, F)):
        run_case(sg, F, cols, binary, reduce, seed=binary + reduce)


@pytest.mark.parametrize("F,cols", [(64, 64), (100, 1), (7, 7), (260, 1)])
def test_heavy_rows_and_columns_take_the_block_kernels(F, cols):
    """With the lowest threshold most rows of the Reddit-like graph (and most columns of its
    transpose) are on the handle's heavy lists, so the leading blocks of the launch compute them:
    eight warps per row, merged in shared memory.  Sums within the bound, max / min and their
    arg bit-exact with ties (few distinct values) going to the lowest edge position."""
    sg = synth.make("reddit_like", device=DEV, scale=0.01)
    assert int((sg.rowptr[1:] - sg.rowptr[:-1]).max()) > 64 * 8   # rows of more than 8 batches
    for binary, reduce, ties in ((0, 0, False), (4, 0, False), (0, 1, True), (2, 2, True),
                                 (5, 0, False), (4, 1, False)):
        run_case(sg, F, cols, binary, reduce, seed=F + binary, tie_heavy=ties, heavy_threshold=64)


@pytest.mark.parametrize("params,launches", [({"source_blocks": 4}, 8), ({"l2_budget_mb": 12}, 4),
                                             ({"source_blocks": 16, "heavy_threshold": 64}, 32)])
def test_feature_slices_and_source_blocks(params, launches):
    """Cut into slices of 128 features and ranges of neighbour ids, one launch per piece, every
    launch folding its piece into the output of the earlier ones: the same sums within the bound,
    the same extrema and arg (bit-exact, ties to the lowest edge position) as in one launch."""
    sg = synth.make("reddit_like", device=DEV, scale=0.02)     # 32,946 vertices, 70 edges each
    F = 132                                                    # slices of 128 and 4
    for binary, reduce, cols, ties in ((4, 0, F, False), (0, 1, 1, True), (2, 2, F, True)):
        run_case(sg, F, cols, binary, reduce, seed=31 + binary, tie_heavy=ties, params=params,
                 min_launches=launches)


def test_extrema_without_arg_are_not_cut_into_source_blocks():
    """Folding a piece into the earlier ones needs the arg matrix; a caller that does not want it
    still gets the right extrema."""
    sg = synth.make("reddit_like", device=DEV, scale=0.02)
    g = make_graph(sg)
    g.dg_graph_set_param("source_blocks", 4)
    F = 130
    X = synth.features(sg.n, F, 77, DEV)
    out, arg = g.dg_ap_fwd(X, None, binding.DG_BIN_COPY_LHS, binding.DG_RED_MAX, want_arg=False)
    torch.cuda.synchronize()
    assert arg is None
    ref, _, _ = oracle.general_forward(to_np(sg.rowptr), to_np(sg.colidx), to_np(X), None,
                                       binding.DG_BIN_COPY_LHS, binding.DG_RED_MAX, F=F)
    assert np.array_equal(to_np(out).astype(np.float64), ref)


def test_empty_rows_and_empty_graph():
    rowptr = torch.tensor([0, 0, 2, 2, 3], dtype=torch.int64, device=DEV)
    colidx = torch.tensor([0, 3, 1], dtype=torch.int32, device=DEV)
    g = binding.dg_graph_create(4, 3, rowptr, colidx, None)
    X = -torch.ones((4, 5), device=DEV) - torch.arange(4, device=DEV)[:, None]
    out, arg = g.dg_ap_fwd(X, None, binding.DG_BIN_COPY_LHS, binding.DG_RED_MAX)
    torch.cuda.synchronize()
    assert out[0].tolist() == [0.0] * 5 and arg[0].tolist() == [-1] * 5
    assert out[1].tolist() == [-1.0] * 5 and arg[1].tolist() == [0] * 5   # not the initial zero
    assert out[3].tolist() == [-2.0] * 5 and arg[3].tolist() == [2] * 5
    g0 = binding.dg_graph_create(0, 0, torch.zeros(1, dtype=torch.int64, device=DEV),
                                 torch.zeros(0, dtype=torch.int32, device=DEV), None)
    g0.dg_ap_fwd(torch.zeros((0, 4), device=DEV), None, binding.DG_BIN_COPY_LHS, binding.DG_RED_SUM)
    torch.cuda.synchronize()


def test_argument_errors(tiny):
    g = make_graph(tiny)
    X = synth.features(tiny.n, 8, 1, DEV)
    Y = edge_features(tiny.nnz, 8, 2)
    with pytest.raises(binding.DgError) as e:
        g.dg_ap_fwd(None, Y, binding.DG_BIN_MUL, binding.DG_RED_SUM, F=8)
    assert e.value.status == binding.DG_ERR_INVALID_ARG
    with pytest.raises(binding.DgError) as e:
        g.dg_ap_fwd(X, None, binding.DG_BIN_ADD, binding.DG_RED_SUM)
    assert e.value.status == binding.DG_ERR_INVALID_ARG
    with pytest.raises(binding.DgError) as e:
        g.dg_ap_fwd(X, Y, 9, binding.DG_RED_SUM)
    assert e.value.status == binding.DG_ERR_INVALID_ARG
    with pytest.raises(binding.DgError) as e:                      # dV gathers over the CSC
        g.dg_ap_bwd(X, X, Y, binding.DG_BIN_MUL, binding.DG_RED_SUM)
    assert e.value.status == binding.DG_ERR_NOT_TRANSPOSED
    with pytest.raises(binding.DgError) as e:                      # max needs arg
        g.dg_ap_bwd(X, X, Y, binding.DG_BIN_MUL, binding.DG_RED_MAX, want_dV=False)
    assert e.value.status == binding.DG_ERR_INVALID_ARG
    torch.cuda.synchronize()


# ----------------------------------------------------------------------------- edge-weight gradient
@pytest.mark.parametrize("F", [64, 8, 100, 602, 3, 130])
@pytest.mark.parametrize("op", [binding.DG_OP_SUM, binding.DG_OP_MEAN])
def test_edge_weight_gradient_on_tiny(tiny, F, op):
    g = make_graph(tiny)
    H = synth.features(tiny.n, F, 11, DEV)
    G = synth.features(tiny.n, F, 12, DEV)
    dW = g.dg_aggregate_edge_grad(H, G, op)
    torch.cuda.synchronize()
    ref, mag = oracle.edge_weight_grad(to_np(tiny.rowptr), to_np(tiny.colidx), to_np(H), to_np(G), op)
    assert_within_bound(to_np(dW), ref, mag, "dW")


def test_edge_weight_gradient_with_self_loops_and_unaligned_rows(tiny):
    g = make_graph(tiny)
    g.dg_graph_set_param("self_loops", 1)
    F = 64
    base = synth.features(tiny.n * F + 4, 1, 13, DEV).flatten()
    H = base[1:1 + tiny.n * F].view(tiny.n, F)                     # 4 bytes off: scalar path
    G = synth.features(tiny.n, F, 14, DEV)
    dW = g.dg_aggregate_edge_grad(H, G, binding.DG_OP_MEAN)
    torch.cuda.synchronize()
    ref, mag = oracle.edge_weight_grad(to_np(tiny.rowptr), to_np(tiny.colidx),
                                       to_np(H.contiguous()), to_np(G), oracle.OP_MEAN,
                                       self_loops=True)
    assert_within_bound(to_np(dW), ref, mag, "dW, self loops")


@pytest.mark.parametrize("name,scale,F,op", [
    ("reddit_like", 0.02, 602, binding.DG_OP_MEAN),
    ("products_like", 0.02, 100, binding.DG_OP_SUM),
    ("proteins_like", 0.02, 8, binding.DG_OP_SUM),
    ("papers_like", 0.002, 128, binding.DG_OP_SUM),
])
def test_edge_weight_gradient_on_scaled_workloads(name, scale, F, op):
    sg = synth.make(name, device=DEV, scale=scale)
    g = make_graph(sg)
    H = synth.features(sg.n, F, 21, DEV)
    G = synth.features(sg.n, F, 22, DEV)
    dW = g.dg_aggregate_edge_grad(H, G, op)
    torch.cuda.synchronize()
    ref, mag = oracle.edge_weight_grad(to_np(sg.rowptr), to_np(sg.colidx), to_np(H), to_np(G), op)
    assert_within_bound(to_np(dW), ref, mag, "dW")


@pytest.mark.parametrize("op", [binding.DG_OP_SUM, binding.DG_OP_MEAN])
def test_edge_weight_gradient_in_feature_slices_and_source_blocks(op):
    """With a small L2 budget the call is cut into feature slices (which add up in dW) and source
    blocks (which partition the edges), one launch each: same result, same bound."""
    sg = synth.make("reddit_like", device=DEV, scale=0.05)     # 52,093 vertices, 110 edges each
    g = make_graph(sg)
    g.dg_graph_set_param("l2_budget_mb", 32)                    # 2 source blocks x 3 slices of 256
    F = 602
    H = synth.features(sg.n, F, 23, DEV)
    G = synth.features(sg.n, F, 24, DEV)
    before = binding.dg_kernel_launch_count()
    dW = g.dg_aggregate_edge_grad(H, G, op)
    torch.cuda.synchronize()
    assert binding.dg_kernel_launch_count() - before > 4          # really several passes
    ref, mag = oracle.edge_weight_grad(to_np(sg.rowptr), to_np(sg.colidx), to_np(H), to_np(G), op)
    assert_within_bound(to_np(dW), ref, mag, "dW, sliced and blocked")
