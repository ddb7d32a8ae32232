"""GPU parity of dg_graph_reorder (vertex renaming as pre-processing) against the CPU oracle.

Integer work with one correct answer: the order (hub-first by out- or in-degree, or the caller's
permutation), the renamed CSR with its rows sorted by new source id, the position map and the
copied weights are all compared bit for bit.  On top of that the property the step exists for:
aggregating the renamed features on the renamed graph and renaming back equals aggregating on
the original graph (checked against the oracle of the ORIGINAL graph).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_06700_b200 import binding, synth
from parity_util import assert_within_bound, make_graph, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"
ORDERS = [binding.DG_ORDER_OUT_DEGREE, binding.DG_ORDER_IN_DEGREE, binding.DG_ORDER_GIVEN]


def expected_order(rp, ci, order, given):
    n = len(rp) - 1
    if order == binding.DG_ORDER_GIVEN:
        return given
    deg = np.bincount(ci, minlength=n) if order == binding.DG_ORDER_OUT_DEGREE else np.diff(rp)
    return oracle.order_by_degree(deg.astype(np.int64))


def check_reorder(sg, order, seed=0, features=(64,), ops=(binding.DG_OP_MEAN,)):
    g = make_graph(sg)
    rp, ci, w = to_np(sg.rowptr), to_np(sg.colidx), to_np(sg.edge_w)
    given = None
    if order == binding.DG_ORDER_GIVEN:
        given = np.random.default_rng(seed).permutation(sg.n).astype(np.int32)
    r = g.dg_graph_reorder(order, None if given is None else torch.as_tensor(given, device=DEV))
    torch.cuda.synchronize()
    want_order = expected_order(rp, ci, order, given)
    assert np.array_equal(to_np(r.new_of_old), want_order), "new_of_old"
    rp2, ci2, w2, pos2 = oracle.relabel(rp, ci, w, want_order)
    assert np.array_equal(to_np(r.rowptr), rp2), "rowptr"
    assert np.array_equal(to_np(r.colidx), ci2), "colidx"
    assert np.array_equal(to_np(r.pos).astype(np.int64), pos2), "pos"
    if w is None:
        assert r.edge_w is None
    else:
        assert to_np(r.edge_w).tobytes() == w2.tobytes(), "edge_w"
    # the renamed graph is a graph like any other: validate, transpose, aggregate
    r.dg_graph_validate()
    r.dg_graph_transpose()
    colptr, rowidx_T, w_T, _ = oracle.transpose(rp, ci, w)
    for F in features:
        H = synth.features(sg.n, F, 40 + F, DEV)
        G = synth.features(sg.n, F, 41 + F, DEV)
        H2 = binding.dg_permute_rows(r.new_of_old, H)
        G2 = binding.dg_permute_rows(r.new_of_old, G)
        assert torch.equal(H2[r.new_of_old.long()], H)
        for op in ops:
            out = binding.dg_permute_rows(r.new_of_old, r.dg_aggregate_fwd(H2, op), to_old=True)
            dH = binding.dg_permute_rows(r.new_of_old, r.dg_aggregate_bwd(G2, op), to_old=True)
            torch.cuda.synchronize()
            ref, mag = oracle.ap_forward(rp, ci, w, to_np(H), op)
            assert_within_bound(to_np(out), ref, mag, "fwd on the renamed graph")
            ref, mag = oracle.ap_backward(rp, colptr, rowidx_T, w_T, to_np(G), op)
            assert_within_bound(to_np(dH), ref, mag, "bwd on the renamed graph")
    return r


@pytest.mark.parametrize("order", ORDERS)
@pytest.mark.parametrize("weighted", [True, False])
def test_tiny(order, weighted):
    check_reorder(synth.make("tiny", weighted=weighted), order, features=(64, 10),
                  ops=(binding.DG_OP_SUM, binding.DG_OP_MEAN))


@pytest.mark.parametrize("name,scale,F", [("reddit_like", 0.02, 128), ("products_like", 0.02, 100),
                                          ("proteins_like", 0.02, 8), ("papers_like", 0.002, 128)])
@pytest.mark.parametrize("order", ORDERS)
def test_scaled_workloads(name, scale, F, order):
    check_reorder(synth.make(name, device=DEV, scale=scale), order, seed=3, features=(F,))


def test_unsorted_rows_duplicates_self_loops_and_empty_rows():
    rng = np.random.default_rng(5)
    n, nnz = 300, 5000
    dst = np.sort(rng.integers(0, n // 2, size=nnz))          # the upper half of the rows is empty
    src = rng.integers(0, n, size=nnz).astype(np.int32)        # unsorted inside rows, duplicates
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.add.at(rowptr, dst + 1, 1)
    rowptr = np.cumsum(rowptr)

    class SG:
        pass
    sg = SG()
    sg.n, sg.nnz = n, nnz
    sg.rowptr, sg.colidx = torch.as_tensor(rowptr), torch.as_tensor(src)
    sg.edge_w = torch.as_tensor(rng.uniform(0, 1, nnz).astype(np.float32))
    for order in ORDERS:
        check_reorder(sg, order, seed=9, features=(7,), ops=(binding.DG_OP_SUM,))


def test_identity_and_inverse_round_trip():
    sg = synth.make("tiny")
    g = make_graph(sg)
    ident = torch.arange(sg.n, dtype=torch.int32, device=DEV)
    r = g.dg_graph_reorder(binding.DG_ORDER_GIVEN, ident)
    assert torch.equal(r.rowptr.cpu(), sg.rowptr) and torch.equal(r.colidx.cpu(), sg.colidx)
    assert torch.equal(r.pos.cpu(), torch.arange(sg.nnz, dtype=torch.int32))
    p = torch.randperm(sg.n, device=DEV).to(torch.int32)
    inv = torch.empty_like(p)
    inv[p.long()] = torch.arange(sg.n, dtype=torch.int32, device=DEV)
    back = g.dg_graph_reorder(binding.DG_ORDER_GIVEN, p).dg_graph_reorder(binding.DG_ORDER_GIVEN, inv)
    assert torch.equal(back.rowptr.cpu(), sg.rowptr) and torch.equal(back.colidx.cpu(), sg.colidx)
    assert back.edge_w.cpu().numpy().tobytes() == sg.edge_w.numpy().tobytes()


def test_errors_and_empty_graph():
    sg = synth.make("tiny")
    g = make_graph(sg)
    not_perm = torch.zeros(sg.n, dtype=torch.int32, device=DEV)
    with pytest.raises(binding.DgError) as e:
        g.dg_graph_reorder(binding.DG_ORDER_GIVEN, not_perm)
    assert e.value.status == binding.DG_ERR_INVALID_ARG and "permutation" in str(e.value)
    out_of_range = torch.arange(sg.n, dtype=torch.int32, device=DEV)
    out_of_range[3] = sg.n
    with pytest.raises(binding.DgError) as e:
        g.dg_graph_reorder(binding.DG_ORDER_GIVEN, out_of_range)
    assert e.value.status == binding.DG_ERR_INVALID_ARG
    with pytest.raises(binding.DgError):
        g.dg_graph_reorder(binding.DG_ORDER_GIVEN, None)
    with pytest.raises(binding.DgError):
        g.dg_graph_reorder(7)
    g0 = binding.dg_graph_create(0, 0, torch.zeros(1, dtype=torch.int64, device=DEV),
                                 torch.zeros(0, dtype=torch.int32, device=DEV), None)
    r0 = g0.dg_graph_reorder(binding.DG_ORDER_OUT_DEGREE)
    assert r0.n == 0
    g1 = binding.dg_graph_create(5, 0, torch.zeros(6, dtype=torch.int64, device=DEV),
                                 torch.zeros(0, dtype=torch.int32, device=DEV), None)
    r1 = g1.dg_graph_reorder(binding.DG_ORDER_IN_DEGREE)
    assert r1.new_of_old.tolist() == [0, 1, 2, 3, 4] and r1.rowptr.tolist() == [0] * 6
    torch.cuda.synchronize()
