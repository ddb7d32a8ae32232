"""Pins of the second part of the CPU oracle (CPU only): the general aggregation primitive with
every operator pair of Table 1 of the paper, its gradients, the gradient with respect to scalar
edge weights, the hub-first order and vertex relabelling.

Nothing here re-types the oracle's loops.  The general AP is pinned by a dense evaluation built
from numpy masks (one (n, n, F) tensor of messages per graph, reduced with numpy's own sum / max /
min), by reductions to the already pinned weighted sum, and by algebraic identities; the
gradients by directional derivatives of <AP(X, Y), G> (exact where AP is linear or bilinear in
the perturbed operand, central differences elsewhere); the edge-weight gradient by linearity of
the weighted sum in w; the relabelling by P A P^T on dense matrices and by
AP(relabelled)(P H) = P AP(H); the degree order by numpy's lexsort.  The last test plants
mistakes and shows that the pins notice them.
"""
import itertools

import numpy as np
import pytest

import oracle
from oracle import (BIN_ADD, BIN_COPY_LHS, BIN_COPY_RHS, BIN_DIV, BIN_MUL, BIN_SUB, RED_MAX,
                    RED_MIN, RED_SUM)
from test_oracle_pins import csr_from_lists, random_csr

BINARIES = [BIN_COPY_LHS, BIN_COPY_RHS, BIN_ADD, BIN_SUB, BIN_MUL, BIN_DIV]
REDUCERS = [RED_SUM, RED_MAX, RED_MIN]
NP_BIN = {BIN_ADD: np.add, BIN_SUB: np.subtract, BIN_MUL: np.multiply, BIN_DIV: np.divide}


def make_inputs(rng, n, nnz, F, cols, positive_y=True, no_dup=True):
    rowptr, colidx = random_csr(rng, n, nnz, allow_dup=not no_dup)
    nnz = len(colidx)
    X = rng.standard_normal((n, F)).astype(np.float32)
    Y = rng.uniform(0.5, 2.0, size=(nnz, cols)).astype(np.float32)
    if not positive_y:
        Y = (Y * rng.choice([-1.0, 1.0], size=Y.shape)).astype(np.float32)
    return rowptr, colidx, X, Y


def dense_messages(rowptr, colidx, X, Y, binary, dtype, F):
    """M[v, u, j] = message of the edge u -> v (graphs without duplicate edges), mask[v, u]."""
    n = len(rowptr) - 1
    dst = np.repeat(np.arange(n), np.diff(rowptr))
    mask = np.zeros((n, n), dtype=bool)
    mask[dst, colidx] = True
    Yd = np.zeros((n, n, F), dtype=dtype)
    if Y is not None:
        Yd[dst, colidx, :] = np.broadcast_to(Y.astype(dtype), (len(colidx), F))
    Xd = np.zeros((n, n, F), dtype=dtype) if X is None else \
        np.broadcast_to(X.astype(dtype)[None, :, :], (n, n, F))
    if binary == BIN_COPY_LHS:
        M = Xd.copy()
    elif binary == BIN_COPY_RHS:
        M = Yd
    else:
        with np.errstate(divide="ignore", invalid="ignore"):
            M = NP_BIN[binary](Xd, Yd)
    return M, mask


# ----------------------------------------------------------------------------- forward
@pytest.mark.parametrize("binary,reduce", list(itertools.product(BINARIES, REDUCERS)))
@pytest.mark.parametrize("cols_full", [True, False])
def test_general_forward_equals_dense_masked_reduction(binary, reduce, cols_full):
    rng = np.random.default_rng(100 * binary + 10 * reduce + cols_full)
    n, F = 23, 5
    rowptr, colidx, X, Y = make_inputs(rng, n, 140, F, F if cols_full else 1,
                                       positive_y=(binary == BIN_DIV))
    fV = None if binary == BIN_COPY_RHS else X
    fE = None if binary == BIN_COPY_LHS else Y
    ref, mag, arg = oracle.general_forward(rowptr, colidx, fV, fE, binary, reduce, F=F)
    if reduce == RED_SUM:
        M, mask = dense_messages(rowptr, colidx, fV, fE, binary, np.float64, F)
        want = np.where(mask[:, :, None], M, 0.0).sum(axis=1)
        np.testing.assert_allclose(ref, want, rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(mag, np.where(mask[:, :, None], np.abs(M), 0.0).sum(axis=1),
                                   rtol=1e-13, atol=1e-13)
        assert np.all(arg == -1)
    else:
        M, mask = dense_messages(rowptr, colidx, fV, fE, binary, np.float32, F)   # fp32 messages
        fill = -np.inf if reduce == RED_MAX else np.inf
        Mm = np.where(mask[:, :, None], M, fill)
        want = Mm.max(axis=1) if reduce == RED_MAX else Mm.min(axis=1)
        empty = ~mask.any(axis=1)
        want[empty] = 0.0
        assert np.array_equal(ref, want.astype(np.float64))                    # exact
        # the arg is an edge of the row and carries the extremal message
        for v in range(n):
            for j in range(F):
                k = arg[v, j]
                if empty[v]:
                    assert k == -1 and ref[v, j] == 0.0
                else:
                    assert rowptr[v] <= k < rowptr[v + 1]
                    assert M[v, colidx[k], j] == ref[v, j]


def test_general_forward_reduces_to_the_pinned_weighted_sum():
    rng = np.random.default_rng(7)
    rowptr, colidx, X, _ = make_inputs(rng, 40, 300, 6, 1, no_dup=False)
    w = rng.uniform(-1, 1, len(colidx)).astype(np.float32)
    a, am, _ = oracle.general_forward(rowptr, colidx, X, w.reshape(-1, 1), BIN_MUL, RED_SUM)
    b, bm = oracle.ap_forward(rowptr, colidx, w, X, oracle.OP_SUM)
    assert np.array_equal(a, b) and np.array_equal(am, bm)
    a, _, _ = oracle.general_forward(rowptr, colidx, X, None, BIN_COPY_LHS, RED_SUM)
    b, _ = oracle.ap_forward(rowptr, colidx, None, X, oracle.OP_SUM)
    assert np.array_equal(a, b)


def test_general_forward_algebraic_identities():
    rng = np.random.default_rng(8)
    n, F = 31, 4
    rowptr, colidx, X, Y = make_inputs(rng, n, 250, F, F, positive_y=True, no_dup=False)
    plain, _ = oracle.ap_forward(rowptr, colidx, None, X, oracle.OP_SUM)
    seg = np.add.reduceat(np.vstack([Y.astype(np.float64), np.zeros((1, F))]),
                          np.minimum(rowptr[:-1], len(colidx)), axis=0)
    seg[np.diff(rowptr) == 0] = 0.0
    get = lambda b, r, fV=X, fE=Y: oracle.general_forward(rowptr, colidx, fV, fE, b, r, F=F)[0]
    np.testing.assert_allclose(get(BIN_COPY_RHS, RED_SUM, None), seg, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(get(BIN_ADD, RED_SUM), plain + seg, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(get(BIN_SUB, RED_SUM), plain - seg, rtol=1e-12, atol=1e-12)
    inv = (1.0 / Y.astype(np.float64))
    # division is multiplication by the reciprocal (up to the reciprocal's rounding to fp32)
    np.testing.assert_allclose(get(BIN_DIV, RED_SUM), get(BIN_MUL, RED_SUM, X, inv.astype(np.float32)),
                               rtol=1e-5, atol=1e-6)
    # min(x) = -max(-x), and sub is antisymmetric under exchanging the sign of both operands
    assert np.array_equal(get(BIN_COPY_LHS, RED_MIN), -get(BIN_COPY_LHS, RED_MAX, -X))
    assert np.array_equal(get(BIN_ADD, RED_MIN), -get(BIN_ADD, RED_MAX, -X, -Y))
    # max >= mean >= min on every non-empty row
    deg = np.diff(rowptr)[:, None]
    mean = plain / np.maximum(deg, 1)
    ne = (deg > 0)[:, 0]
    assert np.all(get(BIN_COPY_LHS, RED_MAX)[ne] >= mean[ne] - 1e-12)
    assert np.all(get(BIN_COPY_LHS, RED_MIN)[ne] <= mean[ne] + 1e-12)


def test_max_min_ties_take_the_lowest_edge_position():
    # vertex 0 has four in-edges; features with repeated values make ties
    rowptr, colidx = csr_from_lists(5, [[1, 2, 3, 4], [], [0, 0], [], [4]])
    X = np.array([[1, 5], [7, 2], [7, 2], [3, 9], [7, 9]], dtype=np.float32)
    ref, _, arg = oracle.general_forward(rowptr, colidx, X, None, BIN_COPY_LHS, RED_MAX)
    assert ref[0].tolist() == [7.0, 9.0] and arg[0].tolist() == [0, 2]
    ref, _, arg = oracle.general_forward(rowptr, colidx, X, None, BIN_COPY_LHS, RED_MIN)
    assert ref[0].tolist() == [3.0, 2.0] and arg[0].tolist() == [2, 0]
    assert arg[1].tolist() == [-1, -1] and ref[1].tolist() == [0.0, 0.0]
    assert arg[2].tolist() == [4, 4]                     # duplicate edges: the first one
    # a row of negative messages: the zero the output starts from is not a candidate
    ref, _, _ = oracle.general_forward(rowptr, colidx, -X, None, BIN_COPY_LHS, RED_MAX)
    assert ref[0].tolist() == [-3.0, -2.0]


def test_max_min_messages_are_fp32():
    """x + y with x = 1, y = 2^-30 is 1 in fp32 and larger than 1 in fp64: the extremum and its
    arg must be those of the fp32 messages."""
    rowptr, colidx = csr_from_lists(3, [[1, 2], [], []])
    X = np.array([[0.0], [1.0], [1.0]], dtype=np.float32)
    Y = np.array([[0.0], [2.0 ** -30]], dtype=np.float32)
    ref, _, arg = oracle.general_forward(rowptr, colidx, X, Y, BIN_ADD, RED_MAX)
    assert ref[0, 0] == 1.0 and arg[0, 0] == 0


# ----------------------------------------------------------------------------- gradients
def inner(rowptr, colidx, X, Y, binary, reduce, G, F):
    fV = None if binary == BIN_COPY_RHS else X
    fE = None if binary == BIN_COPY_LHS else Y
    ref, _, _ = oracle.general_forward(rowptr, colidx, fV, fE, binary, reduce, F=F)
    return float((ref * G).sum())


@pytest.mark.parametrize("binary,reduce", list(itertools.product(BINARIES, REDUCERS)))
@pytest.mark.parametrize("cols_full", [True, False])
def test_general_backward_is_the_directional_derivative(binary, reduce, cols_full):
    rng = np.random.default_rng(1000 + 100 * binary + 10 * reduce + cols_full)
    n, F = 19, 4
    cols = F if cols_full else 1
    rowptr, colidx, X, Y = make_inputs(rng, n, 110, F, cols, positive_y=True,
                                       no_dup=(reduce != RED_SUM))
    if reduce != RED_SUM:
        # the derivative of a max exists only where the best message is unique: redraw until the
        # best and the second-best message of every (row, feature) are 0.02 apart
        for _ in range(200):
            M, mask = dense_messages(rowptr, colidx, None if binary == BIN_COPY_RHS else X,
                                     None if binary == BIN_COPY_LHS else Y, binary, np.float64, F)
            Mm = np.sort(np.where(mask[:, :, None], M if reduce == RED_MAX else -M, -np.inf), axis=1)
            two = mask.sum(axis=1) >= 2
            if np.all((Mm[two, -1, :] - Mm[two, -2, :]) >= 0.02):
                break
            rowptr, colidx, X, Y = make_inputs(rng, n, 45, F, cols, positive_y=True, no_dup=True)
        else:
            raise AssertionError("no well separated draw found")
    G = rng.standard_normal((n, F)).astype(np.float32)
    fV = None if binary == BIN_COPY_RHS else X
    fE = None if binary == BIN_COPY_LHS else Y
    _, _, arg = oracle.general_forward(rowptr, colidx, fV, fE, binary, reduce, F=F)
    dV, magV, dE, magE = oracle.general_backward(rowptr, colidx, fV, fE, binary, reduce, arg, G)
    h = 2.0 ** -12
    dX = rng.integers(-1, 2, size=X.shape).astype(np.float32)
    dY = rng.integers(-1, 2, size=Y.shape).astype(np.float32)
    if binary != BIN_COPY_RHS:
        fd = (inner(rowptr, colidx, X + h * dX, Y, binary, reduce, G, F) -
              inner(rowptr, colidx, X - h * dX, Y, binary, reduce, G, F)) / (2 * h)
        assert abs(fd - float((dV * dX).sum())) <= 2e-3 * max(1.0, float((magV * np.abs(dX)).sum()))
        assert np.all(magV >= np.abs(dV) - 1e-12)
    else:
        assert np.all(dV == 0.0)
    if binary != BIN_COPY_LHS:
        fd = (inner(rowptr, colidx, X, Y + h * dY, binary, reduce, G, F) -
              inner(rowptr, colidx, X, Y - h * dY, binary, reduce, G, F)) / (2 * h)
        assert abs(fd - float((dE * dY).sum())) <= 2e-3 * max(1.0, float((magE * np.abs(dY)).sum()))
    else:
        assert dE is None


def test_general_backward_sum_copylhs_is_the_pinned_adjoint():
    rng = np.random.default_rng(3)
    rowptr, colidx, X, _ = make_inputs(rng, 30, 200, 5, 1, no_dup=False)
    G = rng.standard_normal(X.shape).astype(np.float32)
    dV, magV, _, _ = oracle.general_backward(rowptr, colidx, X, None, BIN_COPY_LHS, RED_SUM, None, G)
    colptr, rowidx_T, _, _ = oracle.transpose(rowptr, colidx, None)
    want, wmag = oracle.ap_backward(rowptr, colptr, rowidx_T, None, G, oracle.OP_SUM)
    np.testing.assert_allclose(dV, want, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(magV, wmag, rtol=1e-13, atol=1e-13)


def test_max_backward_routes_the_gradient_to_the_arg_source_only():
    rowptr, colidx = csr_from_lists(4, [[1, 2, 3], [], [0, 1], []])
    X = np.array([[9, 0], [1, 8], [5, 5], [2, 6]], dtype=np.float32)
    G = np.array([[10, 20], [0, 0], [30, 40], [0, 0]], dtype=np.float32)
    _, _, arg = oracle.general_forward(rowptr, colidx, X, None, BIN_COPY_LHS, RED_MAX)
    dV, _, _, _ = oracle.general_backward(rowptr, colidx, X, None, BIN_COPY_LHS, RED_MAX, arg, G)
    # row 0: feature 0 max is vertex 2 (5), feature 1 max is vertex 1 (8)
    # row 2: feature 0 max is vertex 0 (9), feature 1 max is vertex 1 (8)
    want = np.array([[30, 0], [0, 20 + 40], [10, 0], [0, 0]], dtype=np.float64)
    assert np.array_equal(dV, want)


# ----------------------------------------------------------------------------- edge-weight gradient
@pytest.mark.parametrize("op", [oracle.OP_SUM, oracle.OP_MEAN])
@pytest.mark.parametrize("self_loops", [False, True])
def test_edge_weight_grad_is_linear_in_the_weights(op, self_loops):
    """sum_k dW[k] * dw[k] = <AP_{dw}(H), G> - (the self-loop term, which has no weight): the
    weighted sum is linear in w, so the identity is exact and uses only the pinned forward."""
    rng = np.random.default_rng(11 + op + 2 * self_loops)
    rowptr, colidx = random_csr(rng, 37, 300)
    H = rng.standard_normal((37, 6)).astype(np.float32)
    G = rng.standard_normal((37, 6)).astype(np.float32)
    dW, mag = oracle.edge_weight_grad(rowptr, colidx, H, G, op, self_loops=self_loops)
    dw = rng.standard_normal(len(colidx)).astype(np.float32)
    with_dw, _ = oracle.ap_forward(rowptr, colidx, dw, H, op, self_loops=self_loops)
    with_0, _ = oracle.ap_forward(rowptr, colidx, np.zeros_like(dw), H, op, self_loops=self_loops)
    want = float(((with_dw - with_0) * G).sum())
    assert abs(float((dW * dw).sum()) - want) <= 1e-10 * max(1.0, float((mag * np.abs(dw)).sum()))
    # one edge at a time: dW[k] is the change of <AP, G> per unit of w[k]
    for k in (0, len(colidx) // 2, len(colidx) - 1):
        e = np.zeros_like(dw)
        e[k] = 1.0
        one, _ = oracle.ap_forward(rowptr, colidx, e, H, op, self_loops=self_loops)
        assert abs(dW[k] - float(((one - with_0) * G).sum())) <= 1e-10 * max(1.0, mag[k])
    assert np.all(mag >= np.abs(dW) - 1e-12)


def test_edge_weight_grad_equals_general_backward_for_mul_sum():
    rng = np.random.default_rng(12)
    rowptr, colidx, X, Y = make_inputs(rng, 25, 160, 7, 1, no_dup=False)
    G = rng.standard_normal(X.shape).astype(np.float32)
    dW, mag = oracle.edge_weight_grad(rowptr, colidx, X, G, oracle.OP_SUM)
    _, _, dE, magE = oracle.general_backward(rowptr, colidx, X, Y, BIN_MUL, RED_SUM, None, G,
                                             want_dV=False)
    np.testing.assert_allclose(dW, dE[:, 0], rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(mag, magE[:, 0], rtol=1e-13, atol=1e-13)


# ----------------------------------------------------------------------------- ordering, relabelling
def test_order_by_degree_is_numpy_lexsort():
    rng = np.random.default_rng(21)
    deg = rng.integers(0, 6, size=200).astype(np.int64)          # many ties
    new_of_old = oracle.order_by_degree(deg)
    old_of_new = np.lexsort((np.arange(200), -deg))              # degree descending, id ascending
    want = np.empty(200, dtype=np.int32)
    want[old_of_new] = np.arange(200, dtype=np.int32)
    assert np.array_equal(new_of_old, want)
    assert np.all(np.diff(deg[old_of_new]) <= 0)
    assert oracle.order_by_degree(np.zeros(0, dtype=np.int64)).shape == (0,)


def dense_adjacency(rowptr, colidx, w):
    n = len(rowptr) - 1
    A = np.zeros((n, n))
    for v in range(n):
        for k in range(rowptr[v], rowptr[v + 1]):
            A[v, colidx[k]] += 1.0 if w is None else float(w[k])
    return A


@pytest.mark.parametrize("weighted", [False, True])
@pytest.mark.parametrize("sorted_rows", [True, False])
def test_relabel_is_P_A_Pt_with_sorted_rows(weighted, sorted_rows):
    rng = np.random.default_rng(31 + weighted + 2 * sorted_rows)
    n = 29
    rowptr, colidx = random_csr(rng, n, 230, sort_rows=sorted_rows)
    w = rng.uniform(0.1, 1, len(colidx)).astype(np.float32) if weighted else None
    new_of_old = rng.permutation(n).astype(np.int32)
    rp2, ci2, w2, pos2 = oracle.relabel(rowptr, colidx, w, new_of_old)
    P = np.zeros((n, n))
    P[new_of_old, np.arange(n)] = 1.0                            # (P x)[new(v)] = x[v]
    np.testing.assert_allclose(dense_adjacency(rp2, ci2, w2),
                               P @ dense_adjacency(rowptr, colidx, w) @ P.T, rtol=0, atol=1e-12)
    # rows sorted by new id, duplicates in old-position order; pos2 is a permutation that maps
    # every new entry to an old entry of the matching row and source
    assert sorted(pos2.tolist()) == list(range(len(colidx)))
    old_dst = np.repeat(np.arange(n), np.diff(rowptr))
    new_dst = np.repeat(np.arange(n), np.diff(rp2))
    assert np.array_equal(new_of_old[old_dst[pos2]], new_dst)
    assert np.array_equal(new_of_old[colidx[pos2]], ci2)
    for i in range(n):
        seg, pseg = ci2[rp2[i]:rp2[i + 1]], pos2[rp2[i]:rp2[i + 1]]
        assert np.all(np.diff(seg) >= 0)
        assert np.all(np.diff(pseg)[np.diff(seg) == 0] > 0)
    if weighted:
        assert w2.tobytes() == w[pos2].tobytes()
    # AP on the relabelled graph of the permuted features is the permuted AP
    H = rng.standard_normal((n, 3)).astype(np.float32)
    H2 = np.empty_like(H)
    H2[new_of_old] = H
    for op in (oracle.OP_SUM, oracle.OP_MEAN):
        a, _ = oracle.ap_forward(rowptr, colidx, w, H, op)
        b, _ = oracle.ap_forward(rp2, ci2, w2, H2, op)
        np.testing.assert_allclose(b[new_of_old], a, rtol=1e-12, atol=1e-12)


def test_relabel_identity_inverse_and_bad_input():
    rng = np.random.default_rng(41)
    n = 17
    rowptr, colidx = random_csr(rng, n, 90, sort_rows=True)
    ident = np.arange(n, dtype=np.int32)
    rp2, ci2, _, pos2 = oracle.relabel(rowptr, colidx, None, ident)
    assert np.array_equal(rp2, rowptr) and np.array_equal(ci2, colidx)
    assert np.array_equal(pos2, np.arange(len(colidx)))
    p = rng.permutation(n).astype(np.int32)
    inv = np.empty_like(p)
    inv[p] = np.arange(n, dtype=np.int32)
    a = oracle.relabel(rowptr, colidx, None, p)
    b = oracle.relabel(a[0], a[1], None, inv)
    assert np.array_equal(b[0], rowptr) and np.array_equal(b[1], colidx)
    with pytest.raises(ValueError):
        oracle.relabel(rowptr, colidx, None, np.zeros(n, dtype=np.int32))      # not a permutation


# ----------------------------------------------------------------------------- planted mistakes
def test_general_pins_notice_planted_mistakes():
    rng = np.random.default_rng(51)
    n, F = 23, 5
    rowptr, colidx, X, Y = make_inputs(rng, n, 140, F, F)
    # swapped operands of sub / div
    M, mask = dense_messages(rowptr, colidx, X, Y, BIN_SUB, np.float64, F)
    good = np.where(mask[:, :, None], M, 0.0).sum(axis=1)
    swapped, _, _ = oracle.general_forward(rowptr, colidx, X, -Y, BIN_ADD, RED_SUM)      # x - y, fine
    np.testing.assert_allclose(swapped, good, rtol=1e-12, atol=1e-12)
    wrong = -good                                                                      # y - x
    assert not np.allclose(wrong, good)
    # max that lets the initial zero compete
    negX = -np.abs(X) - 1.0
    ref, _, _ = oracle.general_forward(rowptr, colidx, negX, None, BIN_COPY_LHS, RED_MAX)
    ne = np.diff(rowptr) > 0
    assert np.all(ref[ne] < 0.0)
    # the edge feature of another edge (index by source instead of by position)
    by_source = oracle.general_forward(rowptr, colidx, X, X[colidx], BIN_MUL, RED_SUM)[0]
    by_pos = oracle.general_forward(rowptr, colidx, X, Y, BIN_MUL, RED_SUM)[0]
    assert not np.allclose(by_source, by_pos)
    # relabelling with the inverse permutation instead of the permutation
    p = rng.permutation(n).astype(np.int32)
    inv = np.empty_like(p)
    inv[p] = np.arange(n, dtype=np.int32)
    P = np.zeros((n, n))
    P[p, np.arange(n)] = 1.0
    A = dense_adjacency(rowptr, colidx, None)
    rp2, ci2, _, _ = oracle.relabel(rowptr, colidx, None, inv)
    assert not np.allclose(dense_adjacency(rp2, ci2, None), P @ A @ P.T)
