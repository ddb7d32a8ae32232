"""Pins of the CPU oracle against what the paper and the mathematics fix (CPU only).

The paper prints no numeric AP output, so each oracle function is pinned by something other
than itself: a dense fp64 matrix product assembled edge by edge in Python, closed-form graphs,
the column-sum invariant, the adjoint identity, an O(n*nnz) brute-force transpose, scipy
as a third party, and, for the self-loop switch, the graph with its loops written out.  The planted-mistake tests at the end show that the pins notice a dropped
weight, a transposed operand, a wrong divisor and an unstable sort.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_accounting.txt")


# ----------------------------------------------------------------------------- helpers
def random_csr(rng, n, nnz, sort_rows=True, allow_dup=True):
    """Random directed multigraph in CSR (rows = destinations), with empty rows likely."""
    dst = rng.integers(0, n, size=nnz)
    src = rng.integers(0, n, size=nnz)
    if not allow_dup:
        key = np.unique(dst * n + src)
        dst, src = key // n, key % n
    order = np.lexsort((src, dst)) if sort_rows else np.argsort(dst, kind="stable")
    dst, src = dst[order], src[order]
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.add.at(rowptr, dst + 1, 1)
    rowptr = np.cumsum(rowptr)
    return rowptr.astype(np.int64), src.astype(np.int32)


def dense_from_csr(rowptr, colidx, w, op):
    """Dense fp64 A, one Python statement per edge: A[v, u] += w, rows scaled by 1/deg for mean."""
    n = len(rowptr) - 1
    A = np.zeros((n, n), dtype=np.float64)
    for v in range(n):
        for k in range(rowptr[v], rowptr[v + 1]):
            A[v, colidx[k]] += 1.0 if w is None else float(w[k])
        deg = rowptr[v + 1] - rowptr[v]
        if op == oracle.OP_MEAN and deg > 0:
            A[v, :] /= deg
    return A


def csr_from_lists(n, rows):
    rowptr = np.zeros(n + 1, dtype=np.int64)
    col = []
    for v in range(n):
        col.extend(rows[v])
        rowptr[v + 1] = len(col)
    return rowptr, np.asarray(col, dtype=np.int32)


# ----------------------------------------------------------------------------- forward
@pytest.mark.parametrize("op", [oracle.OP_SUM, oracle.OP_MEAN])
@pytest.mark.parametrize("weighted", [False, True])
@pytest.mark.parametrize("n,nnz,F", [(1, 3, 5), (7, 0, 4), (17, 40, 3), (64, 700, 9)])
def test_forward_equals_dense_product(op, weighted, n, nnz, F):
    rng = np.random.default_rng(1000 + n + nnz)
    rowptr, colidx = random_csr(rng, n, nnz)
    w = rng.random(nnz).astype(np.float32) if weighted else None
    H = rng.standard_normal((n, F)).astype(np.float32)
    ref, mag = oracle.ap_forward(rowptr, colidx, w, H, op)
    A = dense_from_csr(rowptr, colidx, w, op)
    np.testing.assert_allclose(ref, A @ H.astype(np.float64), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(mag, np.abs(A) @ np.abs(H.astype(np.float64)), rtol=1e-12,
                               atol=1e-13)


def test_forward_row_subset_matches_full():
    rng = np.random.default_rng(5)
    rowptr, colidx = random_csr(rng, 50, 400)
    H = rng.standard_normal((50, 6)).astype(np.float32)
    full, fmag = oracle.ap_forward(rowptr, colidx, None, H, oracle.OP_MEAN)
    rows = np.array([49, 0, 7, 7, 23])
    sub, smag = oracle.ap_forward(rowptr, colidx, None, H, oracle.OP_MEAN, rows=rows)
    assert np.array_equal(sub, full[rows]) and np.array_equal(smag, fmag[rows])


def test_identity_and_ring_are_bit_exact():
    n, F = 33, 7
    rng = np.random.default_rng(2)
    H = rng.standard_normal((n, F)).astype(np.float32)
    rowptr, col = csr_from_lists(n, [[v] for v in range(n)])
    for op in (oracle.OP_SUM, oracle.OP_MEAN):
        ref, _ = oracle.ap_forward(rowptr, col, None, H, op)
        assert np.array_equal(ref, H.astype(np.float64))
    rowptr, col = csr_from_lists(n, [[(v - 1) % n] for v in range(n)])
    ref, _ = oracle.ap_forward(rowptr, col, None, H, oracle.OP_SUM)
    assert np.array_equal(ref, np.roll(H, 1, axis=0).astype(np.float64))


def test_star_and_complete_graph():
    n, F = 20, 4
    rng = np.random.default_rng(3)
    H = rng.standard_normal((n, F)).astype(np.float32)
    H64 = H.astype(np.float64)
    rowptr, col = csr_from_lists(n, [list(range(1, n))] + [[] for _ in range(n - 1)])
    ref, _ = oracle.ap_forward(rowptr, col, None, H, oracle.OP_SUM)
    np.testing.assert_allclose(ref[0], H64[1:].sum(0), rtol=1e-13)
    assert np.all(ref[1:] == 0.0)
    mean, _ = oracle.ap_forward(rowptr, col, None, H, oracle.OP_MEAN)
    np.testing.assert_allclose(mean[0], H64[1:].mean(0), rtol=1e-13)
    assert np.all(mean[1:] == 0.0)          # empty rows stay zero, also for mean
    rowptr, col = csr_from_lists(n, [[u for u in range(n) if u != v] for v in range(n)])
    ref, _ = oracle.ap_forward(rowptr, col, None, H, oracle.OP_SUM)
    np.testing.assert_allclose(ref, H64.sum(0)[None, :] - H64, rtol=1e-12, atol=1e-13)


def test_all_ones_features_give_weighted_degree():
    rng = np.random.default_rng(4)
    n, nnz = 40, 300
    rowptr, colidx = random_csr(rng, n, nnz)
    w = rng.random(nnz).astype(np.float32)
    H = np.ones((n, 3), dtype=np.float32)
    wsum = np.array([w[rowptr[v]:rowptr[v + 1]].astype(np.float64).sum() for v in range(n)])
    deg = np.diff(rowptr)
    s, _ = oracle.ap_forward(rowptr, colidx, w, H, oracle.OP_SUM)
    np.testing.assert_allclose(s, np.repeat(wsum[:, None], 3, 1), rtol=1e-13)
    m, _ = oracle.ap_forward(rowptr, colidx, w, H, oracle.OP_MEAN)
    expect = np.where(deg > 0, wsum / np.maximum(deg, 1), 0.0)
    np.testing.assert_allclose(m, np.repeat(expect[:, None], 3, 1), rtol=1e-13)
    u, _ = oracle.ap_forward(rowptr, colidx, None, H, oracle.OP_SUM)
    assert np.array_equal(u[:, 0], deg.astype(np.float64))


@pytest.mark.parametrize("weighted", [False, True])
def test_column_sum_invariant(weighted):
    """sum_v out[v] = sum_u outw(u) H[u]; for mean, sum_v deg(v) out[v] equals the same."""
    rng = np.random.default_rng(6)
    n, nnz, F = 300, 5000, 5
    rowptr, colidx = random_csr(rng, n, nnz)
    w = rng.random(nnz).astype(np.float32) if weighted else None
    H = rng.standard_normal((n, F)).astype(np.float32)
    outw = np.zeros(n)
    np.add.at(outw, colidx, 1.0 if w is None else w.astype(np.float64))
    expect = (outw[:, None] * H.astype(np.float64)).sum(0)
    s, _ = oracle.ap_forward(rowptr, colidx, w, H, oracle.OP_SUM)
    np.testing.assert_allclose(s.sum(0), expect, rtol=1e-10, atol=1e-10)
    m, _ = oracle.ap_forward(rowptr, colidx, w, H, oracle.OP_MEAN)
    deg = np.diff(rowptr).astype(np.float64)
    np.testing.assert_allclose((deg[:, None] * m).sum(0), expect, rtol=1e-10, atol=1e-10)


def test_forward_matches_scipy():
    sp = pytest.importorskip("scipy.sparse")
    rng = np.random.default_rng(7)
    n, nnz, F = 500, 9000, 11
    rowptr, colidx = random_csr(rng, n, nnz)
    w = rng.random(nnz).astype(np.float32)
    H = rng.standard_normal((n, F)).astype(np.float32)
    A = sp.csr_matrix((w.astype(np.float64), colidx, rowptr), shape=(n, n))
    ref, _ = oracle.ap_forward(rowptr, colidx, w, H, oracle.OP_SUM)
    np.testing.assert_allclose(ref, A @ H.astype(np.float64), rtol=1e-11, atol=1e-12)


# ----------------------------------------------------------------------------- transpose
def brute_transpose(rowptr, colidx):
    """For each source u, scan every CSR position in order: O(n * nnz), stable by construction."""
    n = len(rowptr) - 1
    row_of = np.repeat(np.arange(n), np.diff(rowptr))
    colptr, rowidx, perm = [0], [], []
    for u in range(n):
        for k in range(len(colidx)):
            if colidx[k] == u:
                perm.append(k)
                rowidx.append(row_of[k])
        colptr.append(len(perm))
    return np.array(colptr), np.array(rowidx), np.array(perm)


@pytest.mark.parametrize("sort_rows", [True, False])
def test_transpose_matches_brute_force(sort_rows):
    rng = np.random.default_rng(8)
    n, nnz = 37, 260
    rowptr, colidx = random_csr(rng, n, nnz, sort_rows=sort_rows)
    w = rng.random(nnz).astype(np.float32)
    colptr, rowidx_T, w_T, perm = oracle.transpose(rowptr, colidx, w)
    bc, br, bp = brute_transpose(rowptr, colidx)
    assert np.array_equal(colptr, bc) and np.array_equal(rowidx_T, br)
    assert np.array_equal(perm, bp)
    assert w_T.tobytes() == w[bp].tobytes()


def test_transpose_is_an_involution_on_sorted_rows():
    rng = np.random.default_rng(9)
    n, nnz = 200, 3000
    rowptr, colidx = random_csr(rng, n, nnz, sort_rows=True)
    w = rng.random(nnz).astype(np.float32)
    colptr, rowidx_T, w_T, perm = oracle.transpose(rowptr, colidx, w)
    back_ptr, back_idx, back_w, _ = oracle.transpose(colptr, rowidx_T, w_T)
    assert np.array_equal(back_ptr, rowptr) and np.array_equal(back_idx, colidx)
    # duplicate edges carry different weights; (A^T)^T restores their order too
    assert back_w.tobytes() == w.tobytes()


def test_transpose_properties_and_scipy():
    sp = pytest.importorskip("scipy.sparse")
    rng = np.random.default_rng(10)
    n, nnz = 400, 6000
    rowptr, colidx = random_csr(rng, n, nnz, allow_dup=False)
    nnz = len(colidx)
    colptr, rowidx_T, _, perm = oracle.transpose(rowptr, colidx, None)
    assert np.array_equal(np.sort(perm), np.arange(nnz))
    keys = colidx[perm]
    assert np.all(np.diff(keys) >= 0)
    same = np.diff(keys) == 0
    assert np.all(np.diff(perm)[same] > 0)          # stable inside equal keys
    assert np.array_equal(np.diff(colptr), np.bincount(colidx, minlength=n))
    A = sp.csr_matrix((np.arange(1, nnz + 1, dtype=np.float64), colidx, rowptr), shape=(n, n))
    T = A.T.tocsr()
    T.sort_indices()
    assert np.array_equal(T.indptr, colptr) and np.array_equal(T.indices, rowidx_T)
    assert np.array_equal(T.data.astype(np.int64) - 1, perm)


def test_transpose_empty_graph():
    colptr, rowidx_T, w_T, perm = oracle.transpose(np.zeros(6, dtype=np.int64),
                                                   np.zeros(0, dtype=np.int32), None)
    assert np.array_equal(colptr, np.zeros(6)) and rowidx_T.size == 0 and perm.size == 0


# ----------------------------------------------------------------------------- backward
@pytest.mark.parametrize("op", [oracle.OP_SUM, oracle.OP_MEAN])
@pytest.mark.parametrize("weighted", [False, True])
def test_backward_equals_dense_transposed_product(op, weighted):
    rng = np.random.default_rng(11)
    n, nnz, F = 48, 500, 6
    rowptr, colidx = random_csr(rng, n, nnz)
    w = rng.random(nnz).astype(np.float32) if weighted else None
    G = rng.standard_normal((n, F)).astype(np.float32)
    colptr, rowidx_T, w_T, _ = oracle.transpose(rowptr, colidx, w)
    ref, mag = oracle.ap_backward(rowptr, colptr, rowidx_T, w_T, G, op)
    A = dense_from_csr(rowptr, colidx, w, op)
    np.testing.assert_allclose(ref, A.T @ G.astype(np.float64), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(mag, np.abs(A).T @ np.abs(G.astype(np.float64)), rtol=1e-12,
                               atol=1e-13)


@pytest.mark.parametrize("op", [oracle.OP_SUM, oracle.OP_MEAN])
@pytest.mark.parametrize("weighted", [False, True])
def test_adjoint_identity(op, weighted):
    """<AP(H), G> = <H, AP^T(G)> needs no second implementation of either side."""
    rng = np.random.default_rng(12)
    n, nnz, F = 700, 12000, 8
    rowptr, colidx = random_csr(rng, n, nnz)
    w = rng.random(nnz).astype(np.float32) if weighted else None
    H = rng.standard_normal((n, F)).astype(np.float32)
    G = rng.standard_normal((n, F)).astype(np.float32)
    colptr, rowidx_T, w_T, _ = oracle.transpose(rowptr, colidx, w)
    out, _ = oracle.ap_forward(rowptr, colidx, w, H, op)
    dH, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, w_T, G, op)
    lhs = float((out * G.astype(np.float64)).sum())
    rhs = float((H.astype(np.float64) * dH).sum())
    assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))


def test_backward_mean_on_regular_graph():
    """Every vertex has in-degree k, so the mean's backward is (1/k) A^T G."""
    n, k, F = 30, 4, 3
    rng = np.random.default_rng(13)
    rowptr, col = csr_from_lists(n, [sorted((v + d) % n for d in (1, 2, 5, 11))
                                     for v in range(n)])
    G = rng.standard_normal((n, F)).astype(np.float32)
    colptr, rowidx_T, _, _ = oracle.transpose(rowptr, col, None)
    m, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, None, G, oracle.OP_MEAN)
    s, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, None, G, oracle.OP_SUM)
    np.testing.assert_allclose(m, s / k, rtol=1e-13, atol=1e-15)


def test_backward_column_subset_matches_full():
    rng = np.random.default_rng(14)
    rowptr, colidx = random_csr(rng, 60, 500)
    G = rng.standard_normal((60, 5)).astype(np.float32)
    colptr, rowidx_T, _, _ = oracle.transpose(rowptr, colidx, None)
    full, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, None, G, oracle.OP_MEAN)
    cols = np.array([59, 3, 3, 0])
    sub, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, None, G, oracle.OP_MEAN, cols=cols)
    assert np.array_equal(sub, full[cols])


# ----------------------------------------------------------------------------- self loops
def with_explicit_self_loops(rowptr, colidx, w):
    """The same graph with one edge v -> v of weight 1 appended to every row."""
    n = len(rowptr) - 1
    rows, ws = [], []
    for v in range(n):
        lo, hi = rowptr[v], rowptr[v + 1]
        rows.append(list(colidx[lo:hi]) + [v])
        ws.extend(([1.0] * (hi - lo) if w is None else list(w[lo:hi])) + [1.0])
    rp, ci = csr_from_lists(n, rows)
    return rp, ci, np.asarray(ws, dtype=np.float32)


@pytest.mark.parametrize("op", [oracle.OP_SUM, oracle.OP_MEAN])
@pytest.mark.parametrize("weighted", [False, True])
def test_self_loops_equal_the_graph_with_the_loops_written_out(op, weighted):
    """Forward and backward with the switch = the plain operators on A + I (a different path
    through the oracle: there the own row is one more edge of the loop over neighbours)."""
    rng = np.random.default_rng(21)
    n, nnz, F = 50, 400, 5
    rowptr, colidx = random_csr(rng, n, nnz)           # has empty rows and duplicate edges
    w = rng.random(nnz).astype(np.float32) if weighted else None
    H = rng.standard_normal((n, F)).astype(np.float32)
    G = rng.standard_normal((n, F)).astype(np.float32)
    rp2, ci2, w2 = with_explicit_self_loops(rowptr, colidx, w)
    got, gmag = oracle.ap_forward(rowptr, colidx, w, H, op, self_loops=True)
    want, wmag = oracle.ap_forward(rp2, ci2, w2, H, op)
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(gmag, wmag, rtol=1e-13, atol=1e-15)
    colptr, rowidx_T, w_T, _ = oracle.transpose(rowptr, colidx, w)
    cp2, ri2, wT2, _ = oracle.transpose(rp2, ci2, w2)
    got, gmag = oracle.ap_backward(rowptr, colptr, rowidx_T, w_T, G, op, self_loops=True)
    want, wmag = oracle.ap_backward(rp2, cp2, ri2, wT2, G, op)
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(gmag, wmag, rtol=1e-13, atol=1e-15)


def test_gcn_aggregator_dense_and_constant_features():
    """(sum of neighbours + own row) / (in-degree + 1), Section 5.1: against the dense product
    (A + I) H scaled row by row; a constant feature is a fixed point on an unweighted graph,
    isolated vertices included."""
    rng = np.random.default_rng(22)
    n, nnz, F = 40, 70, 4
    rowptr, colidx = random_csr(rng, n, nnz)
    H = rng.standard_normal((n, F)).astype(np.float32)
    A = dense_from_csr(rowptr, colidx, None, oracle.OP_SUM)
    deg = np.diff(rowptr).astype(np.float64)
    assert (deg == 0).any()
    want = (A @ H.astype(np.float64) + H) / (deg + 1.0)[:, None]
    got, _ = oracle.ap_forward(rowptr, colidx, None, H, oracle.OP_MEAN, self_loops=True)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    const = np.full((n, 3), 2.5, dtype=np.float32)
    got, mag = oracle.ap_forward(rowptr, colidx, None, const, oracle.OP_MEAN, self_loops=True)
    np.testing.assert_allclose(got, const, rtol=1e-14)
    np.testing.assert_allclose(mag, const, rtol=1e-14)
    # backward: ((A + I)^T D) G with D = diag(1 / (deg + 1))
    G = rng.standard_normal((n, F)).astype(np.float32)
    colptr, rowidx_T, _, _ = oracle.transpose(rowptr, colidx, None)
    got, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, None, G, oracle.OP_MEAN, self_loops=True)
    want = (A + np.eye(n)).T @ (G.astype(np.float64) / (deg + 1.0)[:, None])
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("op", [oracle.OP_SUM, oracle.OP_MEAN])
def test_adjoint_identity_with_self_loops(op):
    rng = np.random.default_rng(23)
    n, nnz, F = 300, 5000, 6
    rowptr, colidx = random_csr(rng, n, nnz)
    w = rng.random(nnz).astype(np.float32)
    H = rng.standard_normal((n, F)).astype(np.float32)
    G = rng.standard_normal((n, F)).astype(np.float32)
    colptr, rowidx_T, w_T, _ = oracle.transpose(rowptr, colidx, w)
    out, _ = oracle.ap_forward(rowptr, colidx, w, H, op, self_loops=True)
    dH, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, w_T, G, op, self_loops=True)
    lhs = float((out * G.astype(np.float64)).sum())
    rhs = float((H.astype(np.float64) * dH).sum())
    assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))
    # a backward pass that forgets the own row, or scales it by the out-degree, breaks it
    plain, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, w_T, G, op)
    assert abs(lhs - float((H.astype(np.float64) * plain).sum())) > 1e-6 * abs(lhs)


# ----------------------------------------------------------------------------- planted mistakes
def test_pins_notice_planted_mistakes():
    """Each plausible mistake, planted into a copy of the data flow, breaks one of the pins."""
    rng = np.random.default_rng(15)
    n, nnz, F = 40, 350, 4
    rowptr, colidx = random_csr(rng, n, nnz)
    w = rng.random(nnz).astype(np.float32)
    H = rng.standard_normal((n, F)).astype(np.float32)
    A = dense_from_csr(rowptr, colidx, w, oracle.OP_MEAN)
    good, _ = oracle.ap_forward(rowptr, colidx, w, H, oracle.OP_MEAN)
    # dropped weight
    bad, _ = oracle.ap_forward(rowptr, colidx, None, H, oracle.OP_MEAN)
    assert not np.allclose(bad, A @ H.astype(np.float64))
    # mean divided by the weight sum instead of the in-degree
    wsum = np.array([w[rowptr[v]:rowptr[v + 1]].sum() for v in range(n)], dtype=np.float64)
    s, _ = oracle.ap_forward(rowptr, colidx, w, H, oracle.OP_SUM)
    assert not np.allclose(s / np.maximum(wsum, 1e-30)[:, None], good)
    # transposed operand: A^T H is not A H
    assert not np.allclose(A.T @ H.astype(np.float64), good)
    # backward that takes the divisor from the source vertex instead of the destination
    colptr, rowidx_T, w_T, perm = oracle.transpose(rowptr, colidx, w)
    G = rng.standard_normal((n, F)).astype(np.float32)
    right, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, w_T, G, oracle.OP_MEAN)
    sums, _ = oracle.ap_backward(rowptr, colptr, rowidx_T, w_T, G, oracle.OP_SUM)
    outdeg = np.maximum(np.diff(colptr), 1).astype(np.float64)
    assert not np.allclose(sums / outdeg[:, None], right)
    # the five defining properties of the CSC (the check used where the oracle cannot run in
    # full) accept the oracle's result and reject each of: an unstable order inside one column,
    # a repeated position, a shifted column pointer, a wrong destination row
    assert _csc_defining_properties(rowptr, colidx, colptr, rowidx_T, perm)
    u = int(np.argmax(np.diff(colptr)))
    assert colptr[u + 1] - colptr[u] >= 2
    swapped = perm.copy()
    swapped[[colptr[u], colptr[u] + 1]] = swapped[[colptr[u] + 1, colptr[u]]]
    rows_swapped = rowidx_T.copy()
    rows_swapped[[colptr[u], colptr[u] + 1]] = rows_swapped[[colptr[u] + 1, colptr[u]]]
    assert not _csc_defining_properties(rowptr, colidx, colptr, rows_swapped, swapped)
    repeated = perm.copy()
    repeated[colptr[u] + 1] = repeated[colptr[u]]
    assert not _csc_defining_properties(rowptr, colidx, colptr, rowidx_T, repeated)
    shifted = colptr.copy()
    shifted[u + 1] -= 1
    assert not _csc_defining_properties(rowptr, colidx, shifted, rowidx_T, perm)
    wrong_row = rowidx_T.copy()
    wrong_row[colptr[u]] = (wrong_row[colptr[u]] + 1) % n
    assert not _csc_defining_properties(rowptr, colidx, colptr, wrong_row, perm)


def _csc_defining_properties(rowptr, colidx, colptr, rowidx_T, perm):
    """perm is a permutation of the edge positions; the keys colidx[perm] never decrease; perm
    increases inside equal keys; colptr holds the key boundaries; rowidx_T[q] is the CSR row
    that contains position perm[q].  Together they admit exactly one CSC."""
    nnz, n = len(colidx), len(rowptr) - 1
    if sorted(perm.tolist()) != list(range(nnz)):
        return False
    key = colidx[perm].astype(np.int64)
    dk = np.diff(key)
    if np.any(dk < 0) or np.any(np.diff(perm)[dk == 0] <= 0):
        return False
    if not np.array_equal(colptr, np.concatenate([[0], np.cumsum(np.bincount(key, minlength=n))])):
        return False
    return np.array_equal(rowidx_T, np.searchsorted(rowptr, perm, side="right") - 1)


# ----------------------------------------------------------------------------- accounting
def _golden():
    vals = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("--")[0].strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            vals[k] = float(v)
    return vals


def test_paper_accounting_values():
    """Table 2 / Table 3 / Table 8: average degrees and edge x feature work per hop."""
    g = _golden()
    assert round(g["reddit_edges"] / g["reddit_vertices"]) == g["reddit_avg_degree"]
    assert abs(g["products_edges"] / g["products_vertices"] - g["products_avg_degree"]) < 0.05
    # Table 8 counts one extra self term per vertex: 50.5 + 1 = 51.5 rows summed per vertex
    per_vertex = g["products_avg_degree"] + 1.0
    hop1 = g["products_vertices"] * per_vertex * g["products_features"] / 1e9
    hop2 = g["products_vertices"] * per_vertex * 256 / 1e9
    assert abs(hop1 - g["products_hop1_ops_billion"]) < 0.01
    assert abs(hop2 - g["products_hop2_ops_billion"]) < 0.01
    assert abs(hop1 + 2 * hop2 - g["products_total_ops_billion"]) < 0.02
    from paper_2104_06700_b200 import synth
    assert synth.CONFIG_SHAPES["reddit_like"] == (g["reddit_vertices"], g["reddit_edges"],
                                                  g["reddit_features"])
    assert synth.CONFIG_SHAPES["products_like"] == (g["products_vertices"], g["products_edges"],
                                                    g["products_features"])
    assert synth.CONFIG_SHAPES["papers_like"] == (g["papers_vertices"], g["papers_edges"],
                                                  g["papers_features"])
