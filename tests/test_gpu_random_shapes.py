"""Randomised parity: random graphs (empty rows, runs of short rows, a few very long rows and
columns, duplicate edges, optional weights), random feature widths and random launch knobs,
every case compared in full with the oracle.  The seeds are fixed, so a failure reproduces."""
import numpy as np
import pytest
import torch

from paper_2104_06700_b200 import binding, synth
from parity_util import check_fwd_bwd, check_transpose

pytestmark = pytest.mark.gpu
DEV = "cuda"
WIDTHS = [1, 2, 3, 4, 6, 8, 12, 16, 20, 32, 33, 40, 64, 66, 96, 100, 128, 130, 200, 256, 258, 300,
          512, 516, 602, 1024]


def random_graph(rng):
    n = int(rng.integers(1, 3000))
    kind = rng.integers(0, 4)
    if kind == 0:      # mostly short rows, many empty
        deg = rng.poisson(3.0, n) * (rng.random(n) < 0.6)
    elif kind == 1:    # power law with a few heavy rows
        deg = np.minimum((rng.pareto(1.2, n) * 4).astype(np.int64), 6000)
    elif kind == 2:    # uniform medium rows (dense-ish: split pointers when n >= 4096 only)
        deg = rng.integers(20, 120, n)
    else:              # one huge row, the rest tiny
        deg = rng.integers(0, 4, n)
        deg[rng.integers(0, n)] = int(rng.integers(3000, 20000))
    deg = deg.astype(np.int64)
    nnz = int(deg.sum())
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(deg, out=rowptr[1:])
    if rng.random() < 0.5:   # skewed sources: a few very long columns
        col = (n * rng.random(nnz) ** 3).astype(np.int32)
    else:
        col = rng.integers(0, n, nnz).astype(np.int32)
    col = np.minimum(col, n - 1).astype(np.int32)
    if rng.random() < 0.7:   # sort inside rows (duplicates stay)
        row = np.repeat(np.arange(n), deg)
        order = np.lexsort((col, row))
        col = col[order]
    w = rng.random(nnz).astype(np.float32) if rng.random() < 0.5 else None
    return n, nnz, rowptr, col, w


@pytest.mark.parametrize("seed", range(48))
def test_random_graph_width_and_knobs(seed):
    rng = np.random.default_rng(1000 + seed)
    n, nnz, rowptr, col, w = random_graph(rng)
    g = binding.dg_graph_create(n, nnz, torch.as_tensor(rowptr, device=DEV),
                                torch.as_tensor(col, device=DEV),
                                None if w is None else torch.as_tensor(w, device=DEV))
    g.dg_graph_validate()
    g.dg_graph_set_param("heavy_threshold", int(rng.choice([64, 100, 256, 1024, 5000])))
    g.dg_graph_set_param("rows_per_block", int(rng.choice([0, 1, 8, 24, 100, 248])))
    g.dg_graph_set_param("heavy_blocks_per_sm", int(rng.choice([0, 1, 4])))
    g.dg_graph_set_param("slice_features", int(rng.choice([0, 0, 4, 32, 100])))
    csc = check_transpose(g, rowptr, col, w)
    for F in rng.choice(WIDTHS, size=2, replace=False):
        F = int(F)
        H = synth.features(n, F, 7 + seed, DEV)
        G = synth.features(n, F, 8 + seed, DEV)
        op = int(rng.integers(0, 2))
        check_fwd_bwd(g, (rowptr, col, w), H, G, op, csc)
        if F % 2 == 0:
            Hb, Gb = H.to(torch.bfloat16), G.to(torch.bfloat16)
            a = g.dg_aggregate_fwd_bf16(Hb, op)
            b = g.dg_aggregate_fwd(Hb.float(), op)
            assert torch.allclose(a, b, rtol=2e-4, atol=1e-4)
            c = g.dg_aggregate_bwd_bf16(Gb, op)
            d = g.dg_aggregate_bwd(Gb.float(), op)
            assert torch.allclose(c, d, rtol=2e-4, atol=1e-4)


@pytest.mark.parametrize("seed", range(8))
def test_random_dense_graph_with_source_blocks(seed):
    """At least 4096 vertices and 64 edges per vertex: the handle carries split pointers, and a
    random cut into source blocks (or a small L2 budget choosing it) must not change results."""
    rng = np.random.default_rng(5000 + seed)
    n = int(rng.integers(4096, 7000))
    deg = rng.integers(64, 150, n).astype(np.int64)
    deg[rng.integers(0, n, 3)] = rng.integers(1500, 4000, 3)     # a few heavy rows
    nnz = int(deg.sum())
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(deg, out=rowptr[1:])
    col = np.minimum((n * rng.random(nnz) ** 2).astype(np.int64), n - 1).astype(np.int32)
    row = np.repeat(np.arange(n), deg)
    col = col[np.lexsort((col, row))]
    w = rng.random(nnz).astype(np.float32) if seed % 2 else None
    g = binding.dg_graph_create(n, nnz, torch.as_tensor(rowptr, device=DEV),
                                torch.as_tensor(col, device=DEV),
                                None if w is None else torch.as_tensor(w, device=DEV))
    g.dg_graph_set_param("source_blocks", int(rng.choice([0, 2, 4, 8, 16])))
    g.dg_graph_set_param("l2_budget_mb", int(rng.choice([1, 2, 38])))
    g.dg_graph_set_param("heavy_threshold", int(rng.choice([128, 1024])))
    csc = check_transpose(g, rowptr, col, w)
    for F in rng.choice([8, 64, 100, 256, 602, 1024], size=2, replace=False):
        F = int(F)
        H = synth.features(n, F, 17 + seed, DEV)
        G = synth.features(n, F, 18 + seed, DEV)
        check_fwd_bwd(g, (rowptr, col, w), H, G, int(rng.integers(0, 2)), csc)


def test_extreme_shapes():
    """One vertex with thousands of self-loops; a handful of vertices with the widest feature
    rows the library accepts (2^20 columns: 2048 feature slices in one launch)."""
    rng = np.random.default_rng(77)
    n, nnz = 1, 5000
    rowptr = np.array([0, nnz], dtype=np.int64)
    col = np.zeros(nnz, dtype=np.int32)
    w = rng.random(nnz).astype(np.float32)
    g = binding.dg_graph_create(n, nnz, torch.as_tensor(rowptr, device=DEV),
                                torch.as_tensor(col, device=DEV), torch.as_tensor(w, device=DEV))
    csc = check_transpose(g, rowptr, col, w)
    H, G = synth.features(n, 40, 1, DEV), synth.features(n, 40, 2, DEV)
    for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
        check_fwd_bwd(g, (rowptr, col, w), H, G, op, csc)

    n, F = 5, 1 << 20
    rows = [[1, 2], [0], [], [0, 1, 2, 3, 4], [4]]
    rowptr = np.zeros(n + 1, dtype=np.int64)
    rowptr[1:] = np.cumsum([len(r) for r in rows])
    col = np.concatenate([np.asarray(r, dtype=np.int32) for r in rows])
    g = binding.dg_graph_create(n, len(col), torch.as_tensor(rowptr, device=DEV),
                                torch.as_tensor(col, device=DEV), None)
    csc = check_transpose(g, rowptr, col, None)
    H, G = synth.features(n, F, 3, DEV), synth.features(n, F, 4, DEV)
    check_fwd_bwd(g, (rowptr, col, None), H, G, binding.DG_OP_MEAN, csc)
    g.dg_graph_set_param("slice_features", 1)      # would be 2^20 slices: the library widens it
    check_fwd_bwd(g, (rowptr, col, None), H, G, binding.DG_OP_SUM, csc)
    g.dg_graph_set_param("slice_features", 0)
    out = g.dg_aggregate_fwd_bf16(H.to(torch.bfloat16), binding.DG_OP_SUM)
    assert torch.allclose(out, g.dg_aggregate_fwd(H.to(torch.bfloat16).float(), binding.DG_OP_SUM),
                          rtol=1e-4, atol=1e-4)
