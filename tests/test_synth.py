"""Properties of the seeded synthetic workload generators (CPU, reduced scale)."""
import numpy as np
import pytest
import torch

from paper_2104_06700_b200 import synth


def _check_csr(g):
    rp, ci = g.rowptr.cpu().numpy(), g.colidx.cpu().numpy()
    assert rp.dtype == np.int64 and ci.dtype == np.int32
    assert rp[0] == 0 and rp[-1] == g.nnz == ci.size and np.all(np.diff(rp) >= 0)
    assert ci.min() >= 0 and ci.max() < g.n
    row = np.repeat(np.arange(g.n), np.diff(rp))
    key = row.astype(np.int64) * g.n + ci
    assert np.all(np.diff(key) >= 0)            # rows sorted ascending by source id
    return rp, ci, row, key


def test_tiny_matches_its_description():
    g = synth.make("tiny")
    rp, ci, row, key = _check_csr(g)
    assert (g.n, g.nnz, g.F) == (4096, 65536, 64)
    assert np.all(row != ci)                    # no self-loops
    assert np.unique(key).size == g.nnz         # no multi-edges
    outdeg = np.bincount(ci, minlength=g.n)
    assert outdeg.min() >= 1 and outdeg.max() <= 512
    w = g.edge_w.numpy()
    assert w.dtype == np.float32 and 0.0 <= w.min() and w.max() < 1.0
    g2 = synth.make("tiny")
    assert torch.equal(g.colidx, g2.colidx) and torch.equal(g.edge_w, g2.edge_w)


@pytest.mark.parametrize("name", ["reddit_like", "products_like", "proteins_like"])
def test_symmetrised_graphs(name):
    g = synth.make(name, scale=0.004)
    rp, ci, row, key = _check_csr(g)
    assert g.nnz % 2 == 0 and np.all(row != ci) and np.unique(key).size == g.nnz
    rev = np.sort(ci.astype(np.int64) * g.n + row)
    assert np.array_equal(rev, key)             # every edge has its reverse
    if name == "proteins_like":
        assert g.edge_feat.shape == (g.nnz, 8)
        assert torch.allclose(g.edge_w, g.edge_feat.mean(1))
        # both directions of a pair carry the same feature
        lut = dict(zip(key.tolist(), range(g.nnz)))
        for k in range(0, g.nnz, max(1, g.nnz // 50)):
            r = lut[int(ci[k]) * g.n + int(row[k])]
            assert torch.equal(g.edge_feat[k], g.edge_feat[r])


def test_reddit_like_scaled_shape_and_communities():
    g = synth.reddit_like(scale=0.01, sorted_ids=True)
    n0, nnz0, F = synth.CONFIG_SHAPES["reddit_like"]
    assert g.F == F and abs(g.nnz - round(nnz0 * 0.01)) <= 1
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    row = np.repeat(np.arange(g.n), np.diff(rp))
    bounds = np.floor(np.arange(42) * g.n / 41)
    intra = (np.searchsorted(bounds, row, side="right") ==
             np.searchsorted(bounds, ci, side="right")).mean()
    assert 0.78 < intra < 0.86                  # 80 % planted + the chance share of the rest


def test_papers_like_scaled():
    g = synth.make("papers_like", scale=0.0005)
    rp, ci, row, _ = _check_csr(g)
    n0, nnz0, F = synth.CONFIG_SHAPES["papers_like"]
    assert g.F == F and g.nnz == round(nnz0 * 0.0005) and np.all(row != ci)
    indeg = np.diff(rp)
    assert indeg[: g.n // 100].mean() > 5 * indeg[g.n // 2:].mean()   # skew toward low ids
    outdeg = np.bincount(ci, minlength=g.n)
    assert outdeg.max() > 50 * outdeg.mean()                          # heavy tail


def test_features_are_seeded():
    a, b = synth.features(100, 7, 3), synth.features(100, 7, 3)
    assert a.dtype == torch.float32 and torch.equal(a, b)
    assert not torch.equal(a, synth.features(100, 7, 4))
