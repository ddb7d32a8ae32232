"""Seeded synthetic inputs shaped like the paper's workloads (Table 2 of the paper).

This module serves both the CUDA path and the CPU oracle and holds none of the method's
arithmetic: it only draws graphs and feature matrices.  The real datasets (Reddit,
OGBN-Products, ogbn-proteins, OGBN-Papers) are not available offline; these graphs take their
vertex counts, edge counts, feature widths and degree structure and stand in for them.

Every generator returns a :class:`SynthGraph` whose CSR has rows = destination vertices and
column indices = source vertices (Section 3.1 of the paper), sorted ascending inside a row,
``rowptr`` int64 and ``colidx`` int32.  ``scale`` < 1 shrinks a workload for quick tests: the
edge count scales linearly; the two dense-ish graphs keep their density (vertices scale with
sqrt(scale)), the two sparse ones keep their mean degree.  All tensors live on the ``device``
asked for; the generators run on CPU or on a GPU (torch's CPU and CUDA generators give
different streams, so one run must feed both sides of a comparison).

Vertex ids are a random permutation of the construction order unless ``sorted_ids=True``
(real datasets are not stored community by community).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

# (vertices, directed edges, feature width) per workload; edge counts of 2, 3 and 5 are the
# paper's Table 2 values, 4 is the size the benchmark configuration names.
CONFIG_SHAPES = {
    "tiny": (4_096, 65_536, 64),
    "reddit_like": (232_965, 114_615_892, 602),
    "products_like": (2_449_029, 123_718_280, 100),
    "proteins_like": (132_534, 79_122_504, 64),
    "papers_like": (111_059_956, 1_615_685_872, 128),
}
CONFIG_SEEDS = {"tiny": 0, "reddit_like": 1, "products_like": 2, "proteins_like": 3,
                "papers_like": 4}


@dataclasses.dataclass
class SynthGraph:
    name: str
    n: int
    nnz: int
    F: int
    rowptr: torch.Tensor            # int64 [n+1]
    colidx: torch.Tensor            # int32 [nnz]
    edge_w: Optional[torch.Tensor]  # fp32 [nnz] or None
    edge_feat: Optional[torch.Tensor] = None  # fp32 [nnz, 8] (proteins_like only)
    seed: int = 0

    def stats(self) -> dict:
        deg_in = (self.rowptr[1:] - self.rowptr[:-1]).double()
        deg_out = torch.bincount(self.colidx.long(), minlength=self.n).double()
        def q(t, p):
            k = max(1, int(math.ceil(p * t.numel())))
            return float(torch.kthvalue(t.cpu(), k).values) if t.numel() else 0.0
        return {
            "n": self.n, "nnz": self.nnz,
            "n_ref": int((deg_out > 0).sum()), "n_nonempty_rows": int((deg_in > 0).sum()),
            "row_len_max": float(deg_in.max()) if self.n else 0.0,
            "row_len_mean": float(deg_in.mean()) if self.n else 0.0,
            "row_len_p99": q(deg_in, 0.99),
            "col_len_max": float(deg_out.max()) if self.n else 0.0,
            "col_len_mean": float(deg_out.mean()) if self.n else 0.0,
            "col_len_p99": q(deg_out, 0.99),
        }


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _csr_from_edges(dst: torch.Tensor, src: torch.Tensor, n: int):
    """Sort directed edges (src -> dst) by (dst, src).  Returns rowptr, colidx, order."""
    key = dst.long() * n + src.long()
    key, order = torch.sort(key)
    colidx = (key % n).to(torch.int32)
    rows = torch.div(key, n, rounding_mode="floor")
    del key
    counts = torch.bincount(rows, minlength=n)
    del rows
    rowptr = torch.zeros(n + 1, dtype=torch.int64, device=dst.device)
    torch.cumsum(counts, 0, out=rowptr[1:])
    return rowptr, colidx, order


def _sample_cdf(weights: torch.Tensor, count: int, gen: torch.Generator) -> torch.Tensor:
    """Draw ``count`` indices with probability proportional to ``weights`` (inverse CDF)."""
    cdf = torch.cumsum(weights.double(), 0)
    cdf = cdf / cdf[-1]
    u = torch.rand(count, generator=gen, device=weights.device, dtype=torch.float64)
    idx = torch.searchsorted(cdf, u, right=True)
    return idx.clamp_(max=weights.numel() - 1)


def _fix_total(deg: torch.Tensor, total: int, lo: int, hi: int, gen: torch.Generator):
    """Move ``deg`` (int64) by +-1 on random vertices until it sums to ``total``."""
    n = deg.numel()
    for _ in range(64):
        diff = total - int(deg.sum())
        if diff == 0:
            return deg
        if diff > 0:
            cand = torch.nonzero(deg < hi).flatten()
        else:
            cand = torch.nonzero(deg > lo).flatten()
        take = min(abs(diff), cand.numel())
        pick = cand[torch.randperm(cand.numel(), generator=gen, device=deg.device)[:take]]
        deg[pick] += 1 if diff > 0 else -1
    raise RuntimeError("could not reach the requested edge total")


def _exact_undirected(draw_pairs, n: int, pairs: int, gen: torch.Generator, device):
    """Call ``draw_pairs(count)`` until ``pairs`` distinct non-loop unordered pairs exist, then
    keep a random subset of exactly that size.  Returns (lo, hi) int64."""
    keys = torch.empty(0, dtype=torch.int64, device=device)
    want = int(pairs * 1.08) + 16
    for _ in range(32):
        a, b = draw_pairs(want)
        lo, hi = torch.minimum(a, b), torch.maximum(a, b)
        keep = lo != hi
        k = lo[keep] * n + hi[keep]
        keys = torch.unique(torch.cat([keys, k]))
        if keys.numel() >= pairs:
            break
        want = int((pairs - keys.numel()) * 1.5) + 16
    else:
        raise RuntimeError("could not draw enough distinct pairs")
    if keys.numel() > pairs:
        sel = torch.randperm(keys.numel(), generator=gen, device=device)[:pairs]
        keys = keys[sel]
    return torch.div(keys, n, rounding_mode="floor"), keys % n


def _relabel(n: int, sorted_ids: bool, gen: torch.Generator, device):
    if sorted_ids:
        return None
    return torch.randperm(n, generator=gen, device=device)


def _symmetric_csr(lo, hi, n, relabel):
    if relabel is not None:
        lo, hi = relabel[lo], relabel[hi]
    m = lo.numel()
    dst = torch.cat([lo, hi])
    src = torch.cat([hi, lo])
    rowptr, colidx, order = _csr_from_edges(dst, src, n)
    return rowptr, colidx, order % m


def tiny(seed: int = 0, device="cpu", n: int = 4096, nnz: int = 65536, F: int = 64,
         weighted: bool = True) -> SynthGraph:
    """Directed power-law graph: out-degree Zipf(1.5) truncated to [1, 512], destinations drawn
    without replacement from the other vertices (no self-loops, no multi-edges), weights U(0,1)."""
    gen = _gen(seed, "cpu")
    cap = min(512, n - 1)
    k = torch.arange(1, cap + 1, dtype=torch.float64)
    deg = _sample_cdf(k.pow(-1.5), n, gen) + 1
    deg = _fix_total(deg, nnz, 1, cap, gen)
    src_l, dst_l = [], []
    for u in range(n):
        d = int(deg[u])
        t = torch.randperm(n - 1, generator=gen)[:d]
        t = t + (t >= u).long()          # skip u itself
        dst_l.append(t)
        src_l.append(torch.full((d,), u, dtype=torch.int64))
    src, dst = torch.cat(src_l), torch.cat(dst_l)
    rowptr, colidx, _ = _csr_from_edges(dst, src, n)
    w = torch.rand(nnz, generator=gen, dtype=torch.float32) if weighted else None
    g = SynthGraph("tiny", n, nnz, F, rowptr.to(device), colidx.to(device),
                   None if w is None else w.to(device), seed=seed)
    return g


def reddit_like(seed: int = 1, device="cpu", scale: float = 1.0, sorted_ids: bool = False,
                F: int = 602) -> SynthGraph:
    """41 planted communities, 80 % of edges inside a community, log-normal(sigma=1) activity of
    the first endpoint, symmetrised; at scale 1: 232,965 vertices and 114,615,892 edges."""
    n0, nnz0, _ = CONFIG_SHAPES["reddit_like"]
    n = max(64, int(round(n0 * math.sqrt(scale))))  # density-preserving shrink
    pairs = max(64, int(round(nnz0 * scale)) // 2)
    C = 41
    gen = _gen(seed, device)
    act = torch.exp(torch.randn(n, generator=gen, device=device, dtype=torch.float64))
    bounds = (torch.arange(C + 1, device=device, dtype=torch.float64) * n / C).floor().long()

    def draw(count):
        a = _sample_cdf(act, count, gen)
        comm = torch.searchsorted(bounds, a, right=True) - 1
        lo_b, size = bounds[comm], bounds[comm + 1] - bounds[comm]
        r = torch.rand(count, generator=gen, device=device, dtype=torch.float64)
        inside = lo_b + (r * size.double()).long().clamp_(max=n - 1)
        r2 = torch.rand(count, generator=gen, device=device, dtype=torch.float64)
        anywhere = (r2 * n).long().clamp_(max=n - 1)
        intra = torch.rand(count, generator=gen, device=device) < 0.8
        return a, torch.where(intra, inside, anywhere)

    lo, hi = _exact_undirected(draw, n, pairs, gen, device)
    rowptr, colidx, _ = _symmetric_csr(lo, hi, n, _relabel(n, sorted_ids, gen, device))
    return SynthGraph("reddit_like", n, int(colidx.numel()), F, rowptr, colidx, None, seed=seed)


def products_like(seed: int = 2, device="cpu", scale: float = 1.0, sorted_ids: bool = False,
                  F: int = 100) -> SynthGraph:
    """Chung-Lu graph: endpoint weights follow a power law with exponent 2.1 (expected degree
    capped at 2e4), symmetrised; at scale 1: 2,449,029 vertices and 123,718,280 edges."""
    n0, nnz0, _ = CONFIG_SHAPES["products_like"]
    n = max(64, int(round(n0 * scale)))
    pairs = max(64, int(round(nnz0 * scale)) // 2)
    gen = _gen(seed, device)
    u = torch.rand(n, generator=gen, device=device, dtype=torch.float64).clamp_(min=1e-12)
    w = u.pow(-1.0 / 1.1)
    mean_deg = 2.0 * pairs / n
    cap = 2.0e4 * scale ** 0.5 if scale < 1.0 else 2.0e4
    for _ in range(8):  # rescale so that the capped weights average to the mean degree
        w = (w * (mean_deg / w.mean())).clamp_(max=max(cap, 2.0 * mean_deg))
    def draw(count):
        return _sample_cdf(w, count, gen), _sample_cdf(w, count, gen)
    lo, hi = _exact_undirected(draw, n, pairs, gen, device)
    rowptr, colidx, _ = _symmetric_csr(lo, hi, n, _relabel(n, sorted_ids, gen, device))
    return SynthGraph("products_like", n, int(colidx.numel()), F, rowptr, colidx, None,
                      seed=seed)


def proteins_like(seed: int = 3, device="cpu", scale: float = 1.0, sorted_ids: bool = False,
                  F: int = 64) -> SynthGraph:
    """8 clustered blocks with 90 % of edges inside a block, uniform endpoints, symmetrised, and
    an 8-wide U(0,1) edge feature shared by the two directions of a pair.  ``edge_w`` is the
    mean of that feature (the reduction to one scalar happens here, outside the library).
    At scale 1: 132,534 vertices and 79,122,504 edges."""
    n0, nnz0, _ = CONFIG_SHAPES["proteins_like"]
    n = max(64, int(round(n0 * math.sqrt(scale))))  # density-preserving shrink
    pairs = max(64, int(round(nnz0 * scale)) // 2)
    C = 8
    gen = _gen(seed, device)
    bounds = (torch.arange(C + 1, device=device, dtype=torch.float64) * n / C).floor().long()

    def draw(count):
        a = (torch.rand(count, generator=gen, device=device, dtype=torch.float64) * n).long()
        a.clamp_(max=n - 1)
        comm = torch.searchsorted(bounds, a, right=True) - 1
        lo_b, size = bounds[comm], bounds[comm + 1] - bounds[comm]
        r = torch.rand(count, generator=gen, device=device, dtype=torch.float64)
        inside = lo_b + (r * size.double()).long().clamp_(max=n - 1)
        r2 = torch.rand(count, generator=gen, device=device, dtype=torch.float64)
        anywhere = (r2 * n).long().clamp_(max=n - 1)
        intra = torch.rand(count, generator=gen, device=device) < 0.9
        return a, torch.where(intra, inside, anywhere)

    lo, hi = _exact_undirected(draw, n, pairs, gen, device)
    rowptr, colidx, pair_of_edge = _symmetric_csr(lo, hi, n,
                                                  _relabel(n, sorted_ids, gen, device))
    pair_feat = torch.rand((lo.numel(), 8), generator=gen, device=device, dtype=torch.float32)
    edge_feat = pair_feat[pair_of_edge]
    del pair_feat
    edge_w = edge_feat.mean(dim=1)
    return SynthGraph("proteins_like", n, int(colidx.numel()), F, rowptr, colidx, edge_w,
                      edge_feat=edge_feat, seed=seed)


def _powerlaw_outdeg_xmin(mean: float, cap: int, expo: float) -> float:
    """x_min such that floor(x_min * U^(-1/expo)) clipped to [0, cap] has the given mean."""
    k = torch.arange(1, cap + 1, dtype=torch.float64)
    lo, hi = 1e-6, float(cap)
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        m = float(torch.clamp((mid / k).pow(expo), max=1.0).sum())
        if m < mean:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def papers_like(seed: int = 4, device="cpu", scale: float = 1.0, F: int = 128,
                parts: int = 8) -> SynthGraph:
    """Directed citation-like graph: out-degree from a power law with exponent 1.9 on
    [0, 1e5] scaled to the exact edge total, destination floor(n*U^2) (in-degree skewed toward
    low ids), no self-loops, duplicate edges kept; at scale 1: 111,059,956 vertices and
    1,615,685,872 edges.  The CSR is assembled in ``parts`` destination ranges to bound the
    sort's memory."""
    n0, nnz0, _ = CONFIG_SHAPES["papers_like"]
    n = max(64, int(round(n0 * scale)))
    nnz = max(64, int(round(nnz0 * scale)))
    gen = _gen(seed, device)
    cap = max(8, min(100_000, n // 8))
    xmin = _powerlaw_outdeg_xmin(nnz / n, cap, 0.9)
    u = torch.rand(n, generator=gen, device=device, dtype=torch.float64).clamp_(min=1e-15)
    deg = (xmin * u.pow(-1.0 / 0.9)).floor().clamp_(max=cap).long()
    del u
    deg = _fix_total(deg, nnz, 0, cap, gen)
    src = torch.repeat_interleave(torch.arange(n, device=device, dtype=torch.int32), deg)
    del deg
    dst = torch.empty(nnz, dtype=torch.int32, device=device)
    step = 1 << 27
    for s in range(0, nnz, step):
        e = min(nnz, s + step)
        r = torch.rand(e - s, generator=gen, device=device, dtype=torch.float64)
        d = (r * r * n).long().clamp_(max=n - 1)
        for _ in range(64):
            bad = torch.nonzero(d == src[s:e]).flatten()
            if bad.numel() == 0:
                break
            r = torch.rand(bad.numel(), generator=gen, device=device, dtype=torch.float64)
            d[bad] = (r * r * n).long().clamp_(max=n - 1)
        dst[s:e] = d.to(torch.int32)
        del r, d
    colidx = torch.empty(nnz, dtype=torch.int32, device=device)
    counts = torch.zeros(n, dtype=torch.int64, device=device)
    filled = 0
    for p in range(parts):
        v0 = int(n * (p / parts) ** 2)
        v1 = n if p == parts - 1 else int(n * ((p + 1) / parts) ** 2)
        if v1 <= v0:
            continue
        sel = torch.nonzero((dst >= v0) & (dst < v1)).flatten()
        d_p, s_p = dst[sel].long(), src[sel].long()
        del sel
        key, _ = torch.sort(d_p * n + s_p)
        del d_p, s_p
        m = key.numel()
        colidx[filled:filled + m] = (key % n).to(torch.int32)
        rows = torch.div(key, n, rounding_mode="floor")
        del key
        counts += torch.bincount(rows, minlength=n)
        del rows
        filled += m
    assert filled == nnz
    del src, dst
    rowptr = torch.zeros(n + 1, dtype=torch.int64, device=device)
    torch.cumsum(counts, 0, out=rowptr[1:])
    return SynthGraph("papers_like", n, nnz, F, rowptr, colidx, None, seed=seed)


def make(name: str, device="cpu", scale: float = 1.0, seed: Optional[int] = None,
         **kw) -> SynthGraph:
    """Build the named workload graph (``CONFIG_SHAPES`` lists the names)."""
    seed = CONFIG_SEEDS[name] if seed is None else seed
    if name == "tiny":
        return tiny(seed=seed, device=device, **kw)
    fn = {"reddit_like": reddit_like, "products_like": products_like,
          "proteins_like": proteins_like, "papers_like": papers_like}[name]
    return fn(seed=seed, device=device, scale=scale, **kw)


def features(n: int, F: int, seed: int, device="cpu", nonneg: bool = False) -> torch.Tensor:
    """N(0,1) fp32 feature (or upstream-gradient) matrix of shape (n, F); with ``nonneg`` its
    absolute values (the sign pattern of activations behind a ReLU, which every layer after the
    first aggregates: all terms of a sum then have one sign and rounding errors do not cancel)."""
    gen = _gen(seed, device)
    out = torch.empty((n, F), device=device, dtype=torch.float32)
    rows = max(1, (1 << 30) // F)
    for s in range(0, n, rows):
        e = min(n, s + rows)
        torch.randn((e - s, F), generator=gen, device=device, dtype=torch.float32, out=out[s:e])
        if nonneg:
            out[s:e].abs_()
    return out
