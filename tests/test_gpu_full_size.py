"""GPU parity at the full sizes of the benchmark workloads, in the launch configuration bench.py
times (default knobs).

Configs 2-4 (Reddit-, Products- and Proteins-like): the CSC is compared with the oracle's stable
counting sort in full, bit for bit, and forward and backward AP are compared with the oracle on
every output element (a chunk of rows at a time).  The variant with implicit self loops is
compared on a sample of output rows (random rows plus the longest ones, which take the
block-per-row path).

Config 5 (Papers-like, 1.6 G edges): the host cannot hold the oracle's inputs, so the CSC is
checked through the properties that define it uniquely (perm is a permutation; keys
non-decreasing along perm; perm increasing inside equal keys; colptr = key boundaries;
rowidx_T = row of perm), evaluated with torch on the GPU, and AP on sampled rows.  Every output
row depends only on its own CSR row (CSC column), so the oracle can compute sampled rows one by
one: it is given the sub-problem made of those rows, with the neighbour ids renumbered into the
compact matrix of the rows they reference.

Set DG_SKIP_FULL_SIZE=1 to skip these (they take a few minutes).
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2104_06700_b200 import binding, synth
from parity_util import assert_within_bound, to_np

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(os.environ.get("DG_SKIP_FULL_SIZE") == "1",
                                 reason="DG_SKIP_FULL_SIZE=1")]
DEV = "cuda"


def sample_segments(ptr, idx, w, seg_ids):
    """Sub-problem of the segments `seg_ids` of a CSR/CSC given as torch tensors on the GPU.
    Returns host arrays (sub_ptr, sub_idx renumbered, sub_w) and the GPU tensor of the distinct
    neighbour ids, in the order of the renumbering."""
    seg = torch.as_tensor(seg_ids, device=ptr.device, dtype=torch.int64)
    lo, hi = ptr[seg], ptr[seg + 1]
    lens = hi - lo
    sub_ptr = torch.zeros(seg.numel() + 1, dtype=torch.int64, device=ptr.device)
    torch.cumsum(lens, 0, out=sub_ptr[1:])
    total = int(sub_ptr[-1])
    # positions of all edges of the sampled segments, segment by segment, in order
    owner = torch.repeat_interleave(torch.arange(seg.numel(), device=ptr.device), lens)
    pos = lo[owner] + (torch.arange(total, device=ptr.device) - sub_ptr[owner])
    nb = idx[pos].long()
    uniq, inv = torch.unique(nb, return_inverse=True)
    sub_w = None if w is None else to_np(w[pos])
    return to_np(sub_ptr), to_np(inv.to(torch.int32)), sub_w, uniq, pos


def pick_rows(ptr, n, count, longest, seed):
    lens = ptr[1:] - ptr[:-1]
    top = torch.topk(lens, min(longest, n)).indices
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    rnd = torch.randperm(n, generator=gen)[:count].to(ptr.device)
    return torch.unique(torch.cat([top, rnd])).cpu().numpy()


def _pad_ptr(ptr, n_sub):
    """Row pointer of a sub-problem extended by empty segments up to n_sub segments."""
    out = np.full(n_sub + 1, ptr[-1], dtype=np.int64)
    out[:len(ptr)] = ptr
    return out


def _pad_rows(M, n_sub):
    out = np.zeros((n_sub, M.shape[1]), dtype=np.float32)
    out[:M.shape[0]] = M
    return out


def check_sampled_self_loops(g, sg, H, G, op, rows, cols):
    """check_sampled for a handle with the "self_loops" attribute.  The sub-problem keeps the k
    sampled segments as vertices 0..k-1 with their own feature rows, followed by the vertices
    they reference (ids renumbered to k + position), so that the oracle finds every sampled
    vertex's own row and in-degree where its definition looks for them."""
    colptr, rowidx_T, w_T, _ = g.dg_graph_get_csc()
    out = g.dg_aggregate_fwd(H, op)
    k = len(rows)
    ridx = torch.as_tensor(rows, device=DEV)
    sp, si, sw, uniq, _ = sample_segments(sg.rowptr, sg.colidx, sg.edge_w, rows)
    n_sub = k + uniq.numel()
    Hs = np.concatenate([to_np(H[ridx]), to_np(H[uniq])])
    ref, mag = oracle.ap_forward(_pad_ptr(sp, n_sub), si + k, sw, Hs, op, rows=np.arange(k),
                                 self_loops=True)
    assert_within_bound(to_np(out[ridx]), ref, mag, "fwd, self loops")
    del out
    dH = g.dg_aggregate_bwd(G, op)
    k = len(cols)
    cidx = torch.as_tensor(cols, device=DEV)
    sp, si, sw, uniq, _ = sample_segments(colptr, rowidx_T, w_T, cols)
    n_sub = k + uniq.numel()
    Gs = np.concatenate([to_np(G[cidx]), to_np(G[uniq])])
    # in-degrees (CSR row lengths) of the sampled vertices, then of the referenced destinations
    deg = np.concatenate([to_np(sg.rowptr[cidx + 1] - sg.rowptr[cidx]),
                          to_np(sg.rowptr[uniq + 1] - sg.rowptr[uniq])])
    rp = np.zeros(n_sub + 1, dtype=np.int64)
    rp[1:] = np.cumsum(deg)
    ref, mag = oracle.ap_backward(rp, _pad_ptr(sp, n_sub), si + k, sw, Gs, op, cols=np.arange(k),
                                  self_loops=True)
    assert_within_bound(to_np(dH[cidx]), ref, mag, "bwd, self loops")


def test_full_size_reddit_like_with_self_loops():
    """The GCN aggregator in one pass (graph attribute "self_loops") at the benchmark's size and
    launch configuration: source-blocked passes, the own row added once."""
    sg = synth.make("reddit_like", device=DEV)
    g = binding.dg_graph_create(sg.n, sg.nnz, sg.rowptr, sg.colidx, sg.edge_w)
    g.dg_graph_set_param("self_loops", 1)
    g.dg_graph_transpose()
    colptr = g.dg_graph_get_csc()[0]
    rows = pick_rows(sg.rowptr, sg.n, 800, 20, 17)
    cols = pick_rows(colptr, sg.n, 800, 20, 18)
    for F in (602, 256):
        H, G = synth.features(sg.n, F, 81, DEV), synth.features(sg.n, F, 82, DEV)
        for op in (binding.DG_OP_MEAN, binding.DG_OP_SUM):
            check_sampled_self_loops(g, sg, H, G, op, rows, cols)


def check_full(g, csr_host, csc_host, H, G, op, elems_per_chunk=1 << 27):
    """Forward on H and backward on G compared with the oracle on EVERY output element, in
    chunks of rows so that the fp64 reference of one chunk stays near 1 GB."""
    rowptr_h, colidx_h, w_h = csr_host
    o_colptr, o_rowidx, o_w = csc_host
    n, F = H.shape
    out = g.dg_aggregate_fwd(H, op)
    dH = g.dg_aggregate_bwd(G, op)
    torch.cuda.synchronize()
    Hh, Gh = to_np(H), to_np(G)
    step = max(1, elems_per_chunk // F)
    worst_f = worst_b = 0.0
    for s in range(0, n, step):
        rows = np.arange(s, min(n, s + step))
        ref, mag = oracle.ap_forward(rowptr_h, colidx_h, w_h, Hh, op, rows=rows)
        worst_f = max(worst_f, assert_within_bound(to_np(out[s:s + step]), ref, mag, "fwd"))
        ref, mag = oracle.ap_backward(rowptr_h, o_colptr, o_rowidx, o_w, Gh, op, cols=rows)
        worst_b = max(worst_b, assert_within_bound(to_np(dH[s:s + step]), ref, mag, "bwd"))
    return worst_f, worst_b


@pytest.mark.parametrize("name,widths,ops", [
    ("reddit_like", (602, 256), (binding.DG_OP_MEAN,)),
    ("products_like", (100,), (binding.DG_OP_SUM, binding.DG_OP_MEAN)),
    ("proteins_like", (8, 64, 256), (binding.DG_OP_SUM,)),
])
def test_full_size_csc_bit_exact_and_every_output_element(name, widths, ops):
    """Configs 2-4 at full size in the benchmark's launch configuration: the CSC bit for bit and
    every element of the forward and the backward result against the oracle."""
    sg = synth.make(name, device=DEV)
    g = binding.dg_graph_create(sg.n, sg.nnz, sg.rowptr, sg.colidx, sg.edge_w)
    g.dg_graph_validate()
    g.dg_graph_transpose()
    torch.cuda.synchronize()
    colptr, rowidx_T, w_T, perm = g.dg_graph_get_csc()
    csr_host = (to_np(sg.rowptr), to_np(sg.colidx), to_np(sg.edge_w))
    o_colptr, o_rowidx, o_w, o_perm = oracle.transpose(*csr_host)
    assert np.array_equal(to_np(colptr), o_colptr), "colptr"
    assert np.array_equal(to_np(rowidx_T), o_rowidx), "rowidx_T"
    assert np.array_equal(to_np(perm).astype(np.int64), o_perm), "perm"
    if sg.edge_w is not None:
        assert to_np(w_T).tobytes() == o_w.tobytes(), "w_T"
    del o_perm
    for F in widths:
        H = synth.features(sg.n, F, 61, DEV)
        G = synth.features(sg.n, F, 62, DEV)
        for op in ops:
            wf, wb = check_full(g, csr_host, (o_colptr, o_rowidx, o_w), H, G, op)
            assert wf <= 1.0 and wb <= 1.0
        del H, G


def _check_csc_properties(sg, colptr, rowidx_T, perm, chunk=1 << 27):
    """The five properties that pin the CSC uniquely, evaluated with torch on the GPU in chunks.
    perm is int32 on the device (edge positions fit 31 bits)."""
    n, nnz = sg.n, sg.nnz
    seen = torch.zeros(nnz, dtype=torch.bool, device=DEV)
    prev_key = torch.full((1,), -1, dtype=torch.int64, device=DEV)
    prev_pos = torch.full((1,), -1, dtype=torch.int64, device=DEV)
    counts = torch.zeros(n, dtype=torch.int64, device=DEV)
    for s in range(0, nnz, chunk):
        e = min(nnz, s + chunk)
        p = perm[s:e].long()
        assert int(p.min()) >= 0 and int(p.max()) < nnz
        seen[p] = True
        key = sg.colidx[p].long()
        k_ext = torch.cat([prev_key, key])
        p_ext = torch.cat([prev_pos, p])
        dk = k_ext[1:] - k_ext[:-1]
        assert bool((dk >= 0).all()), "keys decrease along perm"
        same = dk == 0
        assert bool(((p_ext[1:] - p_ext[:-1])[same] > 0).all()), "unstable order inside a column"
        # rowidx_T[q] is the row r with rowptr[r] <= perm[q] < rowptr[r+1]
        r = torch.searchsorted(sg.rowptr, p, right=True) - 1
        assert torch.equal(r.to(torch.int32), rowidx_T[s:e]), "rowidx_T"
        counts += torch.bincount(key, minlength=n)
        prev_key, prev_pos = key[-1:].clone(), p[-1:].clone()
        del p, key, k_ext, p_ext, dk, same, r
    assert bool(seen.all()), "perm is not a permutation"
    del seen
    expect = torch.zeros(n + 1, dtype=torch.int64, device=DEV)
    torch.cumsum(counts, 0, out=expect[1:])
    assert torch.equal(expect, colptr), "colptr"


def test_papers_like_full_size():
    """111 M vertices, 1.6 G edges, F = 128, sum: CSC by its defining properties, AP on sampled
    rows and columns; two feature buffers as in the benchmark (backward reads the forward's
    input and overwrites its output)."""
    free, total = torch.cuda.mem_get_info()
    if total < 170e9 or free < 160e9:
        pytest.skip("needs a 180 GB device with at least 160 GB free")
    sg = synth.make("papers_like", device=DEV)
    torch.cuda.empty_cache()
    g = binding.dg_graph_create(sg.n, sg.nnz, sg.rowptr, sg.colidx, None)
    g.dg_graph_validate()
    need_csc, need_scratch = g.dg_graph_transpose_workspace()
    csc = torch.empty(need_csc, dtype=torch.uint8, device=DEV)
    scratch = torch.empty(need_scratch, dtype=torch.uint8, device=DEV)
    g.dg_graph_transpose(csc, scratch)
    torch.cuda.synchronize()
    del scratch
    torch.cuda.empty_cache()
    colptr, rowidx_T, w_T, perm = g.dg_graph_get_csc()
    assert w_T is None
    _check_csc_properties(sg, colptr, rowidx_T, perm)
    torch.cuda.empty_cache()
    F = 128
    H = synth.features(sg.n, F, 71, DEV)
    out = torch.empty_like(H)
    rows = pick_rows(sg.rowptr, sg.n, 3000, 30, 9)
    cols = pick_rows(colptr, sg.n, 3000, 30, 10)
    g.dg_aggregate_fwd(H, binding.DG_OP_SUM, out=out)
    sp, si, _, uniq, _ = sample_segments(sg.rowptr, sg.colidx, None, rows)
    n_sub = max(len(rows), uniq.numel())
    ref, mag = oracle.ap_forward(_pad_ptr(sp, n_sub), si, None, _pad_rows(to_np(H[uniq]), n_sub),
                                 oracle.OP_SUM, rows=np.arange(len(rows)))
    assert_within_bound(to_np(out[torch.as_tensor(rows, device=DEV)]), ref, mag, "fwd")
    g.dg_aggregate_bwd(H, binding.DG_OP_SUM, dH=out)
    sp, si, _, uniq, _ = sample_segments(colptr, rowidx_T, None, cols)
    n_sub = max(len(cols), uniq.numel())
    rp = np.zeros(n_sub + 1, dtype=np.int64)          # sum: the divisor is not used
    ref, mag = oracle.ap_backward(rp, _pad_ptr(sp, n_sub), si, None,
                                  _pad_rows(to_np(H[uniq]), n_sub), oracle.OP_SUM,
                                  cols=np.arange(len(cols)))
    assert_within_bound(to_np(out[torch.as_tensor(cols, device=DEV)]), ref, mag, "bwd")


def test_full_size_products_like_hub_first():
    """dg_graph_reorder at the benchmark's size: the renamed CSR bit for bit against the oracle,
    then forward and backward AP on the renamed handle (the launch configuration the bench times
    for its hub-first records) against the oracle of the ORIGINAL graph, on every element."""
    sg = synth.make("products_like", device=DEV)
    g = binding.dg_graph_create(sg.n, sg.nnz, sg.rowptr, sg.colidx, sg.edge_w)
    r = g.dg_graph_reorder(binding.DG_ORDER_OUT_DEGREE)
    torch.cuda.synchronize()
    rp, ci = to_np(sg.rowptr), to_np(sg.colidx)
    order = oracle.order_by_degree(np.bincount(ci, minlength=sg.n).astype(np.int64))
    assert np.array_equal(to_np(r.new_of_old), order), "new_of_old"
    rp2, ci2, _, pos2 = oracle.relabel(rp, ci, None, order)
    assert np.array_equal(to_np(r.rowptr), rp2), "rowptr"
    assert np.array_equal(to_np(r.colidx), ci2), "colidx"
    assert np.array_equal(to_np(r.pos).astype(np.int64), pos2), "pos"
    del rp2, ci2, pos2
    r.dg_graph_transpose()
    colptr, rowidx_T, _, _ = oracle.transpose(rp, ci, None)
    F = 100
    H = synth.features(sg.n, F, 91, DEV)
    G = synth.features(sg.n, F, 92, DEV)
    H2 = binding.dg_permute_rows(r.new_of_old, H)
    G2 = binding.dg_permute_rows(r.new_of_old, G)
    for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
        out = binding.dg_permute_rows(r.new_of_old, r.dg_aggregate_fwd(H2, op), to_old=True)
        dH = binding.dg_permute_rows(r.new_of_old, r.dg_aggregate_bwd(G2, op), to_old=True)
        torch.cuda.synchronize()
        ref, mag = oracle.ap_forward(rp, ci, None, to_np(H), op)
        assert_within_bound(to_np(out), ref, mag, "fwd, hub-first")
        ref, mag = oracle.ap_backward(rp, colptr, rowidx_T, None, to_np(G), op)
        assert_within_bound(to_np(dH), ref, mag, "bwd, hub-first")


def _row_sub_problem(ptr, idx, rows):
    """The CSR rows `rows` as a graph of their own for the oracle: row i of the sub-problem is
    rows[i], its sources are renumbered into `uniq`, and `pos` gives the position of every
    sub-problem edge in the full arrays.  Padded with empty rows so that row and source ids
    share one range."""
    sp, si, _, uniq, pos = sample_segments(ptr, idx, None, rows)
    n_sub = max(len(rows), uniq.numel())
    return _pad_ptr(sp, n_sub), si, uniq, pos, n_sub


def _column_sub_problem(g, cols):
    """The out-edges of the source vertices `cols` as a CSR graph of their own: its rows are the
    destinations they reach (`dests`, renumbered), its sources are 0..len(cols)-1, the edges of
    a row keep their CSR order, and `k_full` gives the CSR position of every edge in the full
    graph (ascending, because CSR positions grow with the row)."""
    colptr, rowidx_T, _, perm = g.dg_graph_get_csc()
    sp, si, _, dests, posT = sample_segments(colptr, rowidx_T, None, cols)
    owner = np.repeat(np.arange(len(cols), dtype=np.int32), np.diff(sp))
    k_full = to_np(perm[posT]).astype(np.int64)
    order = np.argsort(k_full, kind="stable")          # CSR order = (row, position in row)
    k_full, dest_sub, src_sub = k_full[order], si[order], owner[order]
    assert np.all(np.diff(dest_sub) >= 0)
    n_sub = max(len(cols), dests.numel())
    rp = np.zeros(n_sub + 1, dtype=np.int64)
    np.add.at(rp, dest_sub.astype(np.int64) + 1, 1)
    return np.cumsum(rp), src_sub, dests, k_full, n_sub


@pytest.mark.parametrize("name,F,fE_cols", [("reddit_like", 602, 1), ("products_like", 100, 1),
                                            ("proteins_like", 64, 64)])
def test_full_size_general_calls(name, F, fE_cols):
    """dg_ap_fwd / dg_ap_bwd (copylhs / max with arg, mul / sum with edge features) and
    dg_aggregate_edge_grad at full size with default knobs, i.e. in the launch shapes the
    benchmark times: feature slices x source blocks on the Reddit-like graph, block-per-row heavy
    rows and columns on the Products-like one, the full |E| x F edge-feature stream on the
    Proteins-like one.  Every output row (edge) depends on its own CSR row (CSC column) only, so
    the oracle computes sampled rows and columns as sub-problems: random ones plus the longest,
    which take the block-per-row path.  The extrema and their arg are compared bit for bit; the
    vertex gradient of max is also checked through the identity that every non-empty (v, j)
    hands its dO to exactly one source: sum_u dV[u][j] = sum_{v: arg >= 0} dO[v][j]."""
    sg = synth.make(name, device=DEV)
    g = binding.dg_graph_create(sg.n, sg.nnz, sg.rowptr, sg.colidx, None)
    g.dg_graph_validate()
    g.dg_graph_transpose()
    colptr = g.dg_graph_get_csc()[0]
    H = synth.features(sg.n, F, 61, DEV)
    G = synth.features(sg.n, F, 62, DEV)
    rows = pick_rows(sg.rowptr, sg.n, 150, 12, 63)
    cols = pick_rows(colptr, sg.n, 60, 3, 64)
    ridx, cidx = torch.as_tensor(rows, device=DEV), torch.as_tensor(cols, device=DEV)
    rp_r, ci_r, uniq_r, pos_r, n_r = _row_sub_problem(sg.rowptr, sg.colidx, rows)
    rp_c, ci_c, dests_c, k_c, n_c = _column_sub_problem(g, cols)
    H_r = _pad_rows(to_np(H[uniq_r]), n_r)
    G_r = _pad_rows(to_np(G[ridx]), n_r)
    G_c = _pad_rows(to_np(G[dests_c]), n_c)
    H_c = _pad_rows(to_np(H[cidx]), n_c)
    k = len(rows)
    assert k >= 150 and pos_r.numel() > 1000 and len(k_c) > 1000    # real sub-problems

    # -- copylhs / max: extrema and arg bit-exact on the sampled rows
    out, arg = g.dg_ap_fwd(H, None, binding.DG_BIN_COPY_LHS, binding.DG_RED_MAX)
    torch.cuda.synchronize()
    ref, _, oarg = oracle.general_forward(rp_r, ci_r, H_r, None, binding.DG_BIN_COPY_LHS,
                                          binding.DG_RED_MAX)
    assert np.array_equal(to_np(out[ridx]).astype(np.float64), ref[:k]), "max"
    pos_np = to_np(pos_r).astype(np.int64)
    want_arg = np.where(oarg[:k] >= 0, pos_np[np.maximum(oarg[:k], 0)], -1)
    assert np.array_equal(to_np(arg[ridx]).astype(np.int64), want_arg), "arg"
    assert (want_arg >= 0).mean() > 0.5
    # -- its vertex gradient on the sampled columns, given that arg
    dV, _ = g.dg_ap_bwd(G, H, None, binding.DG_BIN_COPY_LHS, binding.DG_RED_MAX, arg=arg)
    torch.cuda.synchronize()
    arg_c = to_np(arg[dests_c]).astype(np.int64)             # full positions -> sub positions
    at = np.minimum(np.searchsorted(k_c, arg_c), len(k_c) - 1)
    arg_sub = np.full((n_c, F), -1, dtype=np.int64)
    arg_sub[:arg_c.shape[0]] = np.where(k_c[at] == arg_c, at, -1)
    assert (arg_sub >= 0).any()                      # some extrema do come from the sampled sources
    odV, omV, _, _ = oracle.general_backward(rp_c, ci_c, H_c, None, binding.DG_BIN_COPY_LHS,
                                             binding.DG_RED_MAX, arg_sub, G_c)
    assert_within_bound(to_np(dV[cidx]), odV[:len(cols)], omV[:len(cols)], "dV of max")
    routed = torch.where(arg >= 0, G, torch.zeros_like(G)).double()
    total, scale = routed.sum(0), routed.abs().sum(0)
    assert bool(((dV.double().sum(0) - total).abs() <= 1e-5 * scale + 1e-7).all()), "sum of dV"
    del out, arg, dV, routed

    # -- mul / sum with edge features: forward, dV and dE
    fE = torch.rand((sg.nnz, fE_cols), device=DEV, dtype=torch.float32) + 0.5
    out, _ = g.dg_ap_fwd(H, fE, binding.DG_BIN_MUL, binding.DG_RED_SUM)
    dV, dE = g.dg_ap_bwd(G, H, fE, binding.DG_BIN_MUL, binding.DG_RED_SUM)
    torch.cuda.synchronize()
    fE_r = to_np(fE[pos_r])
    ref, mag, _ = oracle.general_forward(rp_r, ci_r, H_r, fE_r, binding.DG_BIN_MUL,
                                         binding.DG_RED_SUM)
    assert_within_bound(to_np(out[ridx]), ref[:k], mag[:k], "mul/sum")
    _, _, odE, omE = oracle.general_backward(rp_r, ci_r, H_r, fE_r, binding.DG_BIN_MUL,
                                             binding.DG_RED_SUM, None, G_r, want_dV=False)
    assert_within_bound(to_np(dE[pos_r]), odE, omE, "dE of mul/sum")
    fE_c = to_np(fE[torch.as_tensor(k_c, device=DEV)])
    odV, omV, _, _ = oracle.general_backward(rp_c, ci_c, H_c, fE_c, binding.DG_BIN_MUL,
                                             binding.DG_RED_SUM, None, G_c, want_dE=False)
    assert_within_bound(to_np(dV[cidx]), odV[:len(cols)], omV[:len(cols)], "dV of mul/sum")
    del out, dV, dE, fE

    # -- gradient with respect to scalar edge weights of the mean
    dW = g.dg_aggregate_edge_grad(H, G, binding.DG_OP_MEAN)
    torch.cuda.synchronize()
    ref, mag = oracle.edge_weight_grad(rp_r, ci_r, H_r, G_r, binding.DG_OP_MEAN)
    assert_within_bound(to_np(dW[pos_r]), ref, mag, "dW")
