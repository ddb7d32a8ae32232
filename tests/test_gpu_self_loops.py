"""GPU parity of the "self_loops" graph attribute (the GCN aggregator of Section 5.1 in one pass:
own row joins the sum, the mean divides by in-degree + 1) against the CPU oracle, element by
element, over the launch shapes the plain operators are tested on: light rows of every lane
layout, block-per-row rows, source-blocked passes, bf16 storage, the host entry point.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_06700_b200 import binding, synth
from parity_util import (assert_within_bound, check_fwd_bwd, check_transpose, make_graph, to_np)

pytestmark = pytest.mark.gpu
DEV = "cuda"
OPS = (binding.DG_OP_SUM, binding.DG_OP_MEAN)


def host_csr(sg):
    return (to_np(sg.rowptr), to_np(sg.colidx), to_np(sg.edge_w))


def looped(sg):
    g = make_graph(sg)
    g.dg_graph_set_param("self_loops", 1)
    return g


@pytest.mark.parametrize("F", [64, 8, 100, 602, 256, 1, 3, 130])
@pytest.mark.parametrize("weighted", [True, False])
def test_tiny_every_lane_layout(F, weighted):
    sg = synth.make("tiny", weighted=weighted)
    g = looped(sg)
    csc = check_transpose(g, *host_csr(sg))
    H = synth.features(sg.n, F, 300 + F, DEV)
    G = synth.features(sg.n, F, 400 + F, DEV)
    for op in OPS:
        check_fwd_bwd(g, host_csr(sg), H, G, op, csc, self_loops=True)


def test_isolated_vertices_keep_their_own_row_bit_for_bit():
    """in-degree 0: (0 + h_v) / 1 = h_v exactly, in both directions; the plain operators give
    zeros there."""
    n, F = 3000, 72
    rows = [[] if v % 3 else [(v + 1) % n, (v + 7) % n] for v in range(n)]
    rowptr = np.zeros(n + 1, dtype=np.int64)
    rowptr[1:] = np.cumsum([len(r) for r in rows])
    colidx = np.asarray([u for r in rows for u in r], dtype=np.int32)
    g = binding.dg_graph_create(n, len(colidx), torch.as_tensor(rowptr, device=DEV),
                                torch.as_tensor(colidx, device=DEV), None)
    g.dg_graph_set_param("self_loops", 1)
    csc = check_transpose(g, rowptr, colidx, None)
    H, G = synth.features(n, F, 1, DEV), synth.features(n, F, 2, DEV)
    for op in OPS:
        check_fwd_bwd(g, (rowptr, colidx, None), H, G, op, csc, self_loops=True)
        out = g.dg_aggregate_fwd(H, op)
        empty = torch.as_tensor([v for v in range(n) if v % 3], device=DEV)
        assert torch.equal(out[empty], H[empty])
    # a vertex nobody points to and that has no in-edges either: backward returns s_u * dOut[u]
    no_out = np.setdiff1d(np.arange(n), colidx)
    lone = torch.as_tensor([u for u in no_out if u % 3], device=DEV)
    assert lone.numel() > 0
    assert torch.equal(g.dg_aggregate_bwd(G, binding.DG_OP_MEAN)[lone], G[lone])


@pytest.mark.parametrize("F", [64, 602])
def test_star_graph_block_per_row_path(F):
    """One destination with 5000 in-edges and one source with 5000 out-edges: both take the
    block-per-row path, whose epilogue adds the own row."""
    n = 6000
    rows = [[] for _ in range(n)]
    rows[0] = list(range(1, 5001))                    # heavy row
    for v in range(1, 5001):
        rows[v] = [5500]                              # heavy column 5500
    rowptr = np.zeros(n + 1, dtype=np.int64)
    rowptr[1:] = np.cumsum([len(r) for r in rows])
    colidx = np.asarray([u for r in rows for u in r], dtype=np.int32)
    w = np.random.default_rng(3).random(len(colidx)).astype(np.float32)
    g = binding.dg_graph_create(n, len(colidx), torch.as_tensor(rowptr, device=DEV),
                                torch.as_tensor(colidx, device=DEV), torch.as_tensor(w, device=DEV))
    g.dg_graph_set_param("self_loops", 1)
    csc = check_transpose(g, rowptr, colidx, w)
    H, G = synth.features(n, F, 5, DEV), synth.features(n, F, 6, DEV)
    for op in OPS:
        check_fwd_bwd(g, (rowptr, colidx, w), H, G, op, csc, self_loops=True)


@pytest.mark.parametrize("blocks", [1, 4, 16])
def test_source_blocked_passes_add_the_own_row_once(blocks):
    sg = synth.make("reddit_like", device=DEV, scale=0.02)
    g = looped(sg)
    g.dg_graph_set_param("source_blocks", blocks)
    g.dg_graph_set_param("heavy_threshold", 256)      # some rows take the block-per-row path
    csc = check_transpose(g, *host_csr(sg))
    for F in (602, 64, 7):
        H = synth.features(sg.n, F, 41, DEV)
        G = synth.features(sg.n, F, 42, DEV)
        for op in OPS:
            check_fwd_bwd(g, host_csr(sg), H, G, op, csc, self_loops=True)


@pytest.mark.parametrize("name,scale,F", [("products_like", 0.05, 100), ("papers_like", 0.002, 128),
                                          ("proteins_like", 0.05, 64)])
def test_scaled_workloads(name, scale, F):
    sg = synth.make(name, device=DEV, scale=scale)
    g = looped(sg)
    csc = check_transpose(g, *host_csr(sg))
    H, G = synth.features(sg.n, F, 51, DEV), synth.features(sg.n, F, 52, DEV)
    for op in OPS:
        check_fwd_bwd(g, host_csr(sg), H, G, op, csc, self_loops=True)


def test_bf16_storage():
    sg = synth.make("tiny")
    g = looped(sg)
    o_colptr, o_rowidx, o_w = check_transpose(g, *host_csr(sg))
    rowptr_h, colidx_h, w_h = host_csr(sg)
    for F in (64, 100, 256):
        Hb = synth.features(sg.n, F, 7, DEV).to(torch.bfloat16)
        Gb = synth.features(sg.n, F, 8, DEV).to(torch.bfloat16)
        for op in OPS:
            out = g.dg_aggregate_fwd_bf16(Hb, op)
            dH = g.dg_aggregate_bwd_bf16(Gb, op)
            ref, mag = oracle.ap_forward(rowptr_h, colidx_h, w_h, to_np(Hb.float()), op,
                                         self_loops=True)
            assert_within_bound(to_np(out), ref, mag, f"fwd bf16 F={F}")
            ref, mag = oracle.ap_backward(rowptr_h, o_colptr, o_rowidx, o_w, to_np(Gb.float()), op,
                                          self_loops=True)
            assert_within_bound(to_np(dH), ref, mag, f"bwd bf16 F={F}")


def test_attribute_changed_after_the_transpose():
    """The mean's backward factors are tabulated by the transpose: a later change of the
    attribute is refused there, the other three passes follow the attribute at once."""
    sg = synth.make("tiny")
    g = make_graph(sg)
    csc = check_transpose(g, *host_csr(sg))
    H = synth.features(sg.n, 32, 1, DEV)
    plain_sum = g.dg_aggregate_bwd(H, binding.DG_OP_SUM).clone()
    g.dg_graph_set_param("self_loops", 1)
    assert g.dg_graph_get_param("self_loops") == 1
    with pytest.raises(binding.DgError) as e:
        g.dg_aggregate_bwd(H, binding.DG_OP_MEAN)
    assert e.value.status == binding.DG_ERR_NOT_TRANSPOSED
    ref, mag = oracle.ap_backward(to_np(sg.rowptr), *csc, to_np(H), oracle.OP_SUM, self_loops=True)
    looped_sum = g.dg_aggregate_bwd(H, binding.DG_OP_SUM)
    assert_within_bound(to_np(looped_sum), ref, mag, "sum backward right after the change")
    assert not torch.allclose(looped_sum, plain_sum)
    g.dg_graph_transpose()
    check_fwd_bwd(g, host_csr(sg), H, H.flip(0).contiguous(), binding.DG_OP_MEAN, csc,
                  self_loops=True)
    with pytest.raises(binding.DgError):
        g.dg_graph_set_param("self_loops", 2)


def test_host_entry_point_in_column_chunks():
    sg = synth.make("tiny")
    g = looped(sg)
    o_colptr, o_rowidx, o_w = check_transpose(g, *host_csr(sg))
    F = 602
    H = synth.features(sg.n, F, 11, "cpu").pin_memory()
    G = synth.features(sg.n, F, 12, "cpu").pin_memory()
    out, dH = torch.empty_like(H).pin_memory(), torch.empty_like(G).pin_memory()
    ws = torch.empty(g.dg_aggregate_host_workspace(F), dtype=torch.uint8, device=DEV)
    g.dg_aggregate_host(H, G, binding.DG_OP_MEAN, out, dH, ws)
    torch.cuda.synchronize()
    ref, mag = oracle.ap_forward(*host_csr(sg), H.numpy(), oracle.OP_MEAN, self_loops=True)
    assert_within_bound(out.numpy(), ref, mag, "host fwd")
    ref, mag = oracle.ap_backward(to_np(sg.rowptr), o_colptr, o_rowidx, o_w, G.numpy(),
                                  oracle.OP_MEAN, self_loops=True)
    assert_within_bound(dH.numpy(), ref, mag, "host bwd")
