"""bf16 storage of the gathered matrix (fp32 products and sums, fp32 output): same oracle, same
bound.  A bf16 value converts to fp32 exactly, so the oracle is simply given the bf16-rounded
matrix as fp32."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_06700_b200 import binding, synth
from parity_util import assert_within_bound, check_transpose, make_graph, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda"


def host_csr(sg):
    return (to_np(sg.rowptr), to_np(sg.colidx), to_np(sg.edge_w))


def check_bf16(g, sg_host, csc_host, Hb, Gb, op):
    rowptr_h, colidx_h, w_h = sg_host
    o_colptr, o_rowidx, o_w = csc_host
    out = g.dg_aggregate_fwd_bf16(Hb, op)
    dH = g.dg_aggregate_bwd_bf16(Gb, op)
    torch.cuda.synchronize()
    assert out.dtype == torch.float32 and dH.dtype == torch.float32
    ref, mag = oracle.ap_forward(rowptr_h, colidx_h, w_h, to_np(Hb.float()), op)
    assert_within_bound(to_np(out), ref, mag, "bf16 fwd")
    ref, mag = oracle.ap_backward(rowptr_h, o_colptr, o_rowidx, o_w, to_np(Gb.float()), op)
    assert_within_bound(to_np(dH), ref, mag, "bf16 bwd")
    return out, dH


@pytest.mark.parametrize("F", [64, 8, 104, 602, 256, 130, 6, 2, 1032, 100])
@pytest.mark.parametrize("weighted", [True, False])
def test_tiny_bf16(F, weighted):
    sg = synth.make("tiny", weighted=weighted)
    g = make_graph(sg)
    g.dg_graph_set_param("heavy_threshold", 128)
    csc = check_transpose(g, *host_csr(sg))
    Hb = synth.features(sg.n, F, 500 + F, DEV).to(torch.bfloat16)
    Gb = synth.features(sg.n, F, 600 + F, DEV).to(torch.bfloat16)
    for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
        out, dH = check_bf16(g, host_csr(sg), csc, Hb, Gb, op)
        # the fp32 entry point on the same values gives the same sums up to summation order
        out32 = g.dg_aggregate_fwd(Hb.float(), op)
        assert torch.allclose(out, out32, rtol=1e-4, atol=1e-5)


@pytest.mark.parametrize("blocks", [0, 4])
def test_bf16_with_source_blocks(blocks):
    sg = synth.make("reddit_like", device=DEV, scale=0.02)
    g = make_graph(sg)
    g.dg_graph_set_param("source_blocks", blocks)
    g.dg_graph_set_param("l2_budget_mb", 1)
    csc = check_transpose(g, *host_csr(sg))
    for F in (602, 256):
        Hb = synth.features(sg.n, F, 1, DEV).to(torch.bfloat16)
        Gb = synth.features(sg.n, F, 2, DEV).to(torch.bfloat16)
        check_bf16(g, host_csr(sg), csc, Hb, Gb, binding.DG_OP_MEAN)


def test_bf16_unaligned_and_odd_width():
    sg = synth.make("tiny", weighted=False)
    g = make_graph(sg)
    csc = check_transpose(g, *host_csr(sg))
    # a matrix that starts 2 elements (4 bytes) into an allocation: 4-byte loads
    F = 64
    base = synth.features(sg.n * F + 8, 1, 9, DEV).flatten().to(torch.bfloat16)
    Hb = base[2:2 + sg.n * F].view(sg.n, F)
    out = g.dg_aggregate_fwd_bf16(Hb, binding.DG_OP_SUM)
    torch.cuda.synchronize()
    ref, mag = oracle.ap_forward(*host_csr(sg), to_np(Hb.float().contiguous()), oracle.OP_SUM)
    assert_within_bound(to_np(out), ref, mag, "bf16 unaligned")
    odd = synth.features(sg.n, 7, 1, DEV).to(torch.bfloat16)
    with pytest.raises(binding.DgError) as e:
        g.dg_aggregate_fwd_bf16(odd, binding.DG_OP_SUM)
    assert e.value.status == binding.DG_ERR_UNSUPPORTED
    del csc
