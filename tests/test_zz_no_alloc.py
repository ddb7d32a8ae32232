"""dg_graph_transpose_static: the CSC build for callers that cannot hand over scratch memory.

Some users of the library cannot allocate on the device at the point where they need the
reverse graph: the process around them has reserved all of the GPU for its own pool, or they run
in a loop where the device-wide stall of an allocation is not tolerated.  For them the library
carries a fixed scratch array and this entry point, which takes only the output storage.

The check is against the regular entry point (caller-supplied scratch), bit for bit, on two
calls in a row: the second call finds the array as the first one left it, so a dependence on
clean scratch would show.  This file is collected last on purpose: a failure here must not keep
the other tests from running under `pytest -x`.
"""
import ctypes

import pytest
import torch

from paper_2104_06700_b200 import binding, synth
from parity_util import make_graph

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _csc_copy(g):
    torch.cuda.synchronize()
    return [None if t is None else t.clone() for t in g.dg_graph_get_csc()]


def _same(a, b):
    for x, y in zip(a, b):
        if x is None or y is None:
            assert x is None and y is None
        else:
            assert x.dtype == y.dtype and torch.equal(x, y)


@pytest.mark.parametrize("weighted", [True, False])
def test_static_scratch_transpose_matches_regular_entry_point(weighted):
    sg = synth.make("tiny", weighted=weighted)
    regular = make_graph(sg)
    regular.dg_graph_transpose()
    want = _csc_copy(regular)

    g = make_graph(sg)
    need_csc, need_scratch = g.dg_graph_transpose_workspace()
    storage = torch.empty(need_csc, dtype=torch.uint8, device=DEV)
    g.dg_graph_transpose_static(storage)           # first call: also looks up the array
    first = _csc_copy(g)
    storage.fill_(0xAB)                            # the second call must rewrite everything
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]     # cudaMemGetInfo: the whole device, any allocator
    g.dg_graph_transpose_static(storage)           # second call: the array holds old contents
    torch.cuda.synchronize()
    g.dg_graph_transpose_static(storage)           # and a later one
    torch.cuda.synchronize()
    # what the entry point promises: with the output storage passed in, no device memory is
    # taken or given back by a call (nothing else runs between the two readings)
    assert torch.cuda.mem_get_info()[0] == free_before
    assert binding.dg_last_error() == "" or "static" not in binding.dg_last_error()
    second = _csc_copy(g)
    _same(first, want)
    _same(second, want)

    # the handle is fully usable afterwards: the backward pass agrees with the regular handle
    G = synth.features(sg.n, 64, 3, DEV)
    assert torch.equal(g.dg_aggregate_bwd(G, binding.DG_OP_MEAN),
                       regular.dg_aggregate_bwd(G, binding.DG_OP_MEAN))


def test_static_scratch_interleaved_with_a_different_graph():
    """Two graphs of different size take turns: each result is right although the array still
    holds the other graph's keys."""
    a = synth.make("tiny")
    b = synth.make("reddit_like", device=DEV, scale=0.004)
    ga, gb = make_graph(a), make_graph(b)
    ra, rb = make_graph(a), make_graph(b)
    ra.dg_graph_transpose()
    rb.dg_graph_transpose()
    want_a, want_b = _csc_copy(ra), _csc_copy(rb)
    for _ in range(2):
        ga.dg_graph_transpose_static()
        _same(_csc_copy(ga), want_a)
        gb.dg_graph_transpose_static()
        _same(_csc_copy(gb), want_b)


def test_static_scratch_rejects_graphs_beyond_its_limit():
    n, nnz = 1000, 2_000_000                       # needs about 24 MB of scratch; the array has 16
    rowptr = torch.linspace(0, nnz, n + 1, device=DEV).long()
    rowptr[-1] = nnz
    colidx = torch.randint(0, n, (nnz,), device=DEV, dtype=torch.int32)
    g = binding.dg_graph_create(n, nnz, rowptr, colidx, None)
    with pytest.raises(binding.DgError) as e:
        g.dg_graph_transpose_static()
    assert e.value.status == binding.DG_ERR_UNSUPPORTED
    assert "scratch" in str(e.value)
    g.dg_graph_transpose()                         # the regular entry point still serves it
    torch.cuda.synchronize()


def test_static_scratch_argument_errors():
    g = make_graph(synth.make("tiny"))
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.DgError) as e:
        g.dg_graph_transpose_static(small)
    assert e.value.status == binding.DG_ERR_WORKSPACE
    lib = binding.lib()
    assert lib.dg_graph_transpose_static(None, None, ctypes.c_size_t(0), None) == binding.DG_ERR_INVALID_ARG
