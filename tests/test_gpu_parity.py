"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

fp32 outputs must satisfy |gpu - ref| <= 1e-5 * sum|terms| + 1e-7 per element; the CSC arrays
(colptr, rowidx_T, perm) and the copied weights must be bit-exact.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_06700_b200 import binding, synth
from parity_util import (assert_within_bound, check_fwd_bwd, check_transpose, make_graph, to_np)

pytestmark = pytest.mark.gpu
DEV = "cuda"


def host_csr(sg):
    return (to_np(sg.rowptr), to_np(sg.colidx), to_np(sg.edge_w))


def csr_graph(n, rows, device=DEV, weights=None):
    rowptr = np.zeros(n + 1, dtype=np.int64)
    col = []
    for v in range(n):
        col.extend(rows[v])
        rowptr[v + 1] = len(col)
    colidx = np.asarray(col, dtype=np.int32)
    w = None if weights is None else torch.as_tensor(weights, dtype=torch.float32, device=device)
    g = binding.dg_graph_create(n, len(col), torch.as_tensor(rowptr, device=device),
                                torch.as_tensor(colidx, device=device), w)
    return g, rowptr, colidx


# ------------------------------------------------------------------ tiny: every combination
@pytest.fixture(scope="module")
def tiny():
    return synth.make("tiny")


@pytest.mark.parametrize("weighted", [True, False])
def test_tiny_transpose_bit_exact(tiny, weighted):
    sg = tiny if weighted else synth.make("tiny", weighted=False)
    g = make_graph(sg)
    g.dg_graph_validate()
    check_transpose(g, *host_csr(sg))


@pytest.mark.parametrize("shift", [1, 2, 3])
def test_transpose_with_colidx_not_16_byte_aligned(tiny, shift):
    """The caller's colidx only has to be 4-byte aligned: the first radix pass reads it in place
    and must not use 16-byte loads on it.  Several tiles and a ragged last one."""
    sg = tiny
    rowptr = sg.rowptr.to(DEV).clone()
    rowptr[sg.n] = rowptr[sg.n - 1]            # last row emptied: the edge count gets ragged
    nnz = int(rowptr[sg.n])
    store = torch.empty(nnz + 4, dtype=torch.int32, device=DEV)
    colidx = store[shift:shift + nnz]
    colidx.copy_(sg.colidx[:nnz])
    w = sg.edge_w[:nnz].to(DEV).clone()
    assert colidx.data_ptr() % 16 == 4 * shift and nnz > 3 * 4096 and nnz % 4096 != 0
    g = binding.dg_graph_create(sg.n, nnz, rowptr, colidx, w)
    g.dg_graph_validate()
    check_transpose(g, to_np(rowptr), to_np(colidx), to_np(w))


@pytest.mark.parametrize("F", [64, 8, 100, 602, 256, 128, 1, 3, 6, 130, 1028])
@pytest.mark.parametrize("op", [binding.DG_OP_SUM, binding.DG_OP_MEAN])
@pytest.mark.parametrize("weighted", [True, False])
def test_tiny_forward_backward(tiny, F, op, weighted):
    sg = tiny if weighted else synth.make("tiny", weighted=False)
    g = make_graph(sg)
    csc = check_transpose(g, *host_csr(sg))
    H = synth.features(sg.n, F, 100 + F, DEV)
    G = synth.features(sg.n, F, 200 + F, DEV)
    check_fwd_bwd(g, host_csr(sg), H, G, op, csc)


def test_tiny_deterministic_bits(tiny):
    g = make_graph(tiny)
    g.dg_graph_transpose()
    H = synth.features(tiny.n, 64, 1, DEV)
    a = g.dg_aggregate_fwd(H, binding.DG_OP_MEAN).clone()
    b = g.dg_aggregate_fwd(H, binding.DG_OP_MEAN)
    c = g.dg_aggregate_bwd(H, binding.DG_OP_MEAN).clone()
    d = g.dg_aggregate_bwd(H, binding.DG_OP_MEAN)
    assert torch.equal(a, b) and torch.equal(c, d)


@pytest.mark.parametrize("slice_f,heavy,rows_per_block,heavy_blocks",
                         [(16, 64, 1, 0), (32, 64, 8, 1), (0, 128, 64, 3), (600, 1024, 32, 0),
                          (4, 4096, 3, 2)])
def test_tiny_launch_shapes(tiny, slice_f, heavy, rows_per_block, heavy_blocks):
    """Feature slicing, the heavy-segment path and the block shape change the launch, not the
    result (columns of the tiny graph reach 488 entries, above the lowered heavy threshold)."""
    g = make_graph(tiny)
    g.dg_graph_set_param("heavy_threshold", heavy)
    g.dg_graph_set_param("slice_features", slice_f)
    g.dg_graph_set_param("rows_per_block", rows_per_block)
    g.dg_graph_set_param("heavy_blocks_per_sm", heavy_blocks)
    assert g.dg_graph_get_param("heavy_threshold") == heavy
    csc = check_transpose(g, *host_csr(tiny))
    for F in (64, 602, 10):
        H = synth.features(tiny.n, F, 5, DEV)
        G = synth.features(tiny.n, F, 6, DEV)
        check_fwd_bwd(g, host_csr(tiny), H, G, binding.DG_OP_MEAN, csc)


def test_unaligned_feature_pointers(tiny):
    """Matrices that start 4 or 8 bytes off a 16-byte boundary take the narrower vector paths."""
    g = make_graph(tiny)
    csc = check_transpose(g, *host_csr(tiny))
    for F, shift in ((64, 1), (64, 2), (602, 1)):
        base = synth.features(tiny.n * F + 4, 1, 9, DEV).flatten()
        H = base[shift:shift + tiny.n * F].view(tiny.n, F)
        G = synth.features(tiny.n, F, 10, DEV)
        outbuf = torch.empty(tiny.n * F + 4, device=DEV)
        out = outbuf[shift:shift + tiny.n * F].view(tiny.n, F)
        g.dg_aggregate_fwd(H, binding.DG_OP_SUM, out=out)
        torch.cuda.synchronize()
        ref, mag = oracle.ap_forward(*host_csr(tiny), to_np(H.contiguous()), oracle.OP_SUM)
        assert_within_bound(to_np(out), ref, mag, f"unaligned F={F} shift={shift}")
        check_fwd_bwd(g, host_csr(tiny), H.contiguous(), G, binding.DG_OP_SUM, csc)


# ------------------------------------------------------------------ closed forms, degenerate
def test_identity_and_ring_bit_exact():
    n, F = 1000, 96
    H = synth.features(n, F, 3, DEV)
    g, *_ = csr_graph(n, [[v] for v in range(n)])
    g.dg_graph_transpose()
    for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
        assert torch.equal(g.dg_aggregate_fwd(H, op), H)
        assert torch.equal(g.dg_aggregate_bwd(H, op), H)
    g, *_ = csr_graph(n, [[(v - 1) % n] for v in range(n)])
    g.dg_graph_transpose()
    assert torch.equal(g.dg_aggregate_fwd(H, binding.DG_OP_SUM), torch.roll(H, 1, 0))
    assert torch.equal(g.dg_aggregate_bwd(H, binding.DG_OP_SUM), torch.roll(H, -1, 0))


@pytest.mark.parametrize("F", [8, 100, 602])
def test_star_graph_heavy_row_and_column(F):
    """Vertex 0 pulls from every other vertex (one CSR row of n-1 entries, a heavy row), and
    every other vertex pulls from vertex 1 (one CSC column of n-1 entries)."""
    n = 6000
    rows = [list(range(1, n))] + [[1] for _ in range(n - 1)]
    w = np.random.default_rng(0).random(2 * (n - 1)).astype(np.float32)
    g, rowptr, colidx = csr_graph(n, rows, weights=w)
    csc = check_transpose(g, rowptr, colidx, w)
    H = synth.features(n, F, 11, DEV)
    G = synth.features(n, F, 12, DEV)
    for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
        check_fwd_bwd(g, (rowptr, colidx, w), H, G, op, csc)


def test_empty_rows_give_zeros_and_empty_graphs_work():
    n, F = 300, 20
    rows = [[] for _ in range(n)]
    rows[7] = [1, 2, 3]
    g, rowptr, colidx = csr_graph(n, rows)
    g.dg_graph_transpose()
    H = synth.features(n, F, 13, DEV)
    out = torch.full((n, F), float("nan"), device=DEV)   # the library overwrites, never reads out
    g.dg_aggregate_fwd(H, binding.DG_OP_MEAN, out=out)
    assert torch.all(out[:7] == 0) and torch.all(out[8:] == 0)
    assert torch.allclose(out[7], H[1:4].mean(0), atol=1e-6)
    # nnz = 0
    g0 = binding.dg_graph_create(5, 0, torch.zeros(6, dtype=torch.int64, device=DEV),
                                 torch.zeros(0, dtype=torch.int32, device=DEV), None)
    g0.dg_graph_validate()
    g0.dg_graph_transpose()
    colptr, rowidx_T, w_T, perm = g0.dg_graph_get_csc()
    assert torch.all(colptr == 0) and rowidx_T.numel() == 0 and w_T is None
    H5 = synth.features(5, 4, 1, DEV)
    assert torch.all(g0.dg_aggregate_fwd(H5, binding.DG_OP_SUM) == 0)
    assert torch.all(g0.dg_aggregate_bwd(H5, binding.DG_OP_MEAN) == 0)
    # n = 0
    g00 = binding.dg_graph_create(0, 0, torch.zeros(1, dtype=torch.int64, device=DEV),
                                  torch.zeros(0, dtype=torch.int32, device=DEV), None)
    g00.dg_graph_transpose()
    e = torch.zeros((0, 4), device=DEV)
    assert g00.dg_aggregate_fwd(e, binding.DG_OP_SUM).shape == (0, 4)


def test_unsorted_rows_duplicates_and_self_loops():
    rng = np.random.default_rng(21)
    n, nnz, F = 500, 20000, 36
    dst = np.sort(rng.integers(0, n, nnz))
    src = rng.integers(0, n, nnz).astype(np.int32)        # unsorted inside rows, with repeats
    rowptr = np.zeros(n + 1, dtype=np.int64)
    np.add.at(rowptr, dst + 1, 1)
    rowptr = np.cumsum(rowptr)
    w = rng.random(nnz).astype(np.float32)
    g = binding.dg_graph_create(n, nnz, torch.as_tensor(rowptr, device=DEV),
                                torch.as_tensor(src, device=DEV), torch.as_tensor(w, device=DEV))
    csc = check_transpose(g, rowptr, src, w)
    H, G = synth.features(n, F, 1, DEV), synth.features(n, F, 2, DEV)
    check_fwd_bwd(g, (rowptr, src, w), H, G, binding.DG_OP_MEAN, csc)


# ------------------------------------------------------------------ source blocking
@pytest.mark.parametrize("blocks,budget_mb", [(2, 31), (4, 31), (16, 31), (0, 1), (0, 2)])
def test_source_blocked_passes_match_the_oracle(blocks, budget_mb):
    """A graph with >= 64 edges per vertex carries split pointers; cutting the source ids into
    2..16 ranges (one launch each, later launches adding to the output) must not change the
    result beyond the summation order.  blocks = 0 lets a small L2 budget choose the cut."""
    sg = synth.make("reddit_like", device=DEV, scale=0.02)
    assert sg.nnz >= 64 * sg.n
    g = make_graph(sg)
    g.dg_graph_set_param("source_blocks", blocks)
    g.dg_graph_set_param("l2_budget_mb", budget_mb)
    g.dg_graph_set_param("heavy_threshold", 256)      # some rows take the block-per-row path
    csc = check_transpose(g, *host_csr(sg))
    for F in (602, 64, 100, 7):
        H = synth.features(sg.n, F, 41, DEV)
        G = synth.features(sg.n, F, 42, DEV)
        for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
            check_fwd_bwd(g, host_csr(sg), H, G, op, csc)


def test_source_blocking_weighted_and_unsorted_rows():
    """Weighted dense-ish graph; then the same edges with every row shuffled: the CSR loses its
    split pointers (rows unsorted) while the CSC, sorted by construction, keeps them."""
    rng = np.random.default_rng(5)
    n, deg, F = 5000, 80, 48
    src = np.stack([np.sort(rng.choice(n, deg, replace=False)) for _ in range(n)]).astype(np.int32)
    rowptr = np.arange(n + 1, dtype=np.int64) * deg
    w = rng.random(n * deg).astype(np.float32)
    H, G = synth.features(n, F, 1, DEV), synth.features(n, F, 2, DEV)
    for shuffle in (False, True):
        cols = src.copy()
        if shuffle:
            for v in range(n):
                rng.shuffle(cols[v])
        cols = cols.reshape(-1)
        g = binding.dg_graph_create(n, n * deg, torch.as_tensor(rowptr, device=DEV),
                                    torch.as_tensor(cols, device=DEV),
                                    torch.as_tensor(w, device=DEV))
        g.dg_graph_set_param("source_blocks", 8)
        csc = check_transpose(g, rowptr, cols, w)
        for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
            check_fwd_bwd(g, (rowptr, cols, w), H, G, op, csc)


def test_deterministic_bits_with_source_blocks_and_heavy_rows():
    """Same call, same data, same bits: also when the pass is cut into source blocks (later
    launches add to the output) and some rows take the block-per-row path."""
    sg = synth.make("reddit_like", device=DEV, scale=0.02)
    g = make_graph(sg)
    g.dg_graph_set_param("source_blocks", 4)
    g.dg_graph_set_param("heavy_threshold", 128)
    g.dg_graph_transpose()
    H = synth.features(sg.n, 602, 3, DEV)
    for op in (binding.DG_OP_SUM, binding.DG_OP_MEAN):
        a = g.dg_aggregate_fwd(H, op).clone()
        b = g.dg_aggregate_bwd(H, op).clone()
        for _ in range(3):
            assert torch.equal(a, g.dg_aggregate_fwd(H, op))
            assert torch.equal(b, g.dg_aggregate_bwd(H, op))


def test_feature_width_limit_and_parameter_ranges(tiny):
    g = make_graph(tiny)
    lib = binding.lib()
    import ctypes
    H = synth.features(tiny.n, 4, 1, DEV)
    st = lib.dg_aggregate_fwd(g._h, ctypes.c_void_p(H.data_ptr()), (1 << 20) + 4, 0,
                              ctypes.c_void_p(H.data_ptr() + 64), None)
    assert st == binding.DG_ERR_UNSUPPORTED
    for name, bad in (("heavy_threshold", 1), ("rows_per_block", 249), ("source_blocks", 3),
                      ("l2_budget_mb", 0), ("heavy_blocks_per_sm", 33), ("slice_features", -1)):
        with pytest.raises(binding.DgError) as e:
            g.dg_graph_set_param(name, bad)
        assert e.value.status == binding.DG_ERR_INVALID_ARG
    for name in ("heavy_threshold", "rows_per_block", "source_blocks", "l2_budget_mb",
                 "heavy_blocks_per_sm", "slice_features"):
        g.dg_graph_get_param(name)


def test_probe_gather_sums_the_rows_it_names():
    rows, rf, count = 1000, 32, 5000
    table = synth.features(rows, rf, 1, DEV)
    idx = torch.randint(0, rows, (count,), device=DEV, dtype=torch.int32)
    sink = torch.zeros(((count + 511) // 512) * 128, device=DEV)
    binding.dg_probe_gather(table, idx, sink)
    torch.cuda.synchronize()
    # warp w sums gathers [512 w, 512 w + 512): 32 lanes x 4 floats hold 4 lane groups x 32 columns
    got = sink.view(-1, 4, rf).sum(1)
    want = torch.stack([table[idx[w * 512:(w + 1) * 512].long()].double().sum(0)
                        for w in range(got.shape[0])])
    assert torch.allclose(got.double(), want, rtol=1e-4, atol=1e-3)


@pytest.mark.parametrize("remote", [False, True])
@pytest.mark.parametrize("rf", [8, 32, 128])
def test_probe_gather_smem_sums_the_rows_it_names(rf, remote):
    """Row r of the stage holds the value r, so a warp's sum over its 4096 gathers is the sum of
    its indices (exact in fp32 at these sizes), from its own or its cluster partner's stage."""
    stage_rows, count = 300, 3 * 4096 + 1000
    idx = torch.randint(0, stage_rows, (count,), device=DEV, dtype=torch.int32)
    warps = (count + 4095) // 4096
    sink = torch.zeros((warps + 32) * 128, device=DEV)
    binding.dg_probe_gather_smem(rf, stage_rows, idx, sink, remote)
    torch.cuda.synchronize()
    groups = 128 // rf
    got = sink[:warps * 128].view(warps, groups, rf).sum(1)
    want = torch.stack([idx[w * 4096:(w + 1) * 4096].double().sum().expand(rf) for w in range(warps)])
    assert torch.equal(got.double(), want)
    with pytest.raises(binding.DgError):
        binding.dg_probe_gather_smem(128, 1000, idx, sink, remote)      # 512 KB stage


# ------------------------------------------------------------------ errors never trap
def test_error_statuses(tiny):
    g = make_graph(tiny)
    H = synth.features(tiny.n, 64, 1, DEV)
    with pytest.raises(binding.DgError) as e:
        g.dg_aggregate_bwd(H, binding.DG_OP_SUM)
    assert e.value.status == binding.DG_ERR_NOT_TRANSPOSED
    with pytest.raises(binding.DgError) as e:
        g.dg_graph_get_csc()
    assert e.value.status == binding.DG_ERR_NOT_TRANSPOSED
    with pytest.raises(binding.DgError) as e:
        g.dg_aggregate_fwd(H, binding.DG_OP_SUM, out=H)           # aliasing
    assert e.value.status == binding.DG_ERR_INVALID_ARG
    with pytest.raises(binding.DgError) as e:
        g.dg_aggregate_fwd(H, 7)                                   # bad op
    assert e.value.status == binding.DG_ERR_INVALID_ARG
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(binding.DgError) as e:
        g.dg_graph_transpose(csc_storage=small)
    assert e.value.status == binding.DG_ERR_WORKSPACE
    with pytest.raises(binding.DgError):
        g.dg_graph_set_param("no_such_knob", 1)
    # a malformed CSR is refused at ingest (no handle is made), not found by a fault later
    for bad_value in (tiny.n + 3, tiny.n, -1):
        bad_col = tiny.colidx.clone().to(DEV)
        bad_col[5] = bad_value
        with pytest.raises(binding.DgError) as e:
            binding.dg_graph_create(tiny.n, tiny.nnz, tiny.rowptr.to(DEV), bad_col, None)
        assert e.value.status == binding.DG_ERR_INVALID_GRAPH and "colidx" in str(e.value)
    bad_ptr = tiny.rowptr.clone().to(DEV)
    bad_ptr[10] = bad_ptr[11] + 1
    with pytest.raises(binding.DgError) as e:
        binding.dg_graph_create(tiny.n, tiny.nnz, bad_ptr, tiny.colidx.to(DEV), None)
    assert e.value.status == binding.DG_ERR_INVALID_GRAPH and "rowptr decreases" in str(e.value)
    bad_ptr = tiny.rowptr.clone().to(DEV)
    bad_ptr[tiny.n] -= 1
    with pytest.raises(binding.DgError) as e:
        binding.dg_graph_create(tiny.n, tiny.nnz, bad_ptr, tiny.colidx.to(DEV), None)
    assert e.value.status == binding.DG_ERR_INVALID_GRAPH
    # arrays that go bad after ingest are found by dg_graph_validate
    col = tiny.colidx.clone().to(DEV)
    gv = binding.dg_graph_create(tiny.n, tiny.nnz, tiny.rowptr.to(DEV), col, None)
    gv.dg_graph_validate()
    col[7] = tiny.n
    with pytest.raises(binding.DgError) as e:
        gv.dg_graph_validate()
    assert e.value.status == binding.DG_ERR_INVALID_GRAPH
    col[7] = 0
    # scratch inside the tail of csc_storage is an overlap, however far from its start
    need_csc, need_scratch = g.dg_graph_transpose_workspace()
    big = torch.empty(need_csc + need_scratch + 512, dtype=torch.uint8, device=DEV)
    tail = ((need_csc - 256) // 256) * 256
    with pytest.raises(binding.DgError) as e:
        g.dg_graph_transpose(csc_storage=big[:need_csc + 256], scratch=big[tail:])
    assert e.value.status == binding.DG_ERR_INVALID_ARG and "overlap" in str(e.value)
    # the context is still healthy
    g.dg_graph_transpose()
    g.dg_aggregate_bwd(H, binding.DG_OP_SUM)
    torch.cuda.synchronize()


def test_host_entry_point(tiny):
    g = make_graph(tiny)
    g.dg_graph_transpose()
    F = 64
    H = synth.features(tiny.n, F, 1).pin_memory()
    G = synth.features(tiny.n, F, 2).pin_memory()
    out = torch.empty_like(H).pin_memory()
    dH = torch.empty_like(H).pin_memory()
    ws = torch.empty(g.dg_aggregate_host_workspace(F), dtype=torch.uint8, device=DEV)
    g.dg_aggregate_host(H, G, binding.DG_OP_MEAN, out, dH, ws)
    torch.cuda.synchronize()
    assert torch.equal(out, g.dg_aggregate_fwd(H.to(DEV), binding.DG_OP_MEAN).cpu())
    assert torch.equal(dH, g.dg_aggregate_bwd(G.to(DEV), binding.DG_OP_MEAN).cpu())


@pytest.mark.parametrize("F,pinned", [(602, True), (300, True), (257, False)])
def test_host_entry_point_in_column_chunks(tiny, F, pinned):
    """Matrices wider than 256 columns go through the host entry point in 128-column chunks
    (upload, kernels and download overlapped); the result is checked against the oracle, twice in
    a row so that the second call reuses the workspace while the first may still be draining."""
    g = make_graph(tiny)
    csc = check_transpose(g, *host_csr(tiny))
    H = synth.features(tiny.n, F, 1)
    G = synth.features(tiny.n, F, 2)
    if pinned:
        H, G = H.pin_memory(), G.pin_memory()
    out, dH = torch.empty_like(H), torch.empty_like(H)
    if pinned:
        out, dH = out.pin_memory(), dH.pin_memory()
    ws = torch.empty(g.dg_aggregate_host_workspace(F), dtype=torch.uint8, device=DEV)
    rowptr_h, colidx_h, w_h = host_csr(tiny)
    for _ in range(2):
        out.fill_(float("nan")); dH.fill_(float("nan"))
        g.dg_aggregate_host(H, G, binding.DG_OP_MEAN, out, dH, ws)
        torch.cuda.synchronize()
        ref, mag = oracle.ap_forward(rowptr_h, colidx_h, w_h, H.numpy(), oracle.OP_MEAN)
        assert_within_bound(out.numpy(), ref, mag, "host fwd")
        ref, mag = oracle.ap_backward(rowptr_h, *csc, G.numpy(), oracle.OP_MEAN)
        assert_within_bound(dH.numpy(), ref, mag, "host bwd")
    # forward only
    out.fill_(float("nan"))
    g.dg_aggregate_host(H, None, binding.DG_OP_SUM, out, None, ws)
    torch.cuda.synchronize()
    ref, mag = oracle.ap_forward(rowptr_h, colidx_h, w_h, H.numpy(), oracle.OP_SUM)
    assert_within_bound(out.numpy(), ref, mag, "host fwd only")


# ------------------------------------------------------------------ mid-size workloads, in full
@pytest.mark.parametrize("name,scale,F,ops", [
    ("reddit_like", 0.02, 602, (binding.DG_OP_MEAN,)),
    ("products_like", 0.02, 100, (binding.DG_OP_SUM, binding.DG_OP_MEAN)),
    ("proteins_like", 0.02, 64, (binding.DG_OP_SUM,)),
    ("papers_like", 0.002, 128, (binding.DG_OP_SUM,)),
])
def test_scaled_workloads_full_comparison(name, scale, F, ops):
    """Several thousand tiles with ragged tails, compared in full with the oracle."""
    sg = synth.make(name, device=DEV, scale=scale)
    g = make_graph(sg)
    g.dg_graph_validate()
    csc = check_transpose(g, *host_csr(sg))
    H = synth.features(sg.n, F, 31, DEV)
    G = synth.features(sg.n, F, 32, DEV)
    for op in ops:
        check_fwd_bwd(g, host_csr(sg), H, G, op, csc)
