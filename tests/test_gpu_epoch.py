"""The GraphSAGE epoch built on the aggregation primitive against a pure-torch reference
(index_add_ for the neighbour sum, autograd for everything): loss and every weight gradient."""
import pytest
import torch

from paper_2104_06700_b200 import binding, graphsage, synth
from parity_util import make_graph

pytestmark = pytest.mark.gpu
DEV = "cuda"


def reference_forward(sg, X, weights, biases):
    n = sg.n
    rows = torch.repeat_interleave(torch.arange(n, device=DEV), (sg.rowptr[1:] - sg.rowptr[:-1]).to(DEV))
    cols = sg.colidx.to(DEV).long()
    deg1 = (sg.rowptr[1:] - sg.rowptr[:-1]).to(DEV).double() + 1.0
    H = X.double()
    for i, (W, b) in enumerate(zip(weights, biases)):
        agg = torch.zeros_like(H).index_add_(0, rows, H[cols])
        Z = (agg + H) / deg1.unsqueeze(1)
        H = Z @ W.double().t() + b.double()
        if i + 1 < len(weights):
            H = torch.relu(H)
    return H


@pytest.mark.parametrize("fused", [False, "table", "row_scale"])
@pytest.mark.parametrize("project_first", [False, True])
@pytest.mark.parametrize("dims", [[64, 32, 7], [20, 16, 16, 5]])
def test_epoch_loss_and_gradients_match_torch_reference(dims, project_first, fused):
    sg = synth.make("tiny", weighted=False)
    g = make_graph(sg)
    if fused:
        g.dg_graph_set_param("self_loops", 1)
    g.dg_graph_transpose()
    torch.manual_seed(0)
    model = graphsage.GraphSAGE(g, dims, project_first=project_first,
                                fused_aggregator=bool(fused)).to(DEV)
    if fused == "table":
        model.scaled_backward = True       # per-edge factors of the transpose
    elif fused == "row_scale":
        model.scaled_backward = False      # dOut scaled row by row, then the sum backward
    X = synth.features(sg.n, dims[0], 3, DEV)
    labels = torch.randint(0, dims[-1], (sg.n,), device=DEV)
    train_idx = torch.arange(0, sg.n, 3, device=DEV)

    logits = model(X)
    loss = torch.nn.functional.cross_entropy(logits[train_idx], labels[train_idx])
    loss.backward()

    Ws = [l.weight.detach().clone().requires_grad_(True) for l in model.lin]
    bs = [l.bias.detach().clone().requires_grad_(True) for l in model.lin]
    ref_logits = reference_forward(sg, X, Ws, bs)
    ref_loss = torch.nn.functional.cross_entropy(ref_logits[train_idx], labels[train_idx])
    ref_loss.backward()

    assert abs(float(loss) - float(ref_loss)) <= 1e-4 * abs(float(ref_loss))
    for lin, W, b in zip(model.lin, Ws, bs):
        for got, want in ((lin.weight.grad, W.grad), (lin.bias.grad, b.grad)):
            scale = float(want.abs().max()) + 1e-12
            assert float((got.double() - want.double()).abs().max()) <= 1e-4 * scale


def test_epoch_function_trains():
    sg = synth.make("tiny", weighted=False)
    g = make_graph(sg)
    g.dg_graph_transpose()
    torch.manual_seed(1)
    model = graphsage.GraphSAGE(g, [64, 32, 7]).to(DEV)
    X = synth.features(sg.n, 64, 4, DEV)
    labels = torch.randint(0, 7, (sg.n,), device=DEV)
    epoch = graphsage.make_epoch(model, X, labels, torch.arange(sg.n, device=DEV))
    losses = [float(epoch()) for _ in range(30)]
    assert losses[-1] < losses[0]
    assert graphsage.aggregation_calls([64, 32, 7]) == [("fwd", 64), ("fwd", 32), ("bwd", 32)]
    assert graphsage.aggregation_calls([64, 32, 7], True) == [("fwd", 32), ("bwd", 32),
                                                              ("fwd", 7), ("bwd", 7)]
    assert graphsage.aggregation_calls([16, 32, 32, 7], True) == [
        ("fwd", 16), ("fwd", 32), ("bwd", 32), ("fwd", 7), ("bwd", 7)]


def test_bf16_aggregation_stays_close_to_fp32():
    """Aggregating bf16-rounded activations changes the loss by bf16 rounding only."""
    sg = synth.make("tiny", weighted=False)
    g = make_graph(sg)
    g.dg_graph_transpose()
    X = synth.features(sg.n, 64, 3, DEV)
    labels = torch.randint(0, 8, (sg.n,), device=DEV)
    losses = []
    for bf in (False, True):
        torch.manual_seed(0)
        model = graphsage.GraphSAGE(g, [64, 32, 8], bf16_aggregate=bf).to(DEV)
        logits = model(X)
        loss = torch.nn.functional.cross_entropy(logits, labels)
        loss.backward()
        losses.append((float(loss), model.lin[0].weight.grad.clone()))
    assert abs(losses[0][0] - losses[1][0]) <= 2e-2 * abs(losses[0][0])
    scale = float(losses[0][1].abs().max())
    assert float((losses[0][1] - losses[1][1]).abs().max()) <= 5e-2 * scale


def test_fused_aggregator_needs_the_matching_handle():
    sg = synth.make("tiny", weighted=False)
    g = make_graph(sg)
    with pytest.raises(ValueError):
        graphsage.GraphSAGE(g, [8, 4], fused_aggregator=True)
    g.dg_graph_set_param("self_loops", 1)
    with pytest.raises(ValueError):
        graphsage.GraphSAGE(g, [8, 4])


@pytest.mark.parametrize("op", [binding.DG_OP_SUM, binding.DG_OP_MEAN])
def test_learnable_edge_weights_gradient_and_refresh(op):
    """The autograd wrapper returns the gradient with respect to the edge weights (one dot product
    per edge, dg_aggregate_edge_grad) next to the one for the features; after an in-place update of
    the weights dg_graph_update_weights brings the CSC of the backward pass up to date.  Reference:
    index_add_ with autograd in fp64."""
    sg = synth.make("tiny")
    rowptr, colidx = sg.rowptr.to(DEV), sg.colidx.to(DEV)
    w = sg.edge_w.to(DEV).clone().requires_grad_(True)
    g = binding.dg_graph_create(sg.n, sg.nnz, rowptr, colidx, w.detach())
    assert w.data_ptr() == g.edge_w.data_ptr()
    g.dg_graph_transpose()
    F = 48
    rows = torch.repeat_interleave(torch.arange(sg.n, device=DEV), rowptr[1:] - rowptr[:-1])
    deg = (rowptr[1:] - rowptr[:-1]).double().clamp(min=1).unsqueeze(1)

    def reference(H, wt):
        out = torch.zeros((sg.n, F), dtype=torch.float64, device=DEV)
        out.index_add_(0, rows, H.double()[colidx.long()] * wt.double().unsqueeze(1))
        return out / deg if op == binding.DG_OP_MEAN else out

    for step in range(2):
        H = synth.features(sg.n, F, 70 + step, DEV).requires_grad_(True)
        G = synth.features(sg.n, F, 80 + step, DEV)
        out = graphsage.aggregate(g, H, op, edge_w=w)
        (out * G).sum().backward()
        Hr = H.detach().clone().requires_grad_(True)
        wr = w.detach().clone().requires_grad_(True)
        (reference(Hr, wr) * G.double()).sum().backward()
        assert torch.allclose(out.detach().double(), reference(H.detach(), w.detach()),
                              rtol=1e-4, atol=1e-4)
        assert torch.allclose(H.grad.double(), Hr.grad.double(), rtol=1e-4, atol=1e-4)
        assert torch.allclose(w.grad.double(), wr.grad.double(), rtol=1e-4, atol=1e-3)
        with torch.no_grad():                       # an optimiser step on the weights, in place
            w -= 0.05 * w.grad
            w.grad = None
        g.dg_graph_update_weights()
