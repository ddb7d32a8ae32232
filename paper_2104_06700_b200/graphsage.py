"""Full-batch GraphSAGE with the GCN aggregator (Section 5.1 of the paper, Models and
Parameters), as the composite workload the epoch-time metric is quoted on.

Only the aggregation primitive runs in libdgagg; everything dense stays in torch, outside the
hot path: per layer  z_v = (sum_{u in N(v)} h_u + h_v) / (deg(v) + 1),  h'_v = act(z_v W + b)
(aggregate first, then the Linear: Table 8 of the paper lists the aggregation widths 100, 256,
256 for the 3-layer model, i.e. the layers' input widths), ReLU between layers, none after the
last, softmax cross-entropy on a training mask, Adam.  The features need no gradient, so an
L-layer epoch runs L forward and L-1 backward aggregations.
"""
from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding


class _Aggregate(torch.autograd.Function):
    """out = A H through dg_aggregate_fwd; the backward pass calls dg_aggregate_bwd."""

    @staticmethod
    def forward(ctx, H: torch.Tensor, graph: "binding.Graph", op: int) -> torch.Tensor:
        ctx.graph, ctx.op = graph, op
        return graph.dg_aggregate_fwd(H.contiguous(), op)

    @staticmethod
    def backward(ctx, dOut: torch.Tensor):
        dH = None
        if ctx.needs_input_grad[0]:
            dH = ctx.graph.dg_aggregate_bwd(dOut.contiguous(), ctx.op)
        return dH, None, None


def aggregate(graph: "binding.Graph", H: torch.Tensor, op: int = binding.DG_OP_SUM) -> torch.Tensor:
    """Differentiable aggregation primitive (the graph must have been transposed)."""
    return _Aggregate.apply(H, graph, op)


class GraphSAGE(torch.nn.Module):
    """`dims` = [in, hidden, ..., classes]; one Linear per layer."""

    def __init__(self, graph: "binding.Graph", dims: Sequence[int]):
        super().__init__()
        self.graph = graph
        self.lin = torch.nn.ModuleList(
            [torch.nn.Linear(dims[i], dims[i + 1]) for i in range(len(dims) - 1)])
        deg = (graph.rowptr[1:] - graph.rowptr[:-1]).to(torch.float32)
        self.register_buffer("inv_deg1", (1.0 / (deg + 1.0)).unsqueeze(1))

    def forward(self, H: torch.Tensor) -> torch.Tensor:
        for i, lin in enumerate(self.lin):
            Z = (aggregate(self.graph, H, binding.DG_OP_SUM) + H) * self.inv_deg1
            H = lin(Z)
            if i + 1 < len(self.lin):
                H = torch.relu(H)
        return H


def make_epoch(model: GraphSAGE, X: torch.Tensor, labels: torch.Tensor, train_idx: torch.Tensor,
               lr: float = 0.01, weight_decay: float = 5e-4):
    """Returns a function that runs one training epoch (forward, loss on the training vertices,
    backward, Adam step) and returns the loss tensor."""
    opt = torch.optim.Adam(model.parameters(), lr=lr, weight_decay=weight_decay)

    def epoch() -> torch.Tensor:
        opt.zero_grad(set_to_none=True)
        logits = model(X)
        loss = torch.nn.functional.cross_entropy(logits[train_idx], labels[train_idx])
        loss.backward()
        opt.step()
        return loss.detach()

    return epoch


def aggregation_calls(dims: Sequence[int]) -> List[tuple]:
    """(direction, width) of every aggregation one epoch runs, for work accounting."""
    widths = list(dims[:-1])
    return [("fwd", w) for w in widths] + [("bwd", w) for w in widths[1:]]
