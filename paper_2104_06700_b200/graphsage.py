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
    """out = A H through dg_aggregate_fwd; the backward pass calls dg_aggregate_bwd.  With
    ``bf16`` the gathered matrices (H in the forward, dOut in the backward pass) are rounded to
    bf16 first and the bf16 entry points are used; sums and results stay fp32."""

    @staticmethod
    def forward(ctx, H: torch.Tensor, graph: "binding.Graph", op: int, bf16: bool) -> torch.Tensor:
        ctx.graph, ctx.op, ctx.bf16 = graph, op, bf16
        if bf16:
            return graph.dg_aggregate_fwd_bf16(H.contiguous().to(torch.bfloat16), op)
        return graph.dg_aggregate_fwd(H.contiguous(), op)

    @staticmethod
    def backward(ctx, dOut: torch.Tensor):
        dH = None
        if ctx.needs_input_grad[0]:
            if ctx.bf16:
                dH = ctx.graph.dg_aggregate_bwd_bf16(dOut.contiguous().to(torch.bfloat16), ctx.op)
            else:
                dH = ctx.graph.dg_aggregate_bwd(dOut.contiguous(), ctx.op)
        return dH, None, None, None


def aggregate(graph: "binding.Graph", H: torch.Tensor, op: int = binding.DG_OP_SUM,
              bf16: bool = False) -> torch.Tensor:
    """Differentiable aggregation primitive (the graph must have been transposed)."""
    return _Aggregate.apply(H, graph, op, bf16)


class GraphSAGE(torch.nn.Module):
    """`dims` = [in, hidden, ..., classes]; one Linear per layer.

    ``project_first``: the aggregator is linear, so ((A H + H) / (deg+1)) W = (A (H W) + H W) /
    (deg+1): a layer whose output is narrower than its input may apply the Linear first and
    aggregate the narrower matrix.  Same function up to fp32 rounding, less aggregation work
    (602 -> 256 columns on the first Reddit-like layer); off by default because the paper
    aggregates first (its Table 8 counts the aggregation at the layers' input widths).
    """

    def __init__(self, graph: "binding.Graph", dims: Sequence[int], project_first: bool = False,
                 bf16_aggregate: bool = False):
        super().__init__()
        self.graph = graph
        self.project_first = project_first
        self.bf16_aggregate = bf16_aggregate   # aggregate bf16-rounded activations (even widths)
        self.lin = torch.nn.ModuleList(
            [torch.nn.Linear(dims[i], dims[i + 1]) for i in range(len(dims) - 1)])
        deg = (graph.rowptr[1:] - graph.rowptr[:-1]).to(torch.float32)
        self.register_buffer("inv_deg1", (1.0 / (deg + 1.0)).unsqueeze(1))

    def forward(self, H: torch.Tensor) -> torch.Tensor:
        for i, lin in enumerate(self.lin):
            if self.project_first and lin.out_features < lin.in_features:
                P = torch.nn.functional.linear(H, lin.weight)           # bias after the mean
                bf = self.bf16_aggregate and P.shape[1] % 2 == 0
                H = (aggregate(self.graph, P, binding.DG_OP_SUM, bf) + P) * self.inv_deg1 + lin.bias
            else:
                bf = self.bf16_aggregate and H.shape[1] % 2 == 0
                Z = (aggregate(self.graph, H, binding.DG_OP_SUM, bf) + H) * self.inv_deg1
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


def aggregation_calls(dims: Sequence[int], project_first: bool = False) -> List[tuple]:
    """(direction, width) of every aggregation one epoch runs, for work accounting.  Aggregating
    first, layer 1 needs no backward aggregation (the features carry no gradient); projecting
    first, the aggregated matrix depends on the layer's weights, so it does."""
    calls = []
    for i in range(len(dims) - 1):
        first = project_first and dims[i + 1] < dims[i]
        w = dims[i + 1] if first else dims[i]
        calls.append(("fwd", w))
        if i > 0 or first:
            calls.append(("bwd", w))
    return calls
