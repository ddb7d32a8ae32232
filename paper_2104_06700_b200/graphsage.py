"""Full-batch GraphSAGE with the GCN aggregator (Section 5.1 of the paper, Models and
Parameters), as the composite workload the epoch-time metric is quoted on.

Only the aggregation primitive runs in libdgagg; everything dense stays in torch, outside the
hot path: per layer  z_v = (sum_{u in N(v)} h_u + h_v) / (deg(v) + 1),  h'_v = act(z_v W + b)
(aggregate first, then the Linear: Table 8 of the paper lists the aggregation widths 100, 256,
256 for the 3-layer model, i.e. the layers' input widths), ReLU between layers, none after the
last, softmax cross-entropy on a training mask, Adam.  The features need no gradient, so an
L-layer epoch runs L forward and L-1 backward aggregations.  With ``fused_aggregator`` the
own row and the division are done by the library inside the aggregation kernels (graph
attribute "self_loops"), which saves the elementwise passes over the n x F matrices.
"""
from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding


class _Aggregate(torch.autograd.Function):
    """out = A H through dg_aggregate_fwd; the backward pass calls dg_aggregate_bwd.  With
    ``bf16`` the gathered matrices (H in the forward, dOut in the backward pass) are rounded to
    bf16 first and the bf16 entry points are used; sums and results stay fp32.

    ``row_scale`` (n x 1, only with op = mean on a handle with self loops): the backward pass
    multiplies dOut by it and runs the *sum* backward on the product instead of the mean
    backward.  Both give A^T D dOut + D dOut; the sum backward needs no per-edge factor, which
    on graphs with long rows saves more kernel time than the one elementwise pass costs."""

    @staticmethod
    def forward(ctx, H: torch.Tensor, graph: "binding.Graph", op: int, bf16: bool,
                row_scale, edge_w=None) -> torch.Tensor:
        ctx.graph, ctx.op, ctx.bf16, ctx.row_scale = graph, op, bf16, row_scale
        ctx.want_dw = edge_w is not None and edge_w.requires_grad
        if ctx.want_dw:
            if edge_w.data_ptr() != graph.edge_w.data_ptr():
                raise ValueError("edge_w must be the tensor the graph handle was created with")
            ctx.save_for_backward(H)
        if bf16:
            return graph.dg_aggregate_fwd_bf16(H.contiguous().to(torch.bfloat16), op)
        return graph.dg_aggregate_fwd(H.contiguous(), op)

    @staticmethod
    def backward(ctx, dOut: torch.Tensor):
        dH = None
        upstream = dOut
        if ctx.needs_input_grad[0]:
            op = ctx.op
            if ctx.row_scale is not None:
                dOut = dOut * ctx.row_scale
                op = binding.DG_OP_SUM
            if ctx.bf16:
                dH = ctx.graph.dg_aggregate_bwd_bf16(dOut.contiguous().to(torch.bfloat16), op)
            else:
                dH = ctx.graph.dg_aggregate_bwd(dOut.contiguous(), op)
        dW = None
        if ctx.want_dw:     # message passing onto the edges: one dot product per edge
            (H,) = ctx.saved_tensors
            dW = ctx.graph.dg_aggregate_edge_grad(H.contiguous(), upstream.contiguous(), ctx.op)
        return dH, None, None, None, None, dW


def aggregate(graph: "binding.Graph", H: torch.Tensor, op: int = binding.DG_OP_SUM,
              bf16: bool = False, row_scale=None, edge_w=None) -> torch.Tensor:
    """Differentiable aggregation primitive (the graph must have been transposed).

    ``edge_w``: pass the weight tensor the handle was created with to get its gradient too
    (learnable edge weights).  The handle reads that tensor in place; after an optimiser step
    on it call ``graph.dg_graph_update_weights()`` so that the CSC used by the backward pass
    carries the new values."""
    return _Aggregate.apply(H, graph, op, bf16, row_scale, edge_w)


class GraphSAGE(torch.nn.Module):
    """`dims` = [in, hidden, ..., classes]; one Linear per layer.

    ``project_first``: the aggregator is linear, so ((A H + H) / (deg+1)) W = (A (H W) + H W) /
    (deg+1): a layer whose output is narrower than its input may apply the Linear first and
    aggregate the narrower matrix.  Same function up to fp32 rounding, less aggregation work
    (602 -> 256 columns on the first Reddit-like layer); off by default because the paper
    aggregates first (its Table 8 counts the aggregation at the layers' input widths).
    """

    def __init__(self, graph: "binding.Graph", dims: Sequence[int], project_first: bool = False,
                 bf16_aggregate: bool = False, fused_aggregator: bool = False):
        super().__init__()
        self.graph = graph
        self.project_first = project_first
        self.bf16_aggregate = bf16_aggregate   # aggregate bf16-rounded activations (even widths)
        # the whole aggregator (own row added, division by in-degree + 1) inside the library's
        # kernels, forward and backward: needs a handle whose "self_loops" attribute was set
        # to 1 before dg_graph_transpose
        self.fused_aggregator = fused_aggregator
        # backward of the fused aggregator: per-edge factors tabulated by the transpose (short
        # rows: the elementwise pass would cost more than the factors), or dOut scaled row by
        # row and the sum backward (long rows)
        self.scaled_backward = graph.nnz < 64 * graph.n
        if fused_aggregator and graph.dg_graph_get_param("self_loops") != 1:
            raise ValueError("fused_aggregator needs a graph handle with self_loops = 1")
        if not fused_aggregator and graph.dg_graph_get_param("self_loops") != 0:
            raise ValueError("this handle adds self loops itself: use fused_aggregator=True")
        self.lin = torch.nn.ModuleList(
            [torch.nn.Linear(dims[i], dims[i + 1]) for i in range(len(dims) - 1)])
        deg = (graph.rowptr[1:] - graph.rowptr[:-1]).to(torch.float32)
        self.register_buffer("inv_deg1", (1.0 / (deg + 1.0)).unsqueeze(1))

    def _gcn(self, M: torch.Tensor) -> torch.Tensor:
        """(sum of the neighbours' rows + own row) / (in-degree + 1)."""
        bf = self.bf16_aggregate and M.shape[1] % 2 == 0
        if self.fused_aggregator:
            return aggregate(self.graph, M, binding.DG_OP_MEAN, bf,
                             None if self.scaled_backward else self.inv_deg1)
        return (aggregate(self.graph, M, binding.DG_OP_SUM, bf) + M) * self.inv_deg1

    def forward(self, H: torch.Tensor) -> torch.Tensor:
        for i, lin in enumerate(self.lin):
            if self.project_first and lin.out_features < lin.in_features:
                P = torch.nn.functional.linear(H, lin.weight)           # bias after the mean
                H = self._gcn(P) + lin.bias
            else:
                H = lin(self._gcn(H))
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
