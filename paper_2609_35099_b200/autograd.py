"""torch.autograd integration of the convolution (plumbing around the C ABI, no arithmetic of its own).

    graph = Graph(n_nodes, senders, receivers)            # prepared once per neighbour list
    out = conv(plan, graph, x, sh, w)                     # differentiable in x, sh, w, to second order

The backward is e3j_conv_bwd; it is itself a differentiable function (of x, sh, w and the incoming cotangent), whose
backward is e3j_conv_bwd_bwd -- what force training needs (a loss on gradients of the energy).  Third derivatives are
not provided.
"""
from __future__ import annotations

import torch

from . import e3j_conv_bwd, e3j_conv_bwd_bwd, e3j_conv_fwd, e3j_graph_prepare


class Graph:
    """Receiver-sorted edge list with the index arrays the kernels want (e3j_graph_prepare), on the device."""

    def __init__(self, n_nodes: int, senders: torch.Tensor, receivers: torch.Tensor):
        self.n_nodes = int(n_nodes)
        self.senders = senders.to(torch.int32).contiguous()
        self.receivers = receivers.to(torch.int32).contiguous()
        self.rowptr, self.sender_perm, self.colptr = e3j_graph_prepare(self.n_nodes, self.senders, self.receivers)


def _c(t):
    return None if t is None else t.contiguous()


class _ConvBackward(torch.autograd.Function):
    @staticmethod
    def forward(ctx, plan, graph, x, sh, w, grad_out):
        ctx.plan, ctx.graph = plan, graph
        ctx.save_for_backward(x, sh, w, grad_out)
        return e3j_conv_bwd(plan, x, sh, w, graph.senders, graph.receivers, grad_out, graph.rowptr, graph.sender_perm,
                            graph.colptr)

    @staticmethod
    @torch.autograd.function.once_differentiable
    def backward(ctx, ct_x, ct_sh, ct_w):
        x, sh, w, grad_out = ctx.saved_tensors
        g = ctx.graph
        gg_out, g_x, g_sh, g_w = e3j_conv_bwd_bwd(ctx.plan, x, sh, w, g.senders, g.receivers, grad_out, g.rowptr,
                                                  g.sender_perm, g.colptr, _c(ct_x), _c(ct_sh), _c(ct_w))
        return None, None, g_x, g_sh, g_w, gg_out


class _Conv(torch.autograd.Function):
    @staticmethod
    def forward(ctx, plan, graph, x, sh, w):
        ctx.plan, ctx.graph = plan, graph
        ctx.save_for_backward(x, sh, w)
        return e3j_conv_fwd(plan, x, sh, w, graph.senders, graph.receivers, graph.rowptr)

    @staticmethod
    def backward(ctx, grad_out):
        x, sh, w = ctx.saved_tensors
        gx, gsh, gw = _ConvBackward.apply(ctx.plan, ctx.graph, x, sh, w, grad_out.contiguous())
        return None, None, gx, gsh, gw


def conv(plan, graph: Graph, x: torch.Tensor, sh: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """out[n_nodes, D, N_q] = message-passing convolution of x [n_nodes, d, N_q] with harmonics sh [n_edges, d'] and
    edge weights w [n_edges, P, N_q] over `graph` (float32 CUDA tensors)."""
    return _Conv.apply(plan, graph, x.contiguous(), sh.contiguous(), w.contiguous())
