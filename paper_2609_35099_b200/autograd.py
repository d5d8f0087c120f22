"""torch.autograd integration of the convolution (plumbing around the C ABI, no arithmetic of its own).

    graph = Graph(n_nodes, senders, receivers)            # prepared once per neighbour list
    out = conv(plan, graph, x, sh, w)                     # differentiable in x, sh, w, to second order
    out = conv_radial(plan, graph, x, sh, h, W)           # weights from the radial layer; first order
    out = conv_vec(plan, graph, x, edge_vec, w)           # harmonics from the edge vectors; first order

The backward is e3j_conv_bwd; it is itself a differentiable function (of x, sh, w and the incoming cotangent), whose
backward is e3j_conv_bwd_bwd -- what force training needs (a loss on gradients of the energy).  Third derivatives are
not provided.
"""
from __future__ import annotations

import torch

from . import (e3j_conv_bwd, e3j_conv_bwd_bwd, e3j_conv_fwd, e3j_conv_radial_bwd, e3j_conv_radial_fwd, e3j_conv_vec_bwd,
               e3j_conv_vec_fwd, e3j_graph_prepare, e3j_graph_validate)


class Graph:
    """Receiver-sorted edge list with the index arrays the kernels want (e3j_graph_prepare), on the device."""

    def __init__(self, n_nodes: int, senders: torch.Tensor, receivers: torch.Tensor, validate: bool = True):
        """validate: check on the device, before anything indexes with them, that the ids lie in [0, n_nodes) and the
        receivers do not decrease (one small kernel and a synchronisation per edge list).  The compute calls
        trust the list: an id outside the range makes them read or write outside their arrays."""
        self.n_nodes = int(n_nodes)
        self.senders = senders.to(torch.int32).contiguous()
        self.receivers = receivers.to(torch.int32).contiguous()
        if validate and e3j_graph_validate(self.n_nodes, self.senders, self.receivers) != 0:
            raise ValueError("edge list: an id outside [0, n_nodes) or receivers that decrease")
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


class _ConvRadial(torch.autograd.Function):
    @staticmethod
    def forward(ctx, plan, graph, x, sh, h, W):
        ctx.plan, ctx.graph = plan, graph
        ctx.save_for_backward(x, sh, h, W)
        return e3j_conv_radial_fwd(plan, x, sh, h, W, graph.senders, graph.receivers, graph.rowptr)

    @staticmethod
    @torch.autograd.function.once_differentiable
    def backward(ctx, grad_out):
        x, sh, h, W = ctx.saved_tensors
        g = ctx.graph
        need = ctx.needs_input_grad[2:]
        gx, gsh, gh, gW = e3j_conv_radial_bwd(ctx.plan, x, sh, h, W, g.senders, g.receivers, grad_out.contiguous(), g.rowptr,
                                              g.sender_perm, g.colptr, grad_x=need[0], grad_sh=need[1], grad_h=need[2],
                                              grad_W=need[3])
        return None, None, gx, gsh, gh, gW


class _ConvVec(torch.autograd.Function):
    @staticmethod
    def forward(ctx, plan, graph, x, edge_vec, w):
        ctx.plan, ctx.graph = plan, graph
        ctx.save_for_backward(x, edge_vec, w)
        return e3j_conv_vec_fwd(plan, x, edge_vec, w, graph.senders, graph.receivers, graph.rowptr)

    @staticmethod
    @torch.autograd.function.once_differentiable
    def backward(ctx, grad_out):
        x, edge_vec, w = ctx.saved_tensors
        g = ctx.graph
        need = ctx.needs_input_grad[2:]
        gx, gvec, gw = e3j_conv_vec_bwd(ctx.plan, x, edge_vec, w, g.senders, g.receivers, grad_out.contiguous(), g.rowptr,
                                        g.sender_perm, g.colptr, grad_x=need[0], grad_vec=need[1], grad_w=need[2])
        return None, None, gx, gvec, gw


def conv_radial(plan, graph: Graph, x, sh, h, W) -> torch.Tensor:
    """The convolution with the edge weights given as the radial network's last layer, w = h W (first derivatives)."""
    return _ConvRadial.apply(plan, graph, x.contiguous(), sh.contiguous(), h.contiguous(), W.contiguous())


def conv_vec(plan, graph: Graph, x, edge_vec, w) -> torch.Tensor:
    """The convolution with the harmonics taken from the edge vectors [n_edges, 3] (first derivatives)."""
    return _ConvVec.apply(plan, graph, x.contiguous(), edge_vec.contiguous(), w.contiguous())
