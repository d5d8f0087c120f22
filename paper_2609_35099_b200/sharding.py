"""Receiver-sharded convolution over several GPUs, one process per GPU (plumbing around the C ABI).

A rank owns a contiguous range of receivers, balanced by edge count, and the edges into them.  Every edge-local
tensor (sh, w and their gradients) and every output row stays with its rank; node rows are all that crosses GPUs:

    forward   x rows of the halo (senders the rank does not own): every rank all-gathers the owned x rows once
              (NCCL over NVLink; 2 KB per node, half a percent of the convolution's traffic), then a row-gather
              kernel builds x_local = [owned rows | halo rows] in local memory, and the local problem runs
              through the ordinary e3j_conv_fwd
    backward  the local e3j_conv_bwd yields grad_x for owned and halo nodes; the halo shares are all-gathered
              and every owner adds the shares for its nodes in rank order (a row-add kernel per source rank:
              no floating-point atomics, bit-identical from run to run)

Nothing here computes: the convolution, the renumbering (e3j_shard_prepare) and the row kernels are the
library's; torch.distributed moves the bytes.  The `ops` argument names the functions that do the work, so that
the same orchestration runs on CPU ranks (gloo) in the tests with stand-ins for the kernels.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def node_cuts(rowptr: np.ndarray, world: int) -> list[int]:
    """Receiver boundaries [c_0 = 0, ..., c_world = n_nodes]: contiguous ranges with about equal edge counts."""
    from .workloads import shard_receivers
    cuts = [shard_receivers(rowptr, r, world)[0] for r in range(world)]
    return cuts + [len(rowptr) - 1]


@dataclass
class Shard:
    rank: int
    world: int
    cuts: list          # node boundaries of all ranks
    lo: int
    hi: int
    e_lo: int           # the rank's slice of the receiver-sorted edge list
    e_hi: int
    senders: object     # local ids, tensor [e_hi - e_lo]
    receivers: object
    halo_ids: object    # global ids of the halo nodes, ascending, tensor [n_halo]

    @property
    def n_owned(self) -> int:
        return self.hi - self.lo

    @property
    def n_local(self) -> int:
        return self.n_owned + int(self.halo_ids.numel())


class CudaOps:
    """The library's kernels (the product path)."""

    def __init__(self, plan):
        import paper_2609_35099_b200 as e3j
        self.e3j, self.plan = e3j, plan

    def shard_prepare(self, n_nodes, lo, hi, senders, receivers):
        return self.e3j.e3j_shard_prepare(n_nodes, lo, hi, senders, receivers)

    def rows_gather(self, dst, src, ids):
        return self.e3j.e3j_rows_gather(dst, src, ids)

    def rows_add(self, dst, src, ids):
        return self.e3j.e3j_rows_add(dst, src, ids)

    def graph_prepare(self, n_local, senders, receivers):
        return self.e3j.e3j_graph_prepare(n_local, senders, receivers)

    def conv_fwd(self, x_local, sh, w, senders, receivers, graph, **kw):
        return self.e3j.e3j_conv_fwd(self.plan, x_local, sh, w, senders, receivers, graph[0], **kw)

    def conv_bwd(self, x_local, sh, w, senders, receivers, grad_out_local, graph, **kw):
        return self.e3j.e3j_conv_bwd(self.plan, x_local, sh, w, senders, receivers, grad_out_local, *graph, **kw)


def make_shard(ops, rank: int, world: int, n_nodes: int, senders, receivers, rowptr_host: np.ndarray) -> Shard:
    """The rank's local problem from the global graph (global sender / receiver tensors on the rank's device)."""
    cuts = node_cuts(rowptr_host, world)
    lo, hi = cuts[rank], cuts[rank + 1]
    e_lo, e_hi = int(rowptr_host[lo]), int(rowptr_host[hi])
    ls, lr, halo = ops.shard_prepare(n_nodes, lo, hi, senders[e_lo:e_hi].contiguous(), receivers[e_lo:e_hi].contiguous())
    return Shard(rank, world, cuts, lo, hi, e_lo, e_hi, ls, lr, halo)


def _all_gather_padded(t, rows: int, group):
    """All-gather of a [n, ...] tensor whose first dimension differs between ranks: padded to `rows` rows."""
    import torch
    import torch.distributed as dist
    pad = torch.zeros((rows,) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
    pad[:t.shape[0]] = t
    out = [torch.empty_like(pad) for _ in range(dist.get_world_size(group))]
    dist.all_gather(out, pad, group=group)
    return out


def halo_source_rows(shard: Shard, rows_per_rank: int):
    """Row of every halo node in the concatenation of the ranks' padded owned-row blocks."""
    import torch
    cuts = torch.tensor(shard.cuts, dtype=torch.int64, device=shard.halo_ids.device)
    h = shard.halo_ids.to(torch.int64)
    owner = torch.bucketize(h, cuts[1:], right=True)
    return (owner * rows_per_rank + (h - cuts[owner])).to(torch.int32)


def gather_x(ops, shard: Shard, x_owned, group=None):
    """x_local [n_local, d, N_q] = [owned rows | halo rows]; one all-gather of the owned rows."""
    import torch
    rows = max(b - a for a, b in zip(shard.cuts[:-1], shard.cuts[1:]))
    blocks = _all_gather_padded(x_owned, rows, group)
    x_local = torch.empty((shard.n_local,) + tuple(x_owned.shape[1:]), dtype=x_owned.dtype, device=x_owned.device)
    x_local[:shard.n_owned] = x_owned
    if shard.halo_ids.numel():
        everything = torch.cat(blocks)   # remote rows are in local memory before any kernel reads them
        ops.rows_gather(x_local[shard.n_owned:], everything, halo_source_rows(shard, rows))
    return x_local


def add_shares(ops, shard: Shard, grad_x_owned, shares):
    """grad_x_owned += the shares of the other ranks for this rank's nodes, in rank order.
    shares[r] = (halo ids of rank r, ascending, [n]; their grad_x rows [n, d, N_q])."""
    import torch
    for r, (ids, rows) in enumerate(shares):
        if r == shard.rank or ids.numel() == 0:
            continue
        bounds = torch.searchsorted(ids.to(torch.int64), torch.tensor([shard.lo, shard.hi], device=ids.device))
        a, b = int(bounds[0]), int(bounds[1])
        if b > a:
            ops.rows_add(grad_x_owned, rows[a:b].contiguous(), (ids[a:b] - shard.lo).to(torch.int32).contiguous())
    return grad_x_owned


def reduce_grad_x(ops, shard: Shard, grad_x_local, group=None):
    """grad_x of the owned nodes: the local part plus every other rank's halo shares for them."""
    import torch
    import torch.distributed as dist
    n_halo = torch.tensor([int(shard.halo_ids.numel())], dtype=torch.int64, device=grad_x_local.device)
    counts = [torch.zeros_like(n_halo) for _ in range(shard.world)]
    dist.all_gather(counts, n_halo, group=group)
    counts = [int(c.item()) for c in counts]
    rows = max(max(counts), 1)
    ids = _all_gather_padded(shard.halo_ids, rows, group)
    vals = _all_gather_padded(grad_x_local[shard.n_owned:], rows, group)
    shares = [(i[:c], v[:c]) for i, v, c in zip(ids, vals, counts)]
    return add_shares(ops, shard, grad_x_local[:shard.n_owned].clone(), shares)
