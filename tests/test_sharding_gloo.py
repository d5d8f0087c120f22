"""Host logic of the multi-process path (CPU, gloo, world size 2).

The convolution shards by receiver: every edge-local tensor and every output row lives with its
receiver, forward needs all sender rows (halo), backward returns grad_x shares that are summed
across ranks.  Here the oracle stands in for the compute on each rank; the test checks the shard
boundaries, that the gathered shards reproduce the unsharded result, and that the bench's
max-over-ranks reduction works on this backend.
"""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import conv as oconv
from paper_2609_35099_b200 import workloads


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        c = workloads.CONFIGS[1]
        wl = workloads.make_graph(1)
        cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
        x, y, w, g = workloads.make_features(wl, cp.P, cp.D)
        n = wl.n_nodes
        rowptr = np.searchsorted(wl.receivers, np.arange(n + 1), side="left")
        lo, hi = workloads.shard_receivers(rowptr, rank, world)
        e0, e1 = int(rowptr[lo]), int(rowptr[hi])
        # local problem: receivers lo..hi-1 renumbered from 0; senders keep global ids (halo rows of x)
        rcv = wl.receivers[e0:e1]
        snd = wl.senders[e0:e1]
        out_full = oconv.conv_fwd(cp, x, y[e0:e1], w[e0:e1], snd, rcv)  # rows outside [lo,hi) stay zero
        assert np.all(out_full[:lo] == 0) and np.all(out_full[hi:] == 0)
        dx, dy, dw = oconv.conv_bwd(cp, x, y[e0:e1], w[e0:e1], snd, rcv, g)

        # forward: gather the row shards
        out_t = torch.from_numpy(out_full)
        dist.all_reduce(out_t)  # shards are disjoint in rows, so the sum is the concatenation
        # backward: grad_x shares are summed over ranks (fixed rank order inside gloo's ring is not
        # guaranteed, so compare with a tolerance); edge-local gradients are concatenated
        dx_t = torch.from_numpy(dx)
        dist.all_reduce(dx_t)
        bounds = [None] * world
        dist.all_gather_object(bounds, (lo, hi, e0, e1))
        t = torch.tensor([float(rank + 1)], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == world

        if rank == 0:
            ref = oconv.conv_fwd(cp, x, y, w, wl.senders, wl.receivers)
            rx, ry, rw = oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)
            assert np.abs(out_t.numpy() - ref).max() < 1e-12
            assert np.abs(dx_t.numpy() - rx).max() < 1e-11
            # contiguous cover of receivers and edges
            assert bounds[0][0] == 0 and bounds[-1][1] == n
            assert bounds[0][2] == 0 and bounds[-1][3] == wl.n_edges
            for a, b in zip(bounds[:-1], bounds[1:]):
                assert a[1] == b[0] and a[3] == b[2]
            # edge balance within one receiver row
            sizes = [b[3] - b[2] for b in bounds]
            assert max(sizes) - min(sizes) <= 2 * np.diff(rowptr).max()
        assert np.abs(dy - oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)[1][e0:e1]).max() < 1e-12
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_receiver_sharding_two_ranks(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))


def test_shard_receivers_edge_cases():
    rowptr = np.array([0, 0, 5, 5, 9, 20, 20])
    cuts = [workloads.shard_receivers(rowptr, r, 3) for r in range(3)]
    assert cuts[0][0] == 0 and cuts[-1][1] == 6
    for a, b in zip(cuts[:-1], cuts[1:]):
        assert a[1] == b[0]
    # empty graph: one rank takes every (empty) row
    cuts = [workloads.shard_receivers(np.zeros(4, dtype=np.int64), r, 2) for r in range(2)]
    assert cuts[0][0] == 0 and cuts[-1][1] == 3 and cuts[0][1] == cuts[1][0]


# ---------------------------------------------------------------------------------------------------------
# The orchestration of paper_2609_35099_b200/sharding.py with real exchanged arrays on CPU ranks.  Stand-ins for
# the library's kernels: the oracle for the convolution, index expressions for the row kernels, and the
# definition of the local renumbering written with numpy set operations.
class _CpuOps:
    def __init__(self, cp):
        self.cp = cp

    def shard_prepare(self, n_nodes, lo, hi, senders, receivers):
        s, r = senders.numpy(), receivers.numpy()
        halo = np.unique(s[(s < lo) | (s >= hi)])                     # ascending global ids
        ls = np.where((s >= lo) & (s < hi), s - lo, (hi - lo) + np.searchsorted(halo, s))
        return (torch.from_numpy(ls.astype(np.int32)), torch.from_numpy((r - lo).astype(np.int32)),
                torch.from_numpy(halo.astype(np.int32)))

    def rows_gather(self, dst, src, ids):
        dst[:] = src[ids.long()]
        return dst

    def rows_add(self, dst, src, ids):
        assert len(torch.unique(ids)) == len(ids)
        dst[ids.long()] += src
        return dst

    def conv_fwd(self, x_local, sh, w, senders, receivers, graph=None):
        return torch.from_numpy(oconv.conv_fwd(self.cp, x_local.numpy(), sh, w, senders.numpy(), receivers.numpy()))

    def conv_bwd(self, x_local, sh, w, senders, receivers, grad_out_local, graph=None):
        return tuple(torch.from_numpy(a) for a in oconv.conv_bwd(self.cp, x_local.numpy(), sh, w, senders.numpy(),
                                                                 receivers.numpy(), grad_out_local.numpy()))


def _sharded_worker(rank, world, port, out_dir):
    from paper_2609_35099_b200 import sharding
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        c = workloads.CONFIGS[1]
        wl = workloads.make_graph(1)
        cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
        x, y, w, g = workloads.make_features(wl, cp.P, cp.D)
        n = wl.n_nodes
        rowptr = np.searchsorted(wl.receivers, np.arange(n + 1), side="left")
        ops = _CpuOps(cp)
        sh = sharding.make_shard(ops, rank, world, n, torch.from_numpy(wl.senders), torch.from_numpy(wl.receivers), rowptr)
        assert sh.halo_ids.numel() > 0 and sh.n_local <= n
        x_local = sharding.gather_x(ops, sh, torch.from_numpy(x[sh.lo:sh.hi]))          # all-gather + row gather
        want_ids = np.concatenate([np.arange(sh.lo, sh.hi), sh.halo_ids.numpy()])
        assert np.array_equal(x_local.numpy(), x[want_ids])                               # exchanged bytes, not copies
        ys, ws_ = y[sh.e_lo:sh.e_hi], w[sh.e_lo:sh.e_hi]
        out_local = ops.conv_fwd(x_local, ys, ws_, sh.senders, sh.receivers)
        g_local = torch.zeros((sh.n_local, cp.D, cp.nq), dtype=torch.float32)
        g_local[:sh.n_owned] = torch.from_numpy(g[sh.lo:sh.hi])
        gx_local, gy, gw = ops.conv_bwd(x_local, ys, ws_, sh.senders, sh.receivers, g_local)
        gx_owned = sharding.reduce_grad_x(ops, sh, gx_local)                              # all-gather + ordered adds
        ref = oconv.conv_fwd(cp, x, y, w, wl.senders, wl.receivers)
        rx, ry, rw = oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)
        assert np.abs(out_local.numpy()[:sh.n_owned] - ref[sh.lo:sh.hi]).max() < 1e-12
        assert np.all(out_local.numpy()[sh.n_owned:] == 0)                                # halo nodes receive nothing here
        assert np.abs(gx_owned.numpy() - rx[sh.lo:sh.hi]).max() < 1e-11
        assert np.abs(gy.numpy() - ry[sh.e_lo:sh.e_hi]).max() < 1e-12
        assert np.abs(gw.numpy() - rw[sh.e_lo:sh.e_hi]).max() < 1e-12
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_convolution_with_exchanged_halo_rows(tmp_path, world):
    mp.spawn(_sharded_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))
