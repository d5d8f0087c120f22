"""The receiver-sharded call path on one GPU: the shards of a three-rank split run one after the other through
the library's kernels (local renumbering, halo row gather, convolution, ordered addition of the grad_x shares)
and are compared with the unsharded call and the oracle.  The exchange between real ranks is covered on CPU
ranks in test_sharding_gloo.py; here the gathered blocks are simply the full arrays."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2609_35099_b200 as e3j
from oracle import conv as oconv
from paper_2609_35099_b200 import sharding, workloads
from parity_util import assert_blockwise_close, blocks_of_paths

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _run_sharded(plan, wl, x, y, w, g, world):
    n = wl.n_nodes
    ops = sharding.CudaOps(plan)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    rowptr = np.searchsorted(wl.receivers, np.arange(n + 1), side="left")
    dx, dy, dw, dg = _cuda(x), _cuda(y), _cuda(w), _cuda(g)
    shards, results = [], []
    for r in range(world):
        sh = sharding.make_shard(ops, r, world, n, snd, rcv, rowptr)
        ids = torch.cat([torch.arange(sh.lo, sh.hi, dtype=torch.int32, device=DEV), sh.halo_ids])
        x_local = torch.empty((sh.n_local, plan.d_in, plan.n_channels), device=DEV)
        ops.rows_gather(x_local, dx, ids)
        graph = ops.graph_prepare(sh.n_local, sh.senders, sh.receivers)
        ys, ws_ = dy[sh.e_lo:sh.e_hi].contiguous(), dw[sh.e_lo:sh.e_hi].contiguous()
        out_local = ops.conv_fwd(x_local, ys, ws_, sh.senders, sh.receivers, graph)
        g_local = torch.zeros((sh.n_local, plan.d_out, plan.n_channels), device=DEV)
        g_local[:sh.n_owned] = dg[sh.lo:sh.hi]
        gx_local, gy, gw = ops.conv_bwd(x_local, ys, ws_, sh.senders, sh.receivers, g_local, graph)
        shards.append(sh)
        results.append((out_local, gx_local, gy, gw))
    out = torch.cat([res[0][:sh.n_owned] for sh, res in zip(shards, results)])
    gy = torch.cat([res[2] for res in results])
    gw = torch.cat([res[3] for res in results])
    shares = [(sh.halo_ids, res[1][sh.n_owned:]) for sh, res in zip(shards, results)]
    gx = torch.cat([sharding.add_shares(ops, sh, res[1][:sh.n_owned].clone(), shares) for sh, res in zip(shards, results)])
    torch.cuda.synchronize()
    return shards, out, gx, gy, gw


@pytest.mark.parametrize("config,n_atoms,world", [(2, 648, 3), (1, None, 2), (5, 3000, 4)])
def test_sharded_calls_match_the_unsharded_call(config, n_atoms, world):
    c = workloads.CONFIGS[config]
    wl = workloads.make_graph(config, n_atoms)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    shards, out, gx, gy, gw = _run_sharded(plan, wl, x, y, w, g, world)
    again = _run_sharded(plan, wl, x, y, w, g, world)[1:]
    for a, b in zip((out, gx, gy, gw), again):
        assert torch.equal(a, b), "sharded results differ between two runs"
    # local numbering: owned nodes first, then the halo in ascending global order, no owned node in the halo
    for sh in shards:
        h = sh.halo_ids.cpu().numpy()
        assert np.all(np.diff(h) > 0) and not np.any((h >= sh.lo) & (h < sh.hi))
        s_local = sh.senders.cpu().numpy()
        glob = np.concatenate([np.arange(sh.lo, sh.hi), h])
        assert np.array_equal(glob[s_local], wl.senders[sh.e_lo:sh.e_hi])
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    whole_out = e3j.e3j_conv_fwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv)
    _, whole_gy, whole_gw = e3j.e3j_conv_bwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv, _cuda(g))
    # edge-local gradients do not depend on how the edge list is cut
    assert torch.equal(gy, whole_gy) and torch.equal(gw, whole_gw)
    ref = oconv.conv_fwd(cp, x, y, w, wl.senders, wl.receivers)
    rx, _, _ = oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)
    assert_blockwise_close(out.cpu().numpy(), ref, blocks_of_paths(cp.paths, "out"), what="sharded out")
    assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="sharded grad_x")
    assert_blockwise_close(out.cpu().numpy(), whole_out.cpu().numpy().astype(np.float64), blocks_of_paths(cp.paths, "out"),
                           what="sharded against whole")
