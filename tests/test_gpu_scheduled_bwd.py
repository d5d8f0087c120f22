"""GPU parity of the scheduled backward (e3j_conv_bwd_scheduled over an order from e3j_bwd_schedule_build) against
the float64 oracle and against e3j_conv_bwd: same tolerance as the other calls (1e-5 of each irreducible block's
largest value), bit-identical from run to run; grad_sh and grad_w come from the same per-edge arithmetic as in
e3j_conv_bwd and must be bit-identical to it, grad_x is summed in another fixed order."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2609_35099_b200 as e3j
from oracle import conv as oconv
from paper_2609_35099_b200 import workloads
from parity_util import assert_blockwise_close, blocks_of_paths

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _case(n_atoms):
    c = workloads.CONFIGS[2]
    wl = workloads.make_graph(2, n_atoms)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], 0)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    return wl, plan, cp, workloads.make_features(wl, plan.n_paths, plan.d_out)


@pytest.mark.parametrize("n_atoms", [192, 648, 1029])
def test_scheduled_backward_matches_the_oracle_and_the_plain_backward(n_atoms):
    wl, plan, cp, (x, y, w, g) = _case(n_atoms)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    dx, dy, dw, dg = _cuda(x), _cuda(y), _cuda(w), _cuda(g)
    sched = e3j.e3j_bwd_schedule_build(plan, wl.n_nodes, snd, rcv)
    runs = [e3j.e3j_conv_bwd_scheduled(plan, dx, dy, dw, sched, dg) for _ in range(2)]
    plain = e3j.e3j_conv_bwd(plan, dx, dy, dw, snd, rcv, dg)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    gx, gy, gw = runs[0]
    rx, ry, rw = oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)
    assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="grad_x")
    assert_blockwise_close(gy.cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), what="grad_sh")
    assert_blockwise_close(gw.cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), what="grad_w")
    assert torch.equal(gy, plain[1]) and torch.equal(gw, plain[2])


def test_scheduled_backward_full_size_against_the_plain_backward():
    """Bench workload: the oracle has checked the plain backward at this size; the scheduled one must agree with it to
    rounding in grad_x and exactly in the per-edge gradients."""
    wl, plan, cp, (x, y, w, g) = _case(None)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    dx, dy, dw, dg = _cuda(x), _cuda(y), _cuda(w), _cuda(g)
    sched = e3j.e3j_bwd_schedule_build(plan, wl.n_nodes, snd, rcv)
    gx, gy, gw = e3j.e3j_conv_bwd_scheduled(plan, dx, dy, dw, sched, dg)
    px, py, pw = e3j.e3j_conv_bwd(plan, dx, dy, dw, snd, rcv, dg)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    assert torch.equal(gy, py) and torch.equal(gw, pw)
    scale = float(px.abs().max())
    assert float((gx - px).abs().max()) <= 2e-6 * scale


def test_a_schedule_of_another_shape_is_refused_not_followed():
    """A schedule whose header does not match the kernel (here: zeros) sets the plan's status word; nothing is read
    beyond the header."""
    wl, plan, cp, (x, y, w, g) = _case(192)
    bogus = torch.zeros(e3j.e3j_bwd_schedule_bytes(plan, wl.n_nodes, wl.n_edges), dtype=torch.uint8, device=DEV)
    e3j.e3j_conv_bwd_scheduled(plan, _cuda(x), _cuda(y), _cuda(w), bogus, _cuda(g))
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 3
    # plans without the kernel say so
    c = workloads.CONFIGS[3]
    other = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], 0)
    assert e3j.e3j_bwd_schedule_bytes(other, 10, 10) == 0


def test_scheduled_backward_on_sparse_and_empty_graphs():
    """Isolated nodes, senders without a run in most ranges, duplicate edges, and no edges at all."""
    c = workloads.CONFIGS[2]
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], 0)
    rng = np.random.default_rng(5)
    for n, e in ((400, 900), (50, 2000), (7, 3), (300, 0)):
        snd = rng.integers(0, n, size=e).astype(np.int32)
        rcv = np.sort(rng.integers(0, max(n // 2, 1), size=e)).astype(np.int32)   # the upper half receives nothing
        x = rng.standard_normal((n, plan.d_in, plan.n_channels)).astype(np.float32)
        y = rng.standard_normal((e, plan.d_sh)).astype(np.float32)
        w = rng.standard_normal((e, plan.n_paths, plan.n_channels)).astype(np.float32)
        g = rng.standard_normal((n, plan.d_out, plan.n_channels)).astype(np.float32)
        ds, dr = _cuda(snd), _cuda(rcv)
        sched = e3j.e3j_bwd_schedule_build(plan, n, ds, dr)
        gx, gy, gw = e3j.e3j_conv_bwd_scheduled(plan, _cuda(x), _cuda(y), _cuda(w), sched, _cuda(g))
        px, py, pw = e3j.e3j_conv_bwd(plan, _cuda(x), _cuda(y), _cuda(w), ds, dr, _cuda(g))
        torch.cuda.synchronize()
        assert e3j.e3j_plan_device_status(plan) == 0
        assert torch.equal(gy, py) and torch.equal(gw, pw)
        scale = max(float(px.abs().max()), 1e-30)
        assert float((gx - px).abs().max()) <= 2e-6 * scale, (n, e)


@pytest.mark.parametrize("irreps,lmax,irreps_out,out_lmax", [
    ("128x0e+128x1o", 3, "0e+1o+2e+3o", -1),   # natural-parity outputs
    ("64x0e+64x1o", 3, None, 3),                # two channels per lane, ten edges per tile
    ("128x0e+128x1o", 2, None, 2),              # nine harmonics (4-byte gathers)
])
def test_scheduled_backward_of_the_other_signatures(irreps, lmax, irreps_out, out_lmax):
    wl = workloads.make_graph(2, 648)
    plan = e3j.e3j_plan_create(irreps, lmax, irreps_out, out_lmax, 0)
    assert e3j.e3j_bwd_schedule_bytes(plan, wl.n_nodes, wl.n_edges) > 0
    cp = oconv.Coupling(irreps, lmax, irreps_out, None if out_lmax < 0 else out_lmax)
    rng = np.random.default_rng(17)
    n, e = wl.n_nodes, wl.n_edges
    x = rng.standard_normal((n, plan.d_in, plan.n_channels)).astype(np.float32)
    y = rng.standard_normal((e, plan.d_sh)).astype(np.float32)
    w = rng.standard_normal((e, plan.n_paths, plan.n_channels)).astype(np.float32)
    g = rng.standard_normal((n, plan.d_out, plan.n_channels)).astype(np.float32)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    sched = e3j.e3j_bwd_schedule_build(plan, n, snd, rcv)
    gx, gy, gw = e3j.e3j_conv_bwd_scheduled(plan, _cuda(x), _cuda(y), _cuda(w), sched, _cuda(g))
    px, py, pw = e3j.e3j_conv_bwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv, _cuda(g))
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    assert torch.equal(gy, py) and torch.equal(gw, pw)
    rx, ry, rw = oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)
    assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="grad_x")
    assert_blockwise_close(gy.cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), what="grad_sh")
    assert_blockwise_close(gw.cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), what="grad_w")
