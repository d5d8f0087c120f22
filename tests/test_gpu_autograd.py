"""The torch.autograd wrapper returns what the direct calls return: first derivatives = e3j_conv_bwd, second
derivatives = e3j_conv_bwd_bwd (bit-identical: same kernels, same inputs)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2609_35099_b200 as e3j
from paper_2609_35099_b200 import workloads
from paper_2609_35099_b200.autograd import Graph, conv, conv_radial, conv_vec

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@pytest.mark.parametrize("config,n_atoms", [(2, 192), (1, None)])
def test_autograd_first_and_second_order(config, n_atoms):
    c = workloads.CONFIGS[config]
    wl = workloads.make_graph(config, n_atoms)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], 0)
    x, y, w, g = (_cuda(a) for a in workloads.make_features(wl, plan.n_paths, plan.d_out))
    graph = Graph(wl.n_nodes, _cuda(wl.senders), _cuda(wl.receivers))
    xs, ys, ws = (t.clone().requires_grad_(True) for t in (x, y, w))
    out = conv(plan, graph, xs, ys, ws)
    assert torch.equal(out, e3j.e3j_conv_fwd(plan, x, y, w, graph.senders, graph.receivers, graph.rowptr))
    gx, gy, gw = torch.autograd.grad(out, (xs, ys, ws), grad_outputs=g, create_graph=True)
    dx, dy, dw = e3j.e3j_conv_bwd(plan, x, y, w, graph.senders, graph.receivers, g, graph.rowptr, graph.sender_perm,
                                  graph.colptr)
    assert torch.equal(gx, dx) and torch.equal(gy, dy) and torch.equal(gw, dw)
    # a loss on the gradients (what force matching does): its derivatives are the double backward
    gen = torch.Generator(device=DEV); gen.manual_seed(3)
    ux, uy, uw = (torch.randn(t.shape, generator=gen, device=DEV) for t in (x, y, w))
    loss = (gx * ux).sum() + (gy * uy).sum() + (gw * uw).sum()
    hx, hy, hw = torch.autograd.grad(loss, (xs, ys, ws))
    _, rx, ry, rw = e3j.e3j_conv_bwd_bwd(plan, x, y, w, graph.senders, graph.receivers, g, graph.rowptr,
                                         graph.sender_perm, graph.colptr, ux, uy, uw, gg_out=False)
    torch.cuda.synchronize()
    for a, b, name in ((hx, rx, "x"), (hy, ry, "sh"), (hw, rw, "w")):
        assert float((a - b).abs().max()) <= 1e-6 * float(b.abs().max()), name


def test_autograd_radial_and_edge_vector_forms():
    c = workloads.CONFIGS[2]
    wl = workloads.make_graph(2, 192)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], 0)
    x, y, w, g = (_cuda(a) for a in workloads.make_features(wl, plan.n_paths, plan.d_out))
    h, W = (_cuda(a) for a in workloads.make_radial(wl, plan.n_paths, 64))
    vec = _cuda(wl.vectors.astype(np.float32))
    graph = Graph(wl.n_nodes, _cuda(wl.senders), _cuda(wl.receivers))
    args = (graph.senders, graph.receivers)
    prep = (graph.rowptr, graph.sender_perm, graph.colptr)
    # radial layer; W frozen: its gradient is not asked for and not computed
    xs, hs = x.clone().requires_grad_(True), h.clone().requires_grad_(True)
    out = conv_radial(plan, graph, xs, y, hs, W)
    gx, gh = torch.autograd.grad(out, (xs, hs), grad_outputs=g)
    rx, _, rh, _ = e3j.e3j_conv_radial_bwd(plan, x, y, h, W, *args, g, *prep, grad_sh=False, grad_W=False)
    assert torch.equal(gx, rx) and torch.equal(gh, rh)
    # edge vectors
    vs, ws = vec.clone().requires_grad_(True), w.clone().requires_grad_(True)
    out = conv_vec(plan, graph, x, vs, ws)
    gv, gw = torch.autograd.grad(out, (vs, ws), grad_outputs=g)
    _, rv, rw = e3j.e3j_conv_vec_bwd(plan, x, vec, w, *args, g, *prep, grad_x=False)
    torch.cuda.synchronize()
    assert torch.equal(gv, rv) and torch.equal(gw, rw)


def test_graph_refuses_bad_edge_lists_before_anything_indexes_with_them():
    snd = torch.tensor([0, 1, 2, 1], dtype=torch.int32, device=DEV)
    rcv = torch.tensor([0, 0, 1, 2], dtype=torch.int32, device=DEV)
    assert Graph(3, snd, rcv).rowptr.tolist() == [0, 2, 3, 4]
    with pytest.raises(ValueError):
        Graph(2, snd, rcv)                       # ids up to 2 with two nodes
    with pytest.raises(ValueError):
        Graph(3, snd, torch.tensor([0, 1, 0, 2], dtype=torch.int32, device=DEV))   # receivers decrease
