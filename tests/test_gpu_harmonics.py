"""GPU parity of the harmonics of edge vectors and of the convolution that takes the vectors (through the C ABI)
against the float64 oracle.  Tolerances: float32 arithmetic against float64, 1e-5 of each irreducible block's
largest value for the convolution (as for the other calls); 3e-6 absolute for a harmonic (components are O(1))."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2609_35099_b200 as e3j
from oracle import conv as oconv, sh as osh
from paper_2609_35099_b200 import workloads
from parity_util import assert_blockwise_close, blocks_of_paths

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _vectors(n, seed):
    rng = np.random.default_rng(seed)
    v = rng.standard_normal((n, 3))
    v *= rng.uniform(0.5, 5.0, size=(n, 1)) / np.linalg.norm(v, axis=1, keepdims=True)
    return v.astype(np.float32)


@pytest.mark.parametrize("lmax", [0, 1, 2, 3])
def test_harmonics_and_their_gradient_match_the_oracle(lmax):
    n = 70_001   # several blocks and a ragged tail
    vec = _vectors(n, 3 + lmax)
    g = np.random.default_rng(9).standard_normal((n, (lmax + 1) ** 2)).astype(np.float32)
    y = e3j.e3j_harmonics_fwd(lmax, _cuda(vec))
    gv = e3j.e3j_harmonics_bwd(lmax, _cuda(vec), _cuda(g))
    y2 = e3j.e3j_harmonics_fwd(lmax, _cuda(vec))
    torch.cuda.synchronize()
    assert torch.equal(y, y2)
    want = osh.real_sh_all_of_vectors(lmax, vec.astype(np.float64))
    assert np.abs(y.cpu().numpy() - want).max() < 3e-6
    sample = np.random.default_rng(1).choice(n, 4000, replace=False)   # the oracle's differences are slow
    want_g = osh.real_sh_all_vjp(lmax, vec[sample].astype(np.float64), g[sample].astype(np.float64))
    got_g = gv.cpu().numpy()[sample].astype(np.float64)
    assert np.abs(got_g - want_g).max() <= 1e-5 * max(np.abs(want_g).max(), 1.0)
    # direction only: the gradient has no radial part
    radial = np.einsum("ni,ni->n", gv.cpu().numpy().astype(np.float64), vec.astype(np.float64))
    assert np.abs(radial).max() < 2e-5


def test_harmonics_of_a_zero_vector_are_finite_and_empty_input_is_fine():
    vec = torch.zeros((3, 3), device=DEV)
    y = e3j.e3j_harmonics_fwd(3, vec)
    gv = e3j.e3j_harmonics_bwd(3, vec, torch.ones((3, 16), device=DEV))
    assert torch.isfinite(y).all() and torch.all(y[:, 0] == 1.0)
    assert torch.all(gv == 0.0)
    assert e3j.e3j_harmonics_fwd(2, torch.empty((0, 3), device=DEV)).shape == (0, 9)
    with pytest.raises(RuntimeError):
        e3j.e3j_harmonics_fwd(4, torch.ones((5, 3), device=DEV))


@pytest.mark.parametrize("config,n_atoms,flags", [
    (1, None, 0),                              # table-driven kernels: harmonics through the workspace
    (2, 192, 0),                               # specialised kernels: harmonics formed in the table warp
    (2, 648, 0),
    (2, 192, e3j.E3J_PLAN_GENERIC_ONLY),
    (3, 300, 0),
])
def test_convolution_on_edge_vectors(config, n_atoms, flags):
    c = workloads.CONFIGS[config]
    wl = workloads.make_graph(config, n_atoms)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], flags)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    x, _, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    vec = wl.vectors.astype(np.float32)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    dx, dv, dw, dg = _cuda(x), _cuda(vec), _cuda(w), _cuda(g)
    graph = e3j.e3j_graph_prepare(wl.n_nodes, snd, rcv)
    runs = []
    for prepared in (True, False):
        rp, pm, cpt = graph if prepared else (None, None, None)
        out = e3j.e3j_conv_vec_fwd(plan, dx, dv, dw, snd, rcv, rp)
        runs.append((out, *e3j.e3j_conv_vec_bwd(plan, dx, dv, dw, snd, rcv, dg, rp, pm, cpt)))
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    out, gx, gvec, gw = runs[0]
    ref = oconv.conv_vec_fwd(cp, x, vec, w, wl.senders, wl.receivers)
    rx, rvec, rw = oconv.conv_vec_bwd(cp, x, vec, w, wl.senders, wl.receivers, g)
    assert_blockwise_close(out.cpu().numpy(), ref, blocks_of_paths(cp.paths, "out"), what="out")
    assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="grad_x")
    assert_blockwise_close(gw.cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), what="grad_w")
    assert_blockwise_close(gvec.cpu().numpy(), rvec, [(0, 3)], what="grad_vec")
    # the same numbers as the two-step form: harmonics first, then the convolution on them
    y = e3j.e3j_harmonics_fwd(c["sh_lmax"], dv)
    two_step = e3j.e3j_conv_fwd(plan, dx, y, dw, snd, rcv, graph[0])
    assert torch.allclose(out, two_step, rtol=0, atol=1e-6 * float(out.abs().max()))
    # partial gradients (the convolution's backward may take another kernel then: same values, other rounding)
    only_vec = e3j.e3j_conv_vec_bwd(plan, dx, dv, dw, snd, rcv, dg, *graph, grad_x=False, grad_w=False)
    assert only_vec[0] is None and only_vec[2] is None
    assert_blockwise_close(only_vec[1].cpu().numpy(), rvec, [(0, 3)], what="grad_vec alone")


@pytest.mark.parametrize("config,n_atoms,hidden", [(2, 192, 64), (2, 648, 32), (1, None, 16), (3, 300, 64)])
def test_radial_forward_on_edge_vectors(config, n_atoms, hidden):
    """e3j_conv_radial_vec_fwd against the oracle's conv_radial_fwd on the oracle's harmonics of the vectors, and
    against the call that takes ready-made harmonics."""
    c = workloads.CONFIGS[config]
    wl = workloads.make_graph(config, n_atoms)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], 0)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    x, _, _, _ = workloads.make_features(wl, plan.n_paths, plan.d_out)
    h, W = workloads.make_radial(wl, plan.n_paths, hidden)
    vec = wl.vectors.astype(np.float32)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    out = e3j.e3j_conv_radial_vec_fwd(plan, _cuda(x), _cuda(vec), _cuda(h), _cuda(W), snd, rcv)
    out2 = e3j.e3j_conv_radial_vec_fwd(plan, _cuda(x), _cuda(vec), _cuda(h), _cuda(W), snd, rcv)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    assert torch.equal(out, out2)
    y = osh.real_sh_all_of_vectors(c["sh_lmax"], vec.astype(np.float64)).astype(np.float32)
    ref = oconv.conv_radial_fwd(cp, x, y, h, W, wl.senders, wl.receivers)
    assert_blockwise_close(out.cpu().numpy(), ref, blocks_of_paths(cp.paths, "out"), what="out")
    with_sh = e3j.e3j_conv_radial_fwd(plan, _cuda(x), e3j.e3j_harmonics_fwd(c["sh_lmax"], _cuda(vec)), _cuda(h), _cuda(W),
                                      snd, rcv)
    assert torch.allclose(out, with_sh, rtol=0, atol=1e-6 * float(out.abs().max()))
    # the backward: grad_x, grad_h, grad_W as the oracle's radial backward on those harmonics, grad_vec through its
    # harmonics gradient
    g = workloads.make_features(wl, plan.n_paths, plan.d_out)[3]
    gx, gvec, gh, gW = e3j.e3j_conv_radial_vec_bwd(plan, _cuda(x), _cuda(vec), _cuda(h), _cuda(W), snd, rcv, _cuda(g))
    torch.cuda.synchronize()
    rx, ry, rh, rW = oconv.conv_radial_bwd(cp, x, y, h, W, wl.senders, wl.receivers, g)
    rvec = osh.real_sh_all_vjp(c["sh_lmax"], vec.astype(np.float64), ry)
    assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="grad_x")
    assert_blockwise_close(gvec.cpu().numpy(), rvec, [(0, 3)], what="grad_vec")
    assert_blockwise_close(gh.cpu().numpy(), rh, [(0, hidden)], what="grad_h")
    assert np.abs(gW.cpu().numpy() - rW).max() <= 1e-5 * np.abs(rW).max()


def test_convolution_on_edge_vectors_checks_its_workspace():
    """The binding refuses a short workspace; the library itself answers E3J_ERR_WORKSPACE (called directly)."""
    import ctypes
    c = workloads.CONFIGS[2]
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], 0)
    wl = workloads.make_graph(2, 192)
    x, _, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    dx, dv, dw = _cuda(x), _cuda(wl.vectors.astype(np.float32)), _cuda(w)
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(ValueError):
        e3j.e3j_conv_vec_fwd(plan, dx, dv, dw, snd, rcv, workspace=small)
    need = e3j.e3j_conv_vec_bwd_workspace_bytes(plan, wl.n_nodes, wl.n_edges)
    assert need >= e3j.e3j_conv_bwd_workspace_bytes(plan, wl.n_nodes, wl.n_edges) + 2 * 4 * wl.n_edges * plan.d_sh
    out = torch.empty((wl.n_nodes, plan.d_out, plan.n_channels), device=DEV)
    p = lambda t_: ctypes.c_void_p(t_.data_ptr())
    rc = e3j._load().e3j_conv_vec_fwd(plan.handle, wl.n_nodes, wl.n_edges, p(dx), p(dv), p(dw), p(snd), p(rcv), None,
                                      p(out), p(small), 0, None)
    assert rc != 0 and "workspace" in e3j.e3j_status_string(rc).lower()
