"""GPU parity of the calls that take the radial network's last layer (h, W) in place of the edge weights.

The product s = h W runs on the tensor cores with float32 operands split into TF32 pairs; it is compared with
the float64 product, and the convolutions built on it with the oracle's conv_radial_fwd / conv_radial_bwd, per
irreducible block at the tolerance of the other parity tests (1e-5 of the block's largest oracle value).
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2609_35099_b200 as e3j
from oracle import conv as oconv
from paper_2609_35099_b200 import workloads
from parity_util import assert_blockwise_close, blocks_of_paths

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(autouse=True)
def _release_device_memory():
    yield
    import gc
    gc.collect()
    if torch.cuda.is_available():
        torch.cuda.empty_cache()


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@pytest.mark.parametrize("irreps,lmax,edges,hidden", [
    ("128x0e+128x1o", 3, 1000, 64),    # 13 column blocks, several edge tiles, ragged last tile
    ("128x0e+128x1o", 3, 77, 8),       # one short k chunk
    ("128x0e+128x1o", 3, 300, 40),     # ragged second k chunk
    ("8x0e+8x1o", 2, 513, 64),         # 120 columns: one ragged column block
    ("64x0e+64x1o+64x2e+64x3o", 3, 260, 96),   # three k chunks
    ("128x0e+128x1o", 3, 700, 128),    # four k chunks: the largest resident block of W^T
    ("128x0e+128x1o", 3, 390, 160),    # five k chunks: W^T converted per tile (wide hidden layer)
    ("128x0e+128x1o", 3, 0, 64),
])
def test_radial_weights_match_the_float64_product(irreps, lmax, edges, hidden):
    plan = e3j.e3j_plan_create(irreps, lmax, None, lmax)
    rng = np.random.default_rng(hidden + edges)
    C = plan.n_paths * plan.n_channels
    h = rng.standard_normal((edges, hidden)).astype(np.float32)
    W = (rng.standard_normal((hidden, C)) / np.sqrt(hidden)).astype(np.float32)
    out = torch.full((edges, plan.n_paths, plan.n_channels), float("nan"), device=DEV)
    e3j.e3j_radial_weights(plan, _cuda(h), _cuda(W), out=out)
    out2 = torch.full_like(out, float("nan"))
    e3j.e3j_radial_weights(plan, _cuda(h), _cuda(W), out=out2)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    assert torch.equal(out, out2)
    if edges == 0:
        return
    want = (h.astype(np.float64) @ W.astype(np.float64)).reshape(edges, plan.n_paths, plan.n_channels)
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # float32-level accuracy: three TF32 products per float32 product
    assert np.abs(got - want).max() <= 2e-6 * np.abs(want).max()


def _radial_case(config, n_atoms, hidden, flags=0):
    c = workloads.CONFIGS[config]
    wl = workloads.make_graph(config, n_atoms)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"], flags)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    x, y, _, g = workloads.make_features(wl, plan.n_paths, plan.d_out, with_weights=False)
    h, W = workloads.make_radial(wl, plan.n_paths, hidden)
    return wl, plan, cp, x, y, h, W, g


def _layer_blocks(cp):
    return [(p.k * cp.nq, (p.k + 1) * cp.nq) for p in cp.paths]


def run_radial_parity(wl, plan, cp, x, y, h, W, g, prepared=True):
    n = wl.n_nodes
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    dx, dy, dh, dW, dg = _cuda(x), _cuda(y), _cuda(h), _cuda(W), _cuda(g)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv) if prepared else (None, None, None)
    runs = []
    for _ in range(2):
        out = e3j.e3j_conv_radial_fwd(plan, dx, dy, dh, dW, snd, rcv, rowptr)
        grads = e3j.e3j_conv_radial_bwd(plan, dx, dy, dh, dW, snd, rcv, dg, rowptr, perm, colptr)
        runs.append((out, *grads))
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    for a, b in zip(*runs):
        assert torch.equal(a, b), "results differ between two runs"
    out, gx, gy, gh, gW = runs[0]
    ref = oconv.conv_radial_fwd(cp, x, y, h, W, wl.senders, wl.receivers)
    rx, ry, rh, rW = oconv.conv_radial_bwd(cp, x, y, h, W, wl.senders, wl.receivers, g)
    return [
        assert_blockwise_close(out.cpu().numpy(), ref, blocks_of_paths(cp.paths, "out"), what="out"),
        assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="grad_x"),
        assert_blockwise_close(gy.cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), what="grad_sh"),
        assert_blockwise_close(gh.cpu().numpy(), rh, [(0, h.shape[1])], what="grad_h"),
        assert_blockwise_close(gW.cpu().numpy(), rW, _layer_blocks(cp), what="grad_W"),
    ]


@pytest.mark.parametrize("config,n_atoms,hidden,flags", [
    (1, None, 16, 0),                              # table-driven kernels, 72 weight columns
    (2, 192, 64, 0),
    (2, 648, 64, 0),
    (2, 192, 64, e3j.E3J_PLAN_GENERIC_ONLY),
    (2, 648, 64, e3j.E3J_PLAN_RADIAL_MATERIALISE),   # two-step form although the plan has the in-kernel one
    (3, 300, 64, 0),
    (5, 3000, 32, 0),
    (2, 192, 128, 0),                              # two blocks of 64 hidden units in the gradient products
    (2, 192, 160, 0),                              # three, the last one half full; W^T converted per tile
])
def test_conv_radial_small(config, n_atoms, hidden, flags):
    run_radial_parity(*_radial_case(config, n_atoms, hidden, flags))


def test_conv_radial_without_prepared_graph_and_partial_gradients():
    wl, plan, cp, x, y, h, W, g = _radial_case(2, 192, 64)
    run_radial_parity(wl, plan, cp, x, y, h, W, g, prepared=False)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    gx, gy, gh, gW = e3j.e3j_conv_radial_bwd(plan, _cuda(x), _cuda(y), _cuda(h), _cuda(W), snd, rcv, _cuda(g),
                                             grad_x=False, grad_sh=False, grad_W=False)
    assert gx is None and gy is None and gW is None
    _, _, rh, _ = oconv.conv_radial_bwd(cp, x, y, h, W, wl.senders, wl.receivers, g)
    assert_blockwise_close(gh.cpu().numpy(), rh, [(0, h.shape[1])], what="grad_h alone")


def test_conv_radial_full_size():
    """Config 2 at the size bench.py times, every element."""
    run_radial_parity(*_radial_case(2, None, 64))


def test_conv_radial_empty_graph_and_bad_arguments():
    plan = e3j.e3j_plan_create("128x0e+128x1o", 3, None, 3)
    x = torch.randn((5, plan.d_in, plan.n_channels), device=DEV)
    e_i = torch.zeros(0, dtype=torch.int32, device=DEV)
    W = torch.randn((64, plan.n_paths * plan.n_channels), device=DEV)
    out = e3j.e3j_conv_radial_fwd(plan, x, torch.zeros((0, plan.d_sh), device=DEV), torch.zeros((0, 64), device=DEV),
                                  W, e_i, e_i)
    assert torch.count_nonzero(out) == 0
    g = torch.randn((5, plan.d_out, plan.n_channels), device=DEV)
    gx, gy, gh, gW = e3j.e3j_conv_radial_bwd(plan, x, torch.zeros((0, plan.d_sh), device=DEV),
                                             torch.zeros((0, 64), device=DEV), W, e_i, e_i, g)
    assert torch.count_nonzero(gx) == 0 and torch.count_nonzero(gW) == 0 and gh.shape == (0, 64)
    W6 = torch.randn((6, plan.n_paths * plan.n_channels), device=DEV)   # hidden not a multiple of 4
    with pytest.raises(e3j.E3JError) as err:
        e3j.e3j_radial_weights(plan, torch.zeros((3, 6), device=DEV), W6)
    assert err.value.status == e3j.E3J_ERR_UNSUPPORTED


def _seeded_normal(shape, seed):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(seed)
    return torch.randn(shape, generator=gen, device=DEV, dtype=torch.float32)


def _range_boundary_receivers(rowptr, n_ranges):
    """Receivers whose slot groups are cut by a CTA range boundary of the forward that forms its edge scalars in
    the kernel (host restatement of its split: 8 slots per group, tiles of 16 groups, equal tile counts)."""
    deg = np.diff(rowptr)
    groups = (deg + 7) // 8
    first_group = np.concatenate([[0], np.cumsum(groups)])
    n_groups = int(first_group[-1])
    tiles_total = (n_groups + 15) // 16
    tiles_per = (tiles_total + n_ranges - 1) // n_ranges
    cuts = [16 * tiles_per * r for r in range(1, n_ranges) if 16 * tiles_per * r < n_groups]
    rec = np.searchsorted(first_group, cuts, side="right") - 1
    return np.unique(np.concatenate([rec, np.maximum(rec - 1, 0)]))


def test_conv_radial_config5_full_size_sampled():
    """100k atoms, 4.77 M edges: the weights (31 GB as an array) exist only inside the forward kernel.  Sampled
    receivers, every receiver cut by a CTA range boundary included, are recomputed by the oracle; the backward is
    checked on the sampled receivers' edges (grad_sh, grad_h), on sampled senders (grad_x) and, for grad_W and the
    whole of grad_h, by the adjoint identities <grad_W, W> = <grad_h, h> = <grad_out, out>."""
    c = workloads.CONFIGS[5]
    wl = workloads.make_graph(5)
    n, e, H = wl.n_nodes, wl.n_edges, 64
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    rng = np.random.Generator(np.random.PCG64([5, 3]))
    x = rng.standard_normal((n, plan.d_in, plan.n_channels), dtype=np.float32)
    y = workloads.edge_harmonics(wl)
    W = (rng.standard_normal((H, plan.n_paths * plan.n_channels), dtype=np.float32) / np.float32(8.0))
    dx_, dy_, dW_ = _cuda(x), _cuda(y), _cuda(W)
    dh_ = _seeded_normal((e, H), 53)
    dg_ = _seeded_normal((n, plan.d_out, plan.n_channels), 54)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    out = e3j.e3j_conv_radial_fwd(plan, dx_, dy_, dh_, dW_, snd, rcv, rowptr)
    out2 = e3j.e3j_conv_radial_fwd(plan, dx_, dy_, dh_, dW_, snd, rcv, rowptr)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    assert torch.equal(out, out2), "forward differs between two runs"
    del out2
    gx, gy, gh, gW = e3j.e3j_conv_radial_bwd(plan, dx_, dy_, dh_, dW_, snd, rcv, dg_, rowptr, perm, colptr)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0

    rp = rowptr.cpu().numpy()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    deg = np.diff(rp)
    pick = np.unique(np.concatenate([rng.choice(n, 30, replace=False), np.argsort(deg)[-4:], np.argsort(deg)[:4], [0, n - 1],
                                     _range_boundary_receivers(rp, max(1, sms // 8))]))
    out_blocks = blocks_of_paths(cp.paths, "out")
    for b in pick:
        e0, e1 = int(rp[b]), int(rp[b + 1])
        nodes, local = np.unique(np.concatenate([wl.senders[e0:e1], [b]]), return_inverse=True)
        lb = int(local[-1])
        hs = dh_[e0:e1].cpu().numpy()
        l_snd, l_rcv = local[:-1].astype(np.int32), np.full(e1 - e0, lb, np.int32)
        ref = oconv.conv_radial_fwd(cp, x[nodes], y[e0:e1], hs, W, l_snd, l_rcv)
        assert_blockwise_close(out[b].cpu().numpy()[None], ref[lb][None], out_blocks, what=f"out[{b}]")
        gs = np.zeros((len(nodes), plan.d_out, plan.n_channels), np.float32)
        gs[lb] = dg_[b].cpu().numpy()
        _, ry, rh, _ = oconv.conv_radial_bwd(cp, x[nodes], y[e0:e1], hs, W, l_snd, l_rcv, gs)
        if e1 > e0:
            assert_blockwise_close(gy[e0:e1].cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), what=f"grad_sh[{b}]")
            assert_blockwise_close(gh[e0:e1].cpu().numpy(), rh, [(0, H)], what=f"grad_h[{b}]")
    senders_sorted, cptr = perm.cpu().numpy(), colptr.cpu().numpy()
    for a in rng.choice(n, 12, replace=False):
        ids = np.sort(senders_sorted[cptr[a]:cptr[a + 1]])
        nodes, l_rcv = np.unique(wl.receivers[ids], return_inverse=True)
        xs = np.zeros((len(nodes) + 1, plan.d_in, plan.n_channels), np.float32)
        xs[-1] = x[a]
        gs = np.concatenate([dg_[torch.from_numpy(nodes).to(DEV)].cpu().numpy(),
                             np.zeros((1, plan.d_out, plan.n_channels), np.float32)])
        hs = dh_[torch.from_numpy(ids).to(DEV)].cpu().numpy()
        rx, _, _, _ = oconv.conv_radial_bwd(cp, xs, y[ids], hs, W, np.full(len(ids), len(nodes), np.int32),
                                            l_rcv.astype(np.int32), gs)
        assert_blockwise_close(gx[a].cpu().numpy()[None], rx[-1][None], blocks_of_paths(cp.paths, "x"), what=f"grad_x[{a}]")
    # the map is linear in W and in h: <grad_W, W> = <grad_h, h> = <grad_out, out>, sums in float64
    ref = float((dg_.double() * out.double()).sum().item())
    via_W = float((gW.double() * dW_.double()).sum().item())
    via_h = float((gh.double() * dh_.double()).sum().item())
    scale = float((dg_.double() * out.double()).abs().sum().item())
    assert abs(via_W - ref) <= 1e-6 * scale and abs(via_h - ref) <= 1e-6 * scale, (ref, via_W, via_h, scale)


def test_radial_calls_can_be_captured_in_a_cuda_graph():
    """The calls through (h, W) only enqueue kernels once the graph is prepared and the caller owns outputs and
    workspaces (the tensor maps of the gradient products travel as kernel arguments): a captured forward +
    backward replays to the bits of the eager calls."""
    wl, plan, cp, x, y, h, W, g = _radial_case(2, 192, 64)
    n, e = wl.n_nodes, wl.n_edges
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    dx, dy, dh, dW, dg = _cuda(x), _cuda(y), _cuda(h), _cuda(W), _cuda(g)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    u8 = lambda nbytes: torch.empty(max(nbytes, 256), dtype=torch.uint8, device=DEV)
    ws_f = u8(e3j.e3j_conv_radial_fwd_workspace_bytes(plan, n, e, 64))
    ws_b = u8(e3j.e3j_conv_radial_bwd_workspace_bytes(plan, n, e, 64))
    out = torch.empty_like(dg)
    grads = [torch.empty_like(t) for t in (dx, dy, dh, dW)]

    def step():
        e3j.e3j_conv_radial_fwd(plan, dx, dy, dh, dW, snd, rcv, rowptr, out=out, workspace=ws_f)
        e3j.e3j_conv_radial_bwd(plan, dx, dy, dh, dW, snd, rcv, dg, rowptr, perm, colptr, grad_x=grads[0],
                                grad_sh=grads[1], grad_h=grads[2], grad_W=grads[3], workspace=ws_b)

    step()   # eager: first use sets the kernels' attributes, uploads the tables and looks the map encoder up
    torch.cuda.synchronize()
    eager = [t.clone() for t in (out, *grads)]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in (out, *grads):
        t.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(eager, (out, *grads)):
        assert torch.equal(a, b)
    assert e3j.e3j_plan_device_status(plan) == 0
