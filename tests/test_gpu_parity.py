"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by element.

Tolerance (fp32 arithmetic against an fp64 reference): max abs error <= 1e-5 * max|oracle| per
irreducible block; results must be bit-identical from run to run.
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
    """The full-size cases hold tens of GB; hand cached blocks back between tests."""
    yield
    import gc
    gc.collect()
    if torch.cuda.is_available():
        torch.cuda.empty_cache()


def _cuda(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def make_case(config, n_atoms=None, irreps_out="default", flags=0):
    c = workloads.CONFIGS[config]
    iro = c["irreps_out"] if irreps_out == "default" else irreps_out
    olm = c["out_lmax"] if iro is None else -1
    wl = workloads.make_graph(config, n_atoms)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], iro, olm, flags)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], iro, None if olm < 0 else olm)
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    return wl, plan, cp, x, y, w, g


def run_conv_parity(wl, plan, cp, x, y, w, g, prepared=True):
    n, e = wl.n_nodes, wl.n_edges
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    dx, dy, dw, dg = _cuda(x), _cuda(y), _cuda(w), _cuda(g)
    if prepared:
        rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    else:
        rowptr = perm = colptr = None
    out = e3j.e3j_conv_fwd(plan, dx, dy, dw, snd, rcv, rowptr)
    gx, gy, gw = e3j.e3j_conv_bwd(plan, dx, dy, dw, snd, rcv, dg, rowptr, perm, colptr)
    out2 = e3j.e3j_conv_fwd(plan, dx, dy, dw, snd, rcv, rowptr)
    gx2, gy2, gw2 = e3j.e3j_conv_bwd(plan, dx, dy, dw, snd, rcv, dg, rowptr, perm, colptr)
    torch.cuda.synchronize()
    for a, b in ((out, out2), (gx, gx2), (gy, gy2), (gw, gw2)):
        assert torch.equal(a, b), "results differ between two runs"
    ref = oconv.conv_fwd(cp, x, y, w, wl.senders, wl.receivers)
    rx, ry, rw = oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)
    worst = [
        assert_blockwise_close(out.cpu().numpy(), ref, blocks_of_paths(cp.paths, "out"), what="out"),
        assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="grad_x"),
        assert_blockwise_close(gy.cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), what="grad_sh"),
        assert_blockwise_close(gw.cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), what="grad_w"),
    ]
    return worst


@pytest.mark.parametrize("flags", [0, e3j.E3J_PLAN_GENERIC_ONLY])
@pytest.mark.parametrize("config,n_atoms", [(1, None), (2, 192), (3, 300), (5, 3000)])
def test_conv_small(config, n_atoms, flags):
    worst = run_conv_parity(*make_case(config, n_atoms, flags=flags))
    assert max(worst) < 1e-5


@pytest.mark.parametrize("config", [2, 3])
def test_conv_full_size(config):
    """Configs 2 and 3 at their full size, every element."""
    worst = run_conv_parity(*make_case(config))
    assert max(worst) < 1e-5


def test_conv_natural_parity_outputs():
    worst = run_conv_parity(*make_case(2, 192, irreps_out=workloads.NATURAL_PARITY_OUT))
    assert max(worst) < 1e-5


def test_scalar_input_signature():
    """First-layer signature: scalar node features only (128x0e), every output up to l = 3."""
    import dataclasses
    wl = dataclasses.replace(workloads.make_graph(2, 300), irreps_in="128x0e")
    plan = e3j.e3j_plan_create("128x0e", 3, None, 3)
    assert plan.specialised and plan.n_paths == 4 and plan.d_out == 16
    cp = oconv.Coupling("128x0e", 3, None, 3)
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    worst = run_conv_parity(wl, plan, cp, x, y, w, g)
    assert max(worst) < 1e-5


def test_lmax2_signature():
    """The water-box inputs with harmonics and outputs up to l = 2 (9 harmonics per edge: rows of the harmonics
    array are 36 bytes, only 4-byte aligned), forward, backward and standalone tensor product."""
    import dataclasses
    wl = dataclasses.replace(workloads.make_graph(2, 300), sh_lmax=2, out_lmax=2)
    plan = e3j.e3j_plan_create("128x0e+128x1o", 2, None, 2)
    assert plan.specialised and plan.n_paths == 9 and plan.d_out == 29 and plan.d_sh == 9
    cp = oconv.Coupling("128x0e+128x1o", 2, None, 2)
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    assert y.shape[1] == 9
    worst = run_conv_parity(wl, plan, cp, x, y, w, g)
    assert max(worst) < 1e-5
    rows = 333
    out = e3j.e3j_tp_fwd(plan, _cuda(x[:rows]), _cuda(y[:rows]), _cuda(w[:rows]))
    gx1, gx2, gw = e3j.e3j_tp_bwd(plan, _cuda(x[:rows]), _cuda(y[:rows]), _cuda(w[:rows]), _cuda(g[:rows]))
    ident = np.arange(rows, dtype=np.int32)
    ref = oconv.conv_fwd(cp, x[:rows], y[:rows], w[:rows], ident, ident)
    rx, ry, rw = oconv.conv_bwd(cp, x[:rows], y[:rows], w[:rows], ident, ident, g[:rows])
    assert_blockwise_close(out.cpu().numpy(), ref, blocks_of_paths(cp.paths, "out"), what="tp out")
    assert_blockwise_close(gx1.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="tp grad_x1")
    assert_blockwise_close(gx2.cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), what="tp grad_x2")
    assert_blockwise_close(gw.cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), what="tp grad_w")


@pytest.mark.parametrize("irreps,lmax", [("96x0e+96x1o", 3), ("128x0e+128x1o+128x2e+128x3o", 2),
                                         ("64x0e+64x1o+64x2e", 3), ("32x0e+32x1o", 3)])
def test_signatures_generated_with_automatic_tile_parameters(irreps, lmax):
    """Signatures that were not tuned by hand: the generator chose their tiles (96 channels: one channel per lane
    and three warps per row group; four input irreps with harmonics up to l = 2: 18 paths, 64 rows; three input
    irreps at 64 channels: 24 paths; 32 channels: one warp covers an edge with one channel per lane)."""
    import dataclasses
    wl = dataclasses.replace(workloads.make_graph(2, 300), irreps_in=irreps, sh_lmax=lmax, out_lmax=lmax)
    plan = e3j.e3j_plan_create(irreps, lmax, None, lmax)
    assert plan.specialised
    cp = oconv.Coupling(irreps, lmax, None, lmax)
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    worst = run_conv_parity(wl, plan, cp, x, y, w, g)
    assert max(worst) < 1e-5
    assert e3j.e3j_plan_device_status(plan) == 0


@pytest.mark.parametrize("channels", [64, 256])
def test_other_channel_counts_of_the_water_box_signature(channels):
    """The water-box signature with 64 and 256 channels (generated kernels exist for both)."""
    import dataclasses
    irreps = f"{channels}x0e+{channels}x1o"
    wl = dataclasses.replace(workloads.make_graph(2, 240), irreps_in=irreps)
    plan = e3j.e3j_plan_create(irreps, 3, None, 3)
    assert plan.specialised and plan.n_channels == channels
    cp = oconv.Coupling(irreps, 3, None, 3)
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    worst = run_conv_parity(wl, plan, cp, x, y, w, g)
    assert max(worst) < 1e-5


def test_conv_without_prepared_graph():
    worst = run_conv_parity(*make_case(1), prepared=False)
    assert max(worst) < 1e-5


@pytest.mark.parametrize("flags", [0, e3j.E3J_PLAN_GENERIC_ONLY])
def test_isolated_nodes_ragged_rows_and_duplicates(flags):
    """Receivers without edges get zero rows; silent senders zero gradients; duplicate edges
    and self-loops are ordinary edges; one very long row."""
    rng = np.random.default_rng(42)
    c = workloads.CONFIGS[2]
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, 3, flags)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, 3)
    n = 41
    deg = rng.integers(0, 9, size=n)
    deg[[0, 7, 8, 40]] = 0
    deg[20] = 700  # a hub
    rcv = np.repeat(np.arange(n), deg).astype(np.int32)
    snd = rng.integers(0, n - 3, size=len(rcv)).astype(np.int32)  # last nodes never send
    snd[:5] = rcv[:5]  # self loops
    snd[10:14] = snd[10]  # duplicates
    e = len(rcv)
    wl = workloads.Workload(config=2, name="edge", irreps_in=c["irreps_in"], sh_lmax=3, irreps_out=None,
                            out_lmax=3, n_nodes=n, n_edges=e, senders=snd, receivers=rcv)
    x = rng.standard_normal((n, plan.d_in, plan.n_channels)).astype(np.float32)
    y = rng.standard_normal((e, plan.d_sh)).astype(np.float32)
    w = rng.standard_normal((e, plan.n_paths, plan.n_channels)).astype(np.float32)
    g = rng.standard_normal((n, plan.d_out, plan.n_channels)).astype(np.float32)
    worst = run_conv_parity(wl, plan, cp, x, y, w, g)
    assert max(worst) < 1e-5
    out = e3j.e3j_conv_fwd(plan, _cuda(x), _cuda(y), _cuda(w), _cuda(snd), _cuda(rcv))
    assert torch.count_nonzero(out[[0, 7, 8, 40]]) == 0


@pytest.mark.parametrize("degrees", [[1], [7, 8, 1, 14, 15, 6, 32, 33, 64, 2], [63, 65]])
def test_backward_tiles_are_cut_at_receiver_changes(degrees):
    """Rows as long as a tile of the edge-wise backward, one edge shorter and longer, rows of one edge (a new
    receiver block every tile) and rows longer than a look-ahead window, with enough edges that every CTA walks
    through several windows."""
    rng = np.random.default_rng(7)
    c = workloads.CONFIGS[2]
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, 3)
    assert plan.specialised
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, 3)
    n = 148 * 90 // max(1, int(np.mean(degrees))) + 11
    deg = np.resize(np.asarray(degrees), n)
    rcv = np.repeat(np.arange(n), deg).astype(np.int32)
    snd = rng.integers(0, n, size=len(rcv)).astype(np.int32)
    e = len(rcv)
    wl = workloads.Workload(config=2, name="cuts", irreps_in=c["irreps_in"], sh_lmax=3, irreps_out=None,
                            out_lmax=3, n_nodes=n, n_edges=e, senders=snd, receivers=rcv)
    x = rng.standard_normal((n, plan.d_in, plan.n_channels)).astype(np.float32)
    y = rng.standard_normal((e, plan.d_sh)).astype(np.float32)
    w = rng.standard_normal((e, plan.n_paths, plan.n_channels)).astype(np.float32)
    g = rng.standard_normal((n, plan.d_out, plan.n_channels)).astype(np.float32)
    worst = run_conv_parity(wl, plan, cp, x, y, w, g)
    assert max(worst) < 1e-5


@pytest.mark.parametrize("flags", [0, e3j.E3J_PLAN_GENERIC_ONLY])
def test_empty_graph(flags):
    plan = e3j.e3j_plan_create("128x0e+128x1o", 3, None, 3, flags)
    n = 5
    x = torch.randn((n, plan.d_in, plan.n_channels), device=DEV)
    empty_i = torch.zeros(0, dtype=torch.int32, device=DEV)
    out = torch.full((n, plan.d_out, plan.n_channels), 7.0, device=DEV)
    e3j.e3j_conv_fwd(plan, x, torch.zeros((0, plan.d_sh), device=DEV),
                     torch.zeros((0, plan.n_paths, plan.n_channels), device=DEV), empty_i, empty_i, out=out)
    assert torch.count_nonzero(out) == 0
    gx, gy, gw = e3j.e3j_conv_bwd(plan, x, torch.zeros((0, plan.d_sh), device=DEV),
                                  torch.zeros((0, plan.n_paths, plan.n_channels), device=DEV), empty_i,
                                  empty_i, torch.randn_like(out))
    assert torch.count_nonzero(gx) == 0 and gy.numel() == 0 and gw.numel() == 0


@pytest.mark.parametrize("flags", [0, e3j.E3J_PLAN_GENERIC_ONLY])
@pytest.mark.parametrize("rows", [1, 333])
def test_tensor_product(rows, flags):
    c = workloads.CONFIGS[4]
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, 3, flags)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, 3)
    x1, x2, w, g = workloads.make_tp_rows(rows, plan.n_paths, plan.d_out)
    d = [_cuda(a) for a in (x1, x2, w, g)]
    out = e3j.e3j_tp_fwd(plan, d[0], d[1], d[2])
    g1, g2, gw = e3j.e3j_tp_bwd(plan, d[0], d[1], d[2], d[3])
    out_b = e3j.e3j_tp_fwd(plan, d[0], d[1], d[2])
    g1b, g2b, gwb = e3j.e3j_tp_bwd(plan, d[0], d[1], d[2], d[3])
    for a, b in ((out, out_b), (g1, g1b), (g2, g2b), (gw, gwb)):
        assert torch.equal(a, b)
    ref = oconv.tp_fwd(cp, x1, x2, w)
    r1, r2, rw = oconv.tp_bwd(cp, x1, x2, w, g)
    assert_blockwise_close(out.cpu().numpy(), ref, blocks_of_paths(cp.paths, "out"), what="tp out")
    assert_blockwise_close(g1.cpu().numpy(), r1, blocks_of_paths(cp.paths, "x"), what="tp grad_x1")
    assert_blockwise_close(g2.cpu().numpy(), r2, blocks_of_paths(cp.paths, "sh"), what="tp grad_x2")
    assert_blockwise_close(gw.cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), what="tp grad_w")
    # partial requests: the same numbers for what is asked for
    p1 = e3j.e3j_tp_bwd(plan, d[0], d[1], d[2], d[3], grad_x2=False, grad_w=False)
    p2 = e3j.e3j_tp_bwd(plan, d[0], d[1], d[2], d[3], grad_x1=False)
    torch.cuda.synchronize()
    assert p1[1] is None and p1[2] is None and p2[0] is None
    assert_blockwise_close(p1[0].cpu().numpy(), r1, blocks_of_paths(cp.paths, "x"), what="tp grad_x1 alone")
    assert_blockwise_close(p2[1].cpu().numpy(), r2, blocks_of_paths(cp.paths, "sh"), what="tp grad_x2 without grad_x1")
    assert_blockwise_close(p2[2].cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), what="tp grad_w without grad_x1")


@pytest.mark.parametrize("flags", [0, e3j.E3J_PLAN_GENERIC_ONLY])
@pytest.mark.parametrize("config,n_atoms,pad", [(1, None, 37), (2, 192, 1500), (2, 192, 0)])
def test_padded_edge_lists(config, n_atoms, pad, flags):
    """Padded calls: the real edges give bit for bit what the plain call gives on the unpadded list, whatever
    the padding entries hold (NaN weights, wild sender ids); padding rows of grad_sh / grad_w are zero; the
    number of real edges is never passed from the host."""
    wl, plan, cp, x, y, w, g = make_case(config, n_atoms, flags=flags)
    n, e = wl.n_nodes, wl.n_edges
    rng = np.random.default_rng(5)
    yp = np.concatenate([y, np.full((pad, y.shape[1]), np.nan, np.float32)])
    wp = np.concatenate([w, np.full((pad,) + w.shape[1:], np.nan, np.float32)])
    sndp = np.concatenate([wl.senders, rng.integers(-2 ** 30, 2 ** 30, pad).astype(np.int32)])
    rcvp = np.concatenate([wl.receivers, np.sort(rng.integers(n, 2 ** 30, pad)).astype(np.int32)])
    dx, dg = _cuda(x), _cuda(g)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    out = e3j.e3j_conv_fwd(plan, dx, _cuda(y), _cuda(w), snd, rcv, rowptr)
    gx, gy, gw = e3j.e3j_conv_bwd(plan, dx, _cuda(y), _cuda(w), snd, rcv, dg, rowptr, perm, colptr)
    psnd, prcv, py, pw = _cuda(sndp), _cuda(rcvp), _cuda(yp), _cuda(wp)
    prow, pperm, pcol = e3j.e3j_graph_prepare_padded(n, psnd, prcv)
    assert int(prow[n]) == e and int(pcol[n]) == e
    assert torch.equal(prow, rowptr) and torch.equal(pcol, colptr) and torch.equal(pperm[:e], perm[:e])
    pout = e3j.e3j_conv_fwd_padded(plan, dx, py, pw, psnd, prcv, prow)
    for prepared in (True, False):
        pgx, pgy, pgw = e3j.e3j_conv_bwd_padded(plan, dx, py, pw, psnd, prcv, dg, prow,
                                                pperm if prepared else None, pcol if prepared else None)
        torch.cuda.synchronize()
        assert torch.equal(pout, out) and torch.equal(pgx, gx)
        assert torch.equal(pgy[:e], gy) and torch.equal(pgw[:e], gw)
        assert torch.count_nonzero(pgy[e:]) == 0 and torch.count_nonzero(pgw[e:]) == 0
    ref = oconv.conv_fwd_padded(cp, x, yp, wp, sndp, rcvp)
    assert_blockwise_close(pout.cpu().numpy(), ref, blocks_of_paths(cp.paths, "out"), what="out")
    with pytest.raises(e3j.E3JError):
        e3j.e3j_conv_fwd_padded(plan, dx, py, pw, psnd, prcv, None)


@pytest.mark.parametrize("flags", [0, e3j.E3J_PLAN_GENERIC_ONLY])
def test_padded_list_without_real_edges(flags):
    wl, plan, cp, x, y, w, g = make_case(2, 192, flags=flags)
    n, pad = wl.n_nodes, 64
    rng = np.random.default_rng(6)
    py = _cuda(np.full((pad, y.shape[1]), np.nan, np.float32))
    pw = _cuda(np.full((pad,) + w.shape[1:], np.nan, np.float32))
    psnd = _cuda(rng.integers(0, n, pad).astype(np.int32))
    prcv = _cuda(np.full(pad, n, np.int32))
    prow, pperm, pcol = e3j.e3j_graph_prepare_padded(n, psnd, prcv)
    out = torch.full((n, plan.d_out, plan.n_channels), 7.0, device=DEV)
    e3j.e3j_conv_fwd_padded(plan, _cuda(x), py, pw, psnd, prcv, prow, out=out)
    gx, gy, gw = e3j.e3j_conv_bwd_padded(plan, _cuda(x), py, pw, psnd, prcv, _cuda(g), prow, pperm, pcol)
    torch.cuda.synchronize()
    for t in (out, gx, gy, gw):
        assert torch.count_nonzero(t) == 0


def test_one_plan_on_two_streams():
    """A plan is immutable: calls on two streams with their own workspaces may overlap and give the same bits
    as the serial calls; no bounded wait ran out (device status word stays 0)."""
    wl, plan, cp, x, y, w, g = make_case(2, 600)
    n = wl.n_nodes
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    ins = []
    for k in range(2):
        rng = np.random.default_rng(100 + k)
        ins.append((_cuda(x * (k + 1)), _cuda(y), _cuda(w + k), _cuda(g - k)))
    serial = []
    for dx, dy, dw, dg in ins:
        out = e3j.e3j_conv_fwd(plan, dx, dy, dw, snd, rcv, rowptr)
        serial.append((out,) + e3j.e3j_conv_bwd(plan, dx, dy, dw, snd, rcv, dg, rowptr, perm, colptr))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    res = [None, None]
    for rep in range(5):
        for k, (dx, dy, dw, dg) in enumerate(ins):
            with torch.cuda.stream(streams[k]):
                out = e3j.e3j_conv_fwd(plan, dx, dy, dw, snd, rcv, rowptr, stream=streams[k])
                res[k] = (out,) + e3j.e3j_conv_bwd(plan, dx, dy, dw, snd, rcv, dg, rowptr, perm, colptr,
                                                   stream=streams[k])
    torch.cuda.synchronize()
    for k in range(2):
        for a, b in zip(res[k], serial[k]):
            assert torch.equal(a, b)
    assert e3j.e3j_plan_device_status(plan) == 0


def test_channel_counts_must_be_multiples_of_four():
    plan = e3j.e3j_plan_create("6x0e+6x1o", 1)
    x = torch.zeros((2, plan.d_in, 6), device=DEV)
    sh = torch.zeros((1, plan.d_sh), device=DEV)
    w = torch.zeros((1, plan.n_paths, 6), device=DEV)
    idx = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(e3j.E3JError) as err:
        e3j.e3j_conv_fwd(plan, x, sh, w, idx, idx)
    assert err.value.status == e3j.E3J_ERR_UNSUPPORTED


@pytest.mark.parametrize("config,n_atoms", [(1, None), (2, 192), (3, 200)])
def test_collapsed_output_multiplicities(config, n_atoms):
    """Plans with E3J_PLAN_COLLAPSE_OUTPUTS: paths landing on one (L, parity) share an output block."""
    c = workloads.CONFIGS[config]
    wl = workloads.make_graph(config, n_atoms)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"],
                               e3j.E3J_PLAN_COLLAPSE_OUTPUTS)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    R, offs = oconv.collapse_matrix(cp)
    assert plan.d_out == R.shape[0] < cp.D
    x, y, w, _ = workloads.make_features(wl, plan.n_paths, plan.d_out)
    g = np.random.default_rng(9).standard_normal((wl.n_nodes, plan.d_out, plan.n_channels)).astype(np.float32)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(wl.n_nodes, snd, rcv)
    out = e3j.e3j_conv_fwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv, rowptr)
    gx, gy, gw = e3j.e3j_conv_bwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv, _cuda(g), rowptr, perm, colptr)
    torch.cuda.synchronize()
    ref = oconv.conv_fwd_collapsed(cp, x, y, w, wl.senders, wl.receivers)
    rx, ry, rw = oconv.conv_bwd_collapsed(cp, x, y, w, wl.senders, wl.receivers, g)
    blocks = sorted({(off, off + 2 * p.L + 1) for p, off in zip(cp.paths, offs)})
    assert_blockwise_close(out.cpu().numpy(), ref, blocks, what="out")
    assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), what="grad_x")
    assert_blockwise_close(gy.cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), what="grad_sh")
    assert_blockwise_close(gw.cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), what="grad_w")


@pytest.mark.parametrize("flags", [0, e3j.E3J_PLAN_GENERIC_ONLY])
@pytest.mark.parametrize("config,n_atoms,natural", [(1, None, False), (2, 192, False), (2, 1200, False),
                                                    (2, 192, True), (3, 200, False)])
def test_double_backward(config, n_atoms, natural, flags):
    """Cotangents of the backward's inputs against the oracle; a missing cotangent is zero; outputs that are
    not wanted are skipped; two runs give the same bits.  (Configs 2 and 3 have fused kernels, config 1 and the
    generic plans take the composition.)"""
    _check_double_backward(*make_case(config, n_atoms, flags=flags,
                                      **({"irreps_out": workloads.NATURAL_PARITY_OUT} if natural else {})))


@pytest.mark.parametrize("irreps,lmax,n_atoms,fused", [
    ("128x0e+128x1o", 2, 300, True),             # l <= 2
    ("256x0e+256x1o", 3, 192, True),             # 256 channels: two warps per edge
    ("64x0e+64x1o", 3, 300, True),
    ("128x0e", 3, 300, True),                    # scalar inputs
    ("128x0e+128x1o+128x2e", 3, 192, False),     # the tensor-product signature as a graph call: composition
])
def test_double_backward_of_the_other_generated_signatures(irreps, lmax, n_atoms, fused):
    """Every generated signature except the collapsed one and the 24-path tensor-product one (whose fused sweeps
    were measured slower than the composition: 30 KB of staging per edge leaves one edge per tile) has the fused
    double-backward kernels."""
    import dataclasses
    wl = dataclasses.replace(workloads.make_graph(2, n_atoms), irreps_in=irreps, sh_lmax=lmax, out_lmax=lmax)
    plan = e3j.e3j_plan_create(irreps, lmax, None, lmax)
    assert plan.specialised
    cp = oconv.Coupling(irreps, lmax, None, lmax)
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    before = e3j.e3j_launch_count()
    _check_double_backward(wl, plan, cp, x, y, w, g, partial=False)
    # two calls, each the two fused sweeps with their follow-up kernels (4 launches), plus graph preparation
    assert (e3j.e3j_launch_count() - before <= 20) == fused   # the composition takes more than forty launches


def _check_double_backward(wl, plan, cp, x, y, w, g, partial=True):
    n, e = wl.n_nodes, wl.n_edges
    rng = np.random.default_rng(77)
    ux = rng.standard_normal(x.shape).astype(np.float32)
    uy = rng.standard_normal(y.shape).astype(np.float32)
    uw = rng.standard_normal(w.shape).astype(np.float32)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    dev = [_cuda(a) for a in (x, y, w)]
    run = lambda cx, cy, cw, **kw: e3j.e3j_conv_bwd_bwd(plan, dev[0], dev[1], dev[2], snd, rcv, _cuda(g), rowptr, perm,
                                                        colptr, cx, cy, cw, **kw)
    got = run(_cuda(ux), _cuda(uy), _cuda(uw))
    again = run(_cuda(ux), _cuda(uy), _cuda(uw))
    torch.cuda.synchronize()
    for a, b in zip(got, again):
        assert torch.equal(a, b)
    ref = oconv.conv_bwd_bwd(cp, x, y, w, wl.senders, wl.receivers, g, ux, uy, uw)
    kinds = ("out", "x", "sh", "w")
    for a, r, kind in zip(got, ref, kinds):
        assert_blockwise_close(a.cpu().numpy(), r, blocks_of_paths(cp.paths, kind), what="double backward " + kind)
    if not partial:
        return
    # only the harmonics' cotangent given, only two outputs wanted
    gg, gx, gsh, gw = run(None, _cuda(uy), None, g_sh=False, g_w=None)
    assert gsh is None and gw is None
    zero_x, zero_w = np.zeros_like(x), np.zeros_like(w)
    ref1 = oconv.conv_bwd_bwd(cp, x, y, w, wl.senders, wl.receivers, g, zero_x, uy, zero_w)
    assert_blockwise_close(gg.cpu().numpy(), ref1[0], blocks_of_paths(cp.paths, "out"), what="gg_out (ct_sh only)")
    assert_blockwise_close(gx.cpu().numpy(), ref1[1], blocks_of_paths(cp.paths, "x"), what="g_x (ct_sh only)")
    # no cotangent at all: zeros
    for t in run(None, None, None):
        assert torch.count_nonzero(t) == 0


def test_a_bounded_wait_that_runs_out_is_reported():
    """Every wait in the specialised kernels gives up after a fixed number of polls.  The self-test makes one run
    out on purpose (a barrier that nothing completes, 1000 polls): the wait returns, the kernel ends, the plan's
    status word reads 1 once, and the plan keeps working."""
    wl, plan, cp, x, y, w, g = make_case(2, 192)
    assert e3j.e3j_plan_device_status(plan) == 0
    returned, abort_flag = e3j.e3j_selftest_bounded_wait(plan, 1000)
    assert (returned, abort_flag) == (0, 1)
    assert e3j.e3j_plan_device_status(plan) == 1
    assert e3j.e3j_plan_device_status(plan) == 0      # reading clears it
    run_conv_parity(wl, plan, cp, x, y, w, g)         # the context and the plan are still usable
    assert e3j.e3j_plan_device_status(plan) == 0


def test_optional_gradients_can_be_skipped():
    wl, plan, cp, x, y, w, g = make_case(1)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    full = e3j.e3j_conv_bwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv, _cuda(g))
    only_x = e3j.e3j_conv_bwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv, _cuda(g), grad_sh=False, grad_w=False)
    only_w = e3j.e3j_conv_bwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv, _cuda(g), grad_x=False, grad_sh=False)
    assert only_x[1] is None and only_x[2] is None and torch.equal(only_x[0], full[0])
    assert only_w[0] is None and torch.equal(only_w[2], full[2])


def test_graph_prepare_matches_numpy():
    for config, n_atoms in [(1, None), (2, 192), (5, 3000)]:
        wl = workloads.make_graph(config, n_atoms)
        rowptr, perm, colptr = e3j.e3j_graph_prepare(wl.n_nodes, _cuda(wl.senders), _cuda(wl.receivers))
        n = wl.n_nodes
        assert np.array_equal(rowptr.cpu().numpy(), np.searchsorted(wl.receivers, np.arange(n + 1), side="left"))
        assert np.array_equal(perm.cpu().numpy(), np.argsort(wl.senders, kind="stable"))
        assert np.array_equal(colptr.cpu().numpy(),
                              np.concatenate([[0], np.cumsum(np.bincount(wl.senders, minlength=n))]))
    # a hub sender exercises the long-bucket sort
    rng = np.random.default_rng(3)
    n, e = 50, 5000
    rcv = np.sort(rng.integers(0, n, e)).astype(np.int32)
    snd = np.where(rng.random(e) < 0.5, 7, rng.integers(0, n, e)).astype(np.int32)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, _cuda(snd), _cuda(rcv))
    assert np.array_equal(perm.cpu().numpy(), np.argsort(snd, kind="stable"))


def test_graph_validate_reports_bad_graphs():
    good_s = torch.tensor([0, 1, 2], dtype=torch.int32, device=DEV)
    good_r = torch.tensor([0, 0, 2], dtype=torch.int32, device=DEV)
    assert e3j.e3j_graph_validate(3, good_s, good_r) == 0
    assert e3j.e3j_graph_validate(3, good_s, torch.tensor([1, 0, 2], dtype=torch.int32, device=DEV)) == -7
    assert e3j.e3j_graph_validate(2, good_s, good_r) == -7


def test_workspace_errors_are_reported():
    wl, plan, cp, x, y, w, g = make_case(1)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    tiny = torch.empty(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(ValueError):
        e3j.e3j_conv_bwd(plan, _cuda(x), _cuda(y), _cuda(w), snd, rcv, _cuda(g), workspace=tiny)


@pytest.mark.parametrize("seed", [1, 2])
def test_specialised_and_generic_kernels_agree_on_random_graphs(seed):
    """A cross-check beside the oracle parity tests: on random graphs (sparse rows, rows of tens of edges, hubs of
    up to 2000 edges, padded lists) and for every generated signature the specialised kernels and the
    table-driven ones give the same forward, backward, double backward and tensor products to rounding, the
    specialised backward twice the same bits."""
    rng = np.random.default_rng(seed)
    sigs = [("128x0e+128x1o", 3, None, 3), ("64x0e+64x1o", 3, None, 3), ("256x0e+256x1o", 3, None, 3),
            ("128x0e", 3, None, 3), ("64x0e+64x1o+64x2e+64x3o", 3, None, 3),
            ("128x0e+128x1o", 3, workloads.NATURAL_PARITY_OUT, -1), ("128x0e+128x1o", 2, None, 2),
            ("128x0e+128x1o+128x2e", 3, None, 3)]

    def rel(a, b):
        return (a - b).abs().max().item() / max(b.abs().max().item(), 1e-30)

    for it in range(16):
        irr, lmax, iro, olm = sigs[it % len(sigs)]
        pf = e3j.e3j_plan_create(irr, lmax, iro, olm)
        pg = e3j.e3j_plan_create(irr, lmax, iro, olm, e3j.E3J_PLAN_GENERIC_ONLY)
        assert pf.specialised and not pg.specialised
        n = int(rng.integers(2, 300))
        deg = [rng.integers(0, 12, size=n), rng.integers(0, 3, size=n), rng.integers(20, 90, size=n),
               rng.integers(0, 5, size=n)][it % 4]
        if it % 4 == 3:
            deg[rng.integers(0, n)] = int(rng.integers(100, 2000))
        rcv = np.repeat(np.arange(n), deg).astype(np.int32)
        e, pad = len(rcv), int(rng.integers(0, 150)) if it % 2 else 0
        snd = rng.integers(0, n, size=e).astype(np.int32)
        if e + pad == 0:
            continue
        s = _cuda(np.concatenate([snd, np.zeros(pad, np.int32)]))
        r = _cuda(np.concatenate([rcv, np.full(pad, n, np.int32)]))
        x = torch.randn((n, pf.d_in, pf.n_channels), device=DEV)
        y = torch.randn((e + pad, pf.d_sh), device=DEV)
        w = torch.randn((e + pad, pf.n_paths, pf.n_channels), device=DEV)
        g = torch.randn((n, pf.d_out, pf.n_channels), device=DEV)
        if pad:
            rowptr, perm, colptr = e3j.e3j_graph_prepare_padded(n, s, r)
            fwd, bwd = e3j.e3j_conv_fwd_padded, e3j.e3j_conv_bwd_padded
        else:
            rowptr, perm, colptr = e3j.e3j_graph_prepare(n, s, r)
            fwd, bwd = e3j.e3j_conv_fwd, e3j.e3j_conv_bwd
        errs = [rel(fwd(pf, x, y, w, s, r, rowptr), fwd(pg, x, y, w, s, r, rowptr))]
        bf, bg = bwd(pf, x, y, w, s, r, g, rowptr, perm, colptr), bwd(pg, x, y, w, s, r, g, rowptr, perm, colptr)
        again = bwd(pf, x, y, w, s, r, g, rowptr, perm, colptr)
        assert all(torch.equal(a, b) for a, b in zip(bf, again))
        errs += [rel(a, b) for a, b in zip(bf, bg)]
        if not pad and e:
            cts = [torch.randn_like(t) for t in (x, y, w)]
            errs += [rel(a, b) for a, b in zip(
                e3j.e3j_conv_bwd_bwd(pf, x, y, w, s, r, g, rowptr, perm, colptr, *cts),
                e3j.e3j_conv_bwd_bwd(pg, x, y, w, s, r, g, rowptr, perm, colptr, *cts))]
        rows = int(rng.integers(1, 500))
        x1, x2 = torch.randn((rows, pf.d_in, pf.n_channels), device=DEV), torch.randn((rows, pf.d_sh), device=DEV)
        wt = torch.randn((rows, pf.n_paths, pf.n_channels), device=DEV)
        gt = torch.randn((rows, pf.d_out, pf.n_channels), device=DEV)
        errs.append(rel(e3j.e3j_tp_fwd(pf, x1, x2, wt), e3j.e3j_tp_fwd(pg, x1, x2, wt)))
        errs += [rel(a, b) for a, b in zip(e3j.e3j_tp_bwd(pf, x1, x2, wt, gt), e3j.e3j_tp_bwd(pg, x1, x2, wt, gt))]
        torch.cuda.synchronize()
        assert e3j.e3j_plan_device_status(pf) == 0
        assert max(errs) < 1e-5, (it, irr, n, e, pad, errs)


def test_calls_can_be_captured_in_a_cuda_graph():
    """With a prepared graph and caller-owned outputs and workspaces the calls only enqueue kernels: a stream
    capture of forward + backward + double backward replays to the same bits as the eager calls."""
    wl, plan, cp, x, y, w, g = make_case(2, 192)
    n, e = wl.n_nodes, wl.n_edges
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    dx, dy, dw, dg = _cuda(x), _cuda(y), _cuda(w), _cuda(g)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    u8 = lambda nbytes: torch.empty(max(nbytes, 256), dtype=torch.uint8, device=DEV)
    ws_f, ws_b = u8(e3j.e3j_conv_fwd_workspace_bytes(plan, n, e)), u8(e3j.e3j_conv_bwd_workspace_bytes(plan, n, e))
    ws_d = u8(e3j.e3j_conv_bwd_bwd_workspace_bytes(plan, n, e))
    out, gx, gy, gw = torch.empty_like(dg), torch.empty_like(dx), torch.empty_like(dy), torch.empty_like(dw)
    dd = [torch.empty_like(t) for t in (dg, dx, dy, dw)]

    def step():
        e3j.e3j_conv_fwd(plan, dx, dy, dw, snd, rcv, rowptr, out=out, workspace=ws_f)
        e3j.e3j_conv_bwd(plan, dx, dy, dw, snd, rcv, dg, rowptr, perm, colptr, grad_x=gx, grad_sh=gy, grad_w=gw,
                         workspace=ws_b)
        e3j.e3j_conv_bwd_bwd(plan, dx, dy, dw, snd, rcv, dg, rowptr, perm, colptr, gx, gy, gw, gg_out=dd[0],
                             g_x=dd[1], g_sh=dd[2], g_w=dd[3], workspace=ws_d)

    step()   # eager: first use sets the kernels' attributes and uploads the plan's tables
    torch.cuda.synchronize()
    eager = [t.clone() for t in (out, gx, gy, gw, *dd)]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in (out, gx, gy, gw, *dd):
        t.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(eager, (out, gx, gy, gw, *dd)):
        assert torch.equal(a, b)
    assert e3j.e3j_plan_device_status(plan) == 0


@pytest.mark.parametrize("flags", [0, e3j.E3J_PLAN_GENERIC_ONLY])
def test_misaligned_channel_arrays_are_refused(flags):
    """Rows are moved as 128-bit vectors and 16-byte bulk copies: a per-channel array that starts 4 bytes off a
    16-byte boundary must be refused on the host (no launch), whichever argument it is."""
    wl, plan, cp, x, y, w, g = make_case(2, 192, flags=flags)
    n, e = wl.n_nodes, wl.n_edges
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)

    def shifted(a):   # same values, storage offset by one float
        buf = torch.empty(a.size + 1, dtype=torch.float32, device=DEV)
        view = buf[1:].view(a.shape)
        view.copy_(torch.from_numpy(a))
        assert view.data_ptr() % 16 == 4
        return view

    good = dict(x=_cuda(x), sh=_cuda(y), w=_cuda(w), g=_cuda(g))
    for bad in ("x", "w"):
        args = dict(good)
        args[bad] = shifted({"x": x, "w": w}[bad])
        with pytest.raises(e3j.E3JError, match="status -1"):
            e3j.e3j_conv_fwd(plan, args["x"], args["sh"], args["w"], snd, rcv)
    for bad in ("x", "w", "g"):
        args = dict(good)
        args[bad] = shifted({"x": x, "w": w, "g": g}[bad])
        with pytest.raises(e3j.E3JError, match="status -1"):
            e3j.e3j_conv_bwd(plan, args["x"], args["sh"], args["w"], snd, rcv, args["g"])
    with pytest.raises(e3j.E3JError, match="status -1"):
        e3j.e3j_conv_fwd(plan, good["x"], good["sh"], good["w"], snd, rcv, out=shifted(g))
    # the harmonics may sit anywhere a float can
    out = e3j.e3j_conv_fwd(plan, good["x"], shifted(y), good["w"], snd, rcv)
    ref = e3j.e3j_conv_fwd(plan, good["x"], good["sh"], good["w"], snd, rcv)
    assert torch.equal(out, ref)
    gx, gy, gw = e3j.e3j_conv_bwd(plan, good["x"], shifted(y), good["w"], snd, rcv, good["g"])
    rx, ry, rw = e3j.e3j_conv_bwd(plan, good["x"], good["sh"], good["w"], snd, rcv, good["g"])
    assert torch.equal(gx, rx) and torch.equal(gy, ry) and torch.equal(gw, rw)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0


# ------------------------------------------------------------------ full-size configurations, sampled
def _seeded_normal(shape, seed):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(seed)
    return torch.randn(shape, generator=gen, device=DEV, dtype=torch.float32)


def _checksum(t):
    """Order-independent exact fingerprint of a float tensor (wrapping integer sum of its bit patterns)."""
    return int(t.view(torch.int32).to(torch.int64).sum().item())


def test_config5_full_size_sampled():
    """100k atoms, 4.77 M edges, skewed degrees (26..106): the bench launch configuration at scale.
    Outputs are checked on sampled receivers / edges / senders that the oracle recomputes one by one."""
    c = workloads.CONFIGS[5]
    wl = workloads.make_graph(5)
    n, e = wl.n_nodes, wl.n_edges
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    assert plan.specialised == 1
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    rng = np.random.Generator(np.random.PCG64([5, 1]))
    x = rng.standard_normal((n, plan.d_in, plan.n_channels), dtype=np.float32)
    y = workloads.edge_harmonics(wl)
    dx_, dy_ = _cuda(x), _cuda(y)
    dw_ = _seeded_normal((e, plan.n_paths, plan.n_channels), 51)
    dg_ = _seeded_normal((n, plan.d_out, plan.n_channels), 52)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    assert e3j.e3j_graph_validate(n, snd, rcv) == 0
    out = e3j.e3j_conv_fwd(plan, dx_, dy_, dw_, snd, rcv, rowptr)
    gx, gy, gw = e3j.e3j_conv_bwd(plan, dx_, dy_, dw_, snd, rcv, dg_, rowptr, perm, colptr)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    sums = [_checksum(t) for t in (out, gx, gy, gw)]
    out.zero_(); gx.zero_(); gy.zero_()
    e3j.e3j_conv_fwd(plan, dx_, dy_, dw_, snd, rcv, rowptr, out=out)
    e3j.e3j_conv_bwd(plan, dx_, dy_, dw_, snd, rcv, dg_, rowptr, perm, colptr, grad_x=gx, grad_sh=gy, grad_w=gw)
    torch.cuda.synchronize()
    assert sums == [_checksum(t) for t in (out, gx, gy, gw)], "results differ between two runs"

    deg = np.bincount(wl.receivers, minlength=n)
    rp = rowptr.cpu().numpy()
    # every receiver whose edges are cut by a CTA's edge-range boundary of the forward (their rows go through the
    # partial-row scratch and the fix-up kernel): ranges of ceil4(ceil(E / CTAs)) edges, 2 CTAs per SM
    n_cta = 2 * torch.cuda.get_device_properties(0).multi_processor_count
    chunk = (-(-e // n_cta) + 3) // 4 * 4
    cuts = np.arange(chunk, e, chunk)
    straddled = np.unique(wl.receivers[cuts][wl.receivers[cuts] == wl.receivers[cuts - 1]])
    assert len(straddled) > 100
    pick = np.unique(np.concatenate([rng.choice(n, 40, replace=False), np.argsort(deg)[-8:], np.argsort(deg)[:4],
                                     [0, n - 1], straddled]))
    out_blocks, w_blocks = blocks_of_paths(cp.paths, "out"), blocks_of_paths(cp.paths, "w")
    for b in pick:
        e0, e1 = int(rp[b]), int(rp[b + 1])
        s_ids = wl.senders[e0:e1]
        nodes, local = np.unique(np.concatenate([s_ids, [b]]), return_inverse=True)
        lb = int(local[-1])
        order = np.arange(e1 - e0)
        xs = x[nodes]
        ws = dw_[e0:e1].cpu().numpy()
        gs = np.zeros((len(nodes), plan.d_out, plan.n_channels), np.float32)
        gs[lb] = dg_[b].cpu().numpy()
        l_snd = local[:-1].astype(np.int32)
        l_rcv = np.full(e1 - e0, lb, np.int32)
        ref = oconv.conv_fwd(cp, xs, y[e0:e1], ws, l_snd[order], l_rcv)
        assert_blockwise_close(out[b].cpu().numpy()[None], ref[lb][None], out_blocks, what=f"out[{b}]")
        _, ry, rw = oconv.conv_bwd(cp, xs, y[e0:e1], ws, l_snd, l_rcv, gs)
        if e1 > e0:
            assert_blockwise_close(gw[e0:e1].cpu().numpy(), rw, w_blocks, what=f"grad_w[{b}]")
            assert_blockwise_close(gy[e0:e1].cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), what=f"grad_sh[{b}]")
    # grad_x of sampled senders: all edges they send (scattered over the edge list)
    senders_sorted = perm.cpu().numpy()
    cptr = colptr.cpu().numpy()
    for a in rng.choice(n, 24, replace=False):
        ids = np.sort(senders_sorted[cptr[a]:cptr[a + 1]])
        rc = wl.receivers[ids]
        nodes, l_rcv = np.unique(rc, return_inverse=True)
        xs = np.zeros((len(nodes) + 1, plan.d_in, plan.n_channels), np.float32)
        xs[-1] = x[a]
        gs = np.concatenate([dg_[torch.from_numpy(nodes).to(DEV)].cpu().numpy(),
                             np.zeros((1, plan.d_out, plan.n_channels), np.float32)])
        ws = dw_[torch.from_numpy(ids).to(DEV)].cpu().numpy()
        l_snd = np.full(len(ids), len(nodes), np.int32)
        rx, _, _ = oconv.conv_bwd(cp, xs, y[ids], ws, l_snd, l_rcv.astype(np.int32), gs)
        assert_blockwise_close(gx[a].cpu().numpy()[None], rx[-1][None], blocks_of_paths(cp.paths, "x"), what=f"grad_x[{a}]")

    # the scheduled backward at the same size, into the same tensors: per-edge gradients bit-identical to the call
    # checked above, grad_x equal to rounding (its rows are summed in another fixed order)
    sums_plain = [_checksum(t) for t in (gy, gw)]
    gx_plain = gx.clone()
    sched = e3j.e3j_bwd_schedule_build(plan, n, snd, rcv)
    gx.zero_(); gy.zero_()
    e3j.e3j_conv_bwd_scheduled(plan, dx_, dy_, dw_, sched, dg_, grad_x=gx, grad_sh=gy, grad_w=gw)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    assert sums_plain == [_checksum(t) for t in (gy, gw)]
    assert float((gx - gx_plain).abs().max()) <= 2e-6 * float(gx_plain.abs().max())


def _assert_blockwise_close_on_device(got, want, blocks, tol=1e-5, what=""):
    """parity_util.assert_blockwise_close for a CUDA tensor and a float64 oracle array, evaluated on the GPU (the
    host version spends seconds per gigabyte on conversions)."""
    w = torch.from_numpy(np.ascontiguousarray(want)).to(DEV)
    assert tuple(got.shape) == tuple(w.shape), (what, got.shape, w.shape)
    assert bool(torch.isfinite(got).all()), what
    for lo, hi in blocks:
        gb, wb = got[:, lo:hi].double(), w[:, lo:hi]
        if wb.numel() == 0:
            continue
        scale, err = float(wb.abs().max()), float((gb - wb).abs().max())
        assert err <= tol * scale, f"{what} block {lo}:{hi}: err {err:.3e} > {tol} * {scale:.3e}"


def test_config5_full_size_every_element():
    """Config 5 at full size, every output element: the receivers are taken in chunks of 2500, every chunk's edges
    go to the oracle with locally renumbered nodes; out, grad_w and grad_sh are compared chunk by chunk, grad_x is
    accumulated over the chunks in float64 and compared at the end (about a minute of host time)."""
    c = workloads.CONFIGS[5]
    wl = workloads.make_graph(5)
    n, e = wl.n_nodes, wl.n_edges
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    rng = np.random.Generator(np.random.PCG64([5, 2]))
    x = rng.standard_normal((n, plan.d_in, plan.n_channels), dtype=np.float32)
    y = workloads.edge_harmonics(wl)
    dx_, dy_ = _cuda(x), _cuda(y)
    dw_ = _seeded_normal((e, plan.n_paths, plan.n_channels), 61)
    dg_ = _seeded_normal((n, plan.d_out, plan.n_channels), 62)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    rowptr, perm, colptr = e3j.e3j_graph_prepare(n, snd, rcv)
    out = e3j.e3j_conv_fwd(plan, dx_, dy_, dw_, snd, rcv, rowptr)
    gx, gy, gw = e3j.e3j_conv_bwd(plan, dx_, dy_, dw_, snd, rcv, dg_, rowptr, perm, colptr)
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    rp = rowptr.cpu().numpy()
    g_host = dg_.cpu().numpy()
    out_blocks, w_blocks, sh_blocks = (blocks_of_paths(cp.paths, k) for k in ("out", "w", "sh"))
    ref_gx = np.zeros((n, plan.d_in, plan.n_channels))
    step = 2500
    for b0 in range(0, n, step):
        b1 = min(n, b0 + step)
        e0, e1 = int(rp[b0]), int(rp[b1])
        s_ids, r_ids = wl.senders[e0:e1], wl.receivers[e0:e1]
        nodes, local = np.unique(np.concatenate([s_ids, np.arange(b0, b1)]), return_inverse=True)
        l_snd = local[:e1 - e0].astype(np.int32)
        pos = np.searchsorted(nodes, np.arange(b0, b1))            # local ids of the chunk's receivers (ascending)
        l_rcv = pos[r_ids - b0].astype(np.int32)
        # the oracle wants receivers non-decreasing in its own numbering: local ids of b0..b1-1 ascend with b
        xs = x[nodes]
        gs = np.zeros((len(nodes), plan.d_out, plan.n_channels), np.float32)
        gs[pos] = g_host[b0:b1]
        ws = dw_[e0:e1].cpu().numpy()
        ref = oconv.conv_fwd(cp, xs, y[e0:e1], ws, l_snd, l_rcv)
        _assert_blockwise_close_on_device(out[b0:b1], ref[pos], out_blocks, what=f"out[{b0}:{b1}]")
        rx, ry, rw = oconv.conv_bwd(cp, xs, y[e0:e1], ws, l_snd, l_rcv, gs)
        _assert_blockwise_close_on_device(gw[e0:e1], rw, w_blocks, what=f"grad_w[{e0}:{e1}]")
        _assert_blockwise_close_on_device(gy[e0:e1], ry, sh_blocks, what=f"grad_sh[{e0}:{e1}]")
        ref_gx[nodes] += rx
    _assert_blockwise_close_on_device(gx, ref_gx, blocks_of_paths(cp.paths, "x"), what="grad_x")


def test_tensor_product_full_size_sampled():
    """Config 4 at 2^20 rows (75 GB of forward I/O); sampled rows against the oracle."""
    c = workloads.CONFIGS[4]
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, 3)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, 3)
    rows = 1 << 20
    free, _ = torch.cuda.mem_get_info()
    need = 4 * rows * (2 * plan.d_in * plan.n_channels + 2 * plan.d_sh + 2 * plan.n_paths * plan.n_channels
                       + plan.d_out * plan.n_channels)
    if free < need * 1.1:
        pytest.skip("not enough free device memory for 2^20 rows")
    x1 = _seeded_normal((rows, plan.d_in, plan.n_channels), 41)
    x2 = _seeded_normal((rows, plan.d_sh), 42)
    w = _seeded_normal((rows, plan.n_paths, plan.n_channels), 43)
    out = e3j.e3j_tp_fwd(plan, x1, x2, w)
    pick = np.unique(np.concatenate([np.random.default_rng(4).choice(rows, 40, replace=False), [0, rows - 1]]))
    idx = torch.from_numpy(pick).to(DEV)
    h = lambda t: t[idx].cpu().numpy()
    ref = oconv.tp_fwd(cp, h(x1), h(x2), h(w))
    assert_blockwise_close(h(out), ref, blocks_of_paths(cp.paths, "out"), what="tp out")
    # the output buffer doubles as the cotangent of the backward (as a training step would feed it back)
    g1, g2, gw = e3j.e3j_tp_bwd(plan, x1, x2, w, out)
    r1, r2, rw = oconv.tp_bwd(cp, h(x1), h(x2), h(w), h(out))
    assert_blockwise_close(h(g1), r1, blocks_of_paths(cp.paths, "x"), what="tp grad_x1")
    assert_blockwise_close(h(g2), r2, blocks_of_paths(cp.paths, "sh"), what="tp grad_x2")
    assert_blockwise_close(h(gw), rw, blocks_of_paths(cp.paths, "w"), what="tp grad_w")


@pytest.mark.parametrize("config,n_atoms,collapse", [(1, None, False), (2, 192, False), (3, 60, False), (2, 192, True)])
def test_float64_entry_points(config, n_atoms, collapse):
    """e3j_conv_fwd_f64 / e3j_conv_bwd_f64 against the oracle at float64 accuracy (the oracle promotes the same
    float32-representable inputs): 1e-12 of each irreducible block's largest value; two runs give the same bits."""
    flags = e3j.E3J_PLAN_COLLAPSE_OUTPUTS if collapse else 0
    wl, plan, cp, x, y, w, g = make_case(config, n_atoms, flags=flags)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    if collapse:
        R, offs = oconv.collapse_matrix(cp)
        g = g[:, :R.shape[0]].copy()
        ref = oconv.conv_fwd_collapsed(cp, x, y, w, wl.senders, wl.receivers)
        rx, ry, rw = oconv.conv_bwd_collapsed(cp, x, y, w, wl.senders, wl.receivers, g)
        out_blocks = sorted({(off, off + 2 * p.L + 1) for p, off in zip(cp.paths, offs)})
    else:
        ref = oconv.conv_fwd(cp, x, y, w, wl.senders, wl.receivers)
        rx, ry, rw = oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)
        out_blocks = blocks_of_paths(cp.paths, "out")
    d = [_cuda(a.astype(np.float64)) for a in (x, y, w, g)]
    runs = []
    for _ in range(2):
        out = e3j.e3j_conv_fwd_f64(plan, d[0], d[1], d[2], snd, rcv)
        runs.append((out, *e3j.e3j_conv_bwd_f64(plan, d[0], d[1], d[2], snd, rcv, d[3])))
    torch.cuda.synchronize()
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    out, gx, gy, gw = runs[0]
    assert out.dtype == torch.float64
    assert_blockwise_close(out.cpu().numpy(), ref, out_blocks, tol=1e-12, what="f64 out")
    assert_blockwise_close(gx.cpu().numpy(), rx, blocks_of_paths(cp.paths, "x"), tol=1e-12, what="f64 grad_x")
    assert_blockwise_close(gy.cpu().numpy(), ry, blocks_of_paths(cp.paths, "sh"), tol=1e-12, what="f64 grad_sh")
    assert_blockwise_close(gw.cpu().numpy(), rw, blocks_of_paths(cp.paths, "w"), tol=1e-12, what="f64 grad_w")


def test_backward_without_grad_sh_or_grad_x_takes_the_specialised_sweep():
    """Leaving grad_sh and / or grad_x out must not change the gradients that are asked for (same kernel, the store
    or the sender sum skipped): bit-identical to the full call, with the launches of the specialised path."""
    wl, plan, cp, x, y, w, g = make_case(2, 192)
    snd, rcv = _cuda(wl.senders), _cuda(wl.receivers)
    graph = e3j.e3j_graph_prepare(wl.n_nodes, snd, rcv)
    d = [_cuda(a) for a in (x, y, w, g)]
    full = e3j.e3j_conv_bwd(plan, d[0], d[1], d[2], snd, rcv, d[3], *graph)
    l0 = e3j.e3j_launch_count()
    no_sh = e3j.e3j_conv_bwd(plan, d[0], d[1], d[2], snd, rcv, d[3], *graph, grad_sh=False)
    assert e3j.e3j_launch_count() - l0 == 2
    l0 = e3j.e3j_launch_count()
    only_w = e3j.e3j_conv_bwd(plan, d[0], d[1], d[2], snd, rcv, d[3], *graph, grad_sh=False, grad_x=False)
    assert e3j.e3j_launch_count() - l0 == 1
    torch.cuda.synchronize()
    assert no_sh[1] is None and torch.equal(no_sh[0], full[0]) and torch.equal(no_sh[2], full[2])
    assert only_w[0] is None and only_w[1] is None and torch.equal(only_w[2], full[2])
    l0 = e3j.e3j_launch_count()
    no_w = e3j.e3j_conv_bwd(plan, d[0], d[1], d[2], snd, rcv, d[3], *graph, grad_w=False)
    assert e3j.e3j_launch_count() - l0 == 2
    torch.cuda.synchronize()
    assert no_w[2] is None and torch.equal(no_w[0], full[0]) and torch.equal(no_w[1], full[1])
