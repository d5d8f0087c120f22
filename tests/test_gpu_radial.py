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
    (3, 300, 64, 0),
    (5, 3000, 32, 0),
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
