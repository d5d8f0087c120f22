"""Pins for the oracle's convolution / tensor-product loops (CPU only).

Nothing here compares the oracle with itself: the forward is pinned by
rotation / inversion equivariance (Wigner matrices recovered from the harmonics,
independent of the coupling tensor), by a brute-force dense contraction on tiny
graphs, and by the scalar special case, which is a sparse matrix product; the
backward by exact adjoint identities of a trilinear map and by central finite
differences.
"""
import numpy as np
import pytest
import scipy.sparse

from oracle import cg, conv, sh
from paper_2609_35099_b200 import workloads


def _random_graph(rng, n, e):
    rcv = np.sort(rng.integers(0, n, size=e)).astype(np.int32)
    snd = rng.integers(0, n, size=e).astype(np.int32)
    return snd, rcv


def _random_inputs(rng, cp, n, e):
    x = rng.standard_normal((n, cp.d, cp.nq)).astype(np.float32)
    y = rng.standard_normal((e, cp.dp)).astype(np.float32)
    s = rng.standard_normal((e, cp.P, cp.nq)).astype(np.float32)
    return x, y, s


def wigner_from_harmonics(l, R, rng):
    """D with Y_l(R u) = D Y_l(u), by least squares on random directions."""
    u = rng.standard_normal((8 * (2 * l + 1), 3))
    u /= np.linalg.norm(u, axis=1, keepdims=True)
    A, B = sh.real_sh(l, u), sh.real_sh(l, u @ R.T)
    D, res, rank, _ = np.linalg.lstsq(A, B, rcond=None)
    assert rank == 2 * l + 1
    return D.T


def block_rotation(irreps, R, rng):
    """Block-diagonal action of the orthogonal matrix R on a list of (l, parity) blocks."""
    det = np.sign(np.linalg.det(R))
    rot = R * det  # proper part
    blocks = []
    for l, p in irreps:
        D = wigner_from_harmonics(l, rot, rng)
        if det < 0:
            D = D * p
        blocks.append(D)
    return scipy.linalg.block_diag(*blocks)


@pytest.mark.parametrize("config,improper", [(1, False), (1, True), (2, False), (3, True)])
def test_forward_is_equivariant(config, improper):
    import scipy.linalg  # noqa: F401
    rng = np.random.default_rng(10 + config)
    c = workloads.CONFIGS[config]
    small = {1: 24, 2: 81, 3: 40}[config]
    wl = workloads.make_graph(config, n_atoms=small) if config != 2 else workloads.make_graph(2, n_atoms=192)
    irr = c["irreps_in"].replace("128x", "2x").replace("64x", "2x").replace("8x", "2x")
    cp = conv.Coupling(irr, c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    n, e = wl.n_nodes, wl.n_edges
    x = rng.standard_normal((n, cp.d, cp.nq)).astype(np.float32).astype(np.float64)
    s = rng.standard_normal((e, cp.P, cp.nq)).astype(np.float32)
    Q, _ = np.linalg.qr(rng.standard_normal((3, 3)))
    if (np.linalg.det(Q) < 0) != improper:
        Q = -Q
    unit = wl.vectors / np.linalg.norm(wl.vectors, axis=1, keepdims=True)
    y0 = sh.real_sh_all(cp.dp and c["sh_lmax"], unit)
    y1 = sh.real_sh_all(c["sh_lmax"], unit @ Q.T)
    in_irreps = [(l, p) for _, l, p in cg.parse_irreps(irr)]
    out_irreps = [(pth.L, pth.p) for pth in cp.paths]
    Din = block_rotation(in_irreps, Q, rng)
    Dout = block_rotation(out_irreps, Q, rng)
    x1 = np.einsum("ij,njq->niq", Din, x)
    # float32 storage of the rotated inputs would cost 1e-7; feed float64 through the
    # float32 interface by splitting into a float32 value and checking at 1e-6, and run a
    # strict float64 check through the dense numpy contraction below
    out0 = _dense_conv(cp, x, y0, s.astype(np.float64), wl.senders, wl.receivers)
    out1 = _dense_conv(cp, x1, y1, s.astype(np.float64), wl.senders, wl.receivers)
    assert np.abs(out1 - np.einsum("ij,njq->niq", Dout, out0)).max() < 1e-10 * max(1.0, np.abs(out0).max())
    # and the C loops agree with that dense contraction on the float32-representable inputs
    o = conv.conv_fwd(cp, x.astype(np.float32), y0.astype(np.float32), s, wl.senders, wl.receivers)
    ref = _dense_conv(cp, x.astype(np.float32).astype(np.float64), y0.astype(np.float32).astype(np.float64),
                      s.astype(np.float64), wl.senders, wl.receivers)
    assert np.abs(o - ref).max() < 1e-11 * max(1.0, np.abs(ref).max())


def _dense_conv(cp, x, y, s, senders, receivers):
    """Brute force: per-edge dense einsum, then an explicit scatter-add."""
    msg = np.einsum("ijk,ejq,ek->eiq", cp.C, x[senders], y) * s[:, cp.i3, :]
    out = np.zeros((x.shape[0], cp.D, cp.nq))
    np.add.at(out, receivers, msg)
    return out


@pytest.mark.parametrize("n,e", [(1, 1), (3, 7), (6, 20), (5, 0)])
def test_forward_matches_brute_force_on_tiny_graphs(n, e):
    rng = np.random.default_rng(100 + n + e)
    cp = conv.Coupling("3x0e+3x1o+3x2e", 2, None, 3)
    snd, rcv = _random_graph(rng, n, e)
    x, y, s = _random_inputs(rng, cp, n, e)
    got = conv.conv_fwd(cp, x, y, s, snd, rcv)
    want = _dense_conv(cp, x.astype(np.float64), y.astype(np.float64), s.astype(np.float64), snd, rcv)
    assert got.shape == want.shape
    assert np.abs(got - want).max() <= 1e-12 * max(1.0, np.abs(want).max(initial=0.0))


def test_scalar_special_case_is_a_sparse_matrix_product():
    rng = np.random.default_rng(7)
    cp = conv.Coupling("5x0e", 0, None, 0)
    assert (cp.P, cp.D, cp.d, cp.dp) == (1, 1, 1, 1)
    n, e = 30, 200
    snd, rcv = _random_graph(rng, n, e)
    x, y, s = _random_inputs(rng, cp, n, e)
    got = conv.conv_fwd(cp, x, y, s, snd, rcv)[:, 0, :]
    for q in range(cp.nq):
        A = scipy.sparse.coo_matrix((s[:, 0, q].astype(np.float64) * y[:, 0], (rcv, snd)), shape=(n, n)).tocsr()
        assert np.allclose(A @ x[:, 0, q].astype(np.float64), got[:, q], atol=1e-12)


def test_unsorted_receivers_are_rejected():
    cp = conv.Coupling("2x0e", 0)
    x, y, s = np.zeros((3, 1, 2), np.float32), np.zeros((2, 1), np.float32), np.zeros((2, 1, 2), np.float32)
    with pytest.raises(ValueError):
        conv.conv_fwd(cp, x, y, s, np.array([0, 1], np.int32), np.array([2, 0], np.int32))


def test_backward_is_the_exact_adjoint():
    """<dm, conv(v,y,s)> = <dx, v>, and likewise in y and s (the map is linear in each argument)."""
    rng = np.random.default_rng(8)
    cp = conv.Coupling("3x0e+3x1o", 2, "0e+1o+1e+2e+2o")
    n, e = 9, 40
    snd, rcv = _random_graph(rng, n, e)
    x, y, s = _random_inputs(rng, cp, n, e)
    dm = rng.standard_normal((n, cp.D, cp.nq)).astype(np.float32)
    dx, dy, ds = conv.conv_bwd(cp, x, y, s, snd, rcv, dm)
    f = lambda a, b, c_: conv.conv_fwd(cp, a, b, c_, snd, rcv)
    dm64 = dm.astype(np.float64)
    lhs_x = np.vdot(dm64, f(x, y, s)); rhs_x = np.vdot(dx, x.astype(np.float64))
    lhs_y = lhs_x; rhs_y = np.vdot(dy, y.astype(np.float64))
    rhs_s = np.vdot(ds, s.astype(np.float64))
    for rhs in (rhs_x, rhs_y, rhs_s):
        assert abs(lhs_x - rhs) <= 1e-12 * abs(lhs_x)
    # independent directions v != x
    v = rng.standard_normal(x.shape).astype(np.float32)
    assert abs(np.vdot(dm64, f(v, y, s)) - np.vdot(dx, v.astype(np.float64))) <= 1e-11 * abs(lhs_x)
    u = rng.standard_normal(y.shape).astype(np.float32)
    assert abs(np.vdot(dm64, f(x, u, s)) - np.vdot(dy, u.astype(np.float64))) <= 1e-11 * abs(lhs_x)
    t = rng.standard_normal(s.shape).astype(np.float32)
    assert abs(np.vdot(dm64, f(x, y, t)) - np.vdot(ds, t.astype(np.float64))) <= 1e-11 * abs(lhs_x)


def test_backward_matches_central_finite_differences():
    rng = np.random.default_rng(9)
    cp = conv.Coupling("2x0e+2x1o", 1, None, 2)
    n, e = 4, 9
    snd, rcv = _random_graph(rng, n, e)
    # values on a coarse binary grid so that +-h stays exactly representable in float32
    grid = lambda shape: (rng.integers(-8, 9, size=shape) / 4.0).astype(np.float32)
    x, y, s = grid((n, cp.d, cp.nq)), grid((e, cp.dp)), grid((e, cp.P, cp.nq))
    dm = grid((n, cp.D, cp.nq))
    dx, dy, ds = conv.conv_bwd(cp, x, y, s, snd, rcv, dm)
    h = np.float32(0.5)
    loss = lambda a, b, c_: float(np.vdot(dm.astype(np.float64), conv.conv_fwd(cp, a, b, c_, snd, rcv)))
    for arr, grad, pos in ((x, dx, 0), (y, dy, 1), (s, ds, 2)):
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, size=min(12, flat.size), replace=False):
            old = flat[idx]
            flat[idx] = old + h; up = loss(x, y, s)
            flat[idx] = old - h; dn = loss(x, y, s)
            flat[idx] = old
            assert (up - dn) / (2 * float(h)) == pytest.approx(grad.reshape(-1)[idx], abs=1e-9)


def test_tensor_product_equals_conv_on_the_identity_graph():
    rng = np.random.default_rng(11)
    cp = conv.Coupling("4x0e+4x1o+4x2e", 3, None, 3)
    B = 13
    x1 = rng.standard_normal((B, cp.d, cp.nq)).astype(np.float32)
    x2 = rng.standard_normal((B, cp.dp)).astype(np.float32)
    w = rng.standard_normal((B, cp.P, cp.nq)).astype(np.float32)
    dz = rng.standard_normal((B, cp.D, cp.nq)).astype(np.float32)
    ar = np.arange(B, dtype=np.int32)
    assert np.abs(conv.tp_fwd(cp, x1, x2, w) - conv.conv_fwd(cp, x1, x2, w, ar, ar)).max() < 1e-12
    a = conv.tp_bwd(cp, x1, x2, w, dz)
    b = conv.conv_bwd(cp, x1, x2, w, ar, ar, dz)
    for u, v in zip(a, b):
        assert np.abs(u - v).max() < 1e-11


def test_empty_receivers_give_zero_rows_and_silent_senders_zero_gradients():
    rng = np.random.default_rng(12)
    cp = conv.Coupling("2x0e+2x1o", 1)
    n = 6
    snd = np.array([0, 0, 1], np.int32); rcv = np.array([2, 2, 4], np.int32)
    x, y, s = _random_inputs(rng, cp, n, 3)
    out = conv.conv_fwd(cp, x, y, s, snd, rcv)
    assert np.all(out[[0, 1, 3, 5]] == 0) and np.abs(out[2]).max() > 0
    dx, dy, ds = conv.conv_bwd(cp, x, y, s, snd, rcv, rng.standard_normal(out.shape).astype(np.float32))
    assert np.all(dx[2:] == 0) and np.abs(dx[0]).max() > 0


def test_padding_edges_take_no_part():
    """Padded edge list (receiver id >= number of nodes marks padding): the real edges give exactly the
    unpadded result whatever the padding entries hold, padding rows of the edge-local cotangents are zero."""
    rng = np.random.default_rng(13)
    cp = conv.Coupling("2x0e+2x1o", 1)
    n, e, pad = 5, 7, 4
    snd = rng.integers(0, n, e).astype(np.int32); rcv = np.sort(rng.integers(0, n, e)).astype(np.int32)
    x, y, s = _random_inputs(rng, cp, n, e)
    dm = rng.standard_normal((n, cp.D, cp.nq)).astype(np.float32)
    ref = conv.conv_fwd(cp, x, y, s, snd, rcv)
    rx, ry, rs = conv.conv_bwd(cp, x, y, s, snd, rcv, dm)
    yp = np.concatenate([y, np.full((pad, cp.dp), np.nan, np.float32)])
    sp = np.concatenate([s, np.full((pad, cp.P, cp.nq), np.inf, np.float32)])
    sndp = np.concatenate([snd, np.full(pad, -5, np.int32)])
    rcvp = np.concatenate([rcv, np.array([n, n, n + 3, 2 ** 30], np.int32)])
    assert np.array_equal(conv.conv_fwd_padded(cp, x, yp, sp, sndp, rcvp), ref)
    dx, dy, ds = conv.conv_bwd_padded(cp, x, yp, sp, sndp, rcvp, dm)
    assert np.array_equal(dx, rx) and np.array_equal(dy[:e], ry) and np.array_equal(ds[:e], rs)
    assert np.all(dy[e:] == 0) and np.all(ds[e:] == 0)
    # nothing but padding: zero output, zero gradients
    out0 = conv.conv_fwd_padded(cp, x, yp[e:], sp[e:], sndp[e:], rcvp[e:])
    assert out0.shape == ref.shape and np.all(out0 == 0)


def test_collapsed_outputs_against_a_direct_sum_over_paths():
    """Collapsed multiplicities: paths landing on the same (L, parity) add into one block.  Checked against
    the sum written path by path (one dense contraction per path, added into the block of its irrep), against
    the uncollapsed result when no two paths share an irrep, and through the adjoint identity."""
    rng = np.random.default_rng(21)
    cp = conv.Coupling("2x0e+2x1o", 2)
    n, e = 5, 9
    snd = rng.integers(0, n, e).astype(np.int32); rcv = np.sort(rng.integers(0, n, e)).astype(np.int32)
    x, y, s = _random_inputs(rng, cp, n, e)
    R, offs = conv.collapse_matrix(cp)
    keys = sorted({(p.L, p.p) for p in cp.paths})
    assert R.shape == (sum(2 * L + 1 for L, _ in keys), cp.D) and len(keys) < cp.P
    got = conv.conv_fwd_collapsed(cp, x, y, s, snd, rcv)
    want = np.zeros_like(got)
    x64, y64, s64 = x.astype(np.float64), y.astype(np.float64), s.astype(np.float64)
    for p, off in zip(cp.paths, offs):
        Ck = cp.C[p.out_off:p.out_off + 2 * p.L + 1]          # [2L+1, d, d'] of this path alone
        for ed in range(e):
            m = np.einsum("mij,iq,j->mq", Ck, x64[snd[ed]], y64[ed]) * s64[ed, p.k][None, :]
            want[rcv[ed], off:off + 2 * p.L + 1] += m
    assert np.abs(got - want).max() < 1e-12
    # adjoint identity through the collapsed map
    dm = rng.standard_normal(got.shape).astype(np.float32)
    dx, dy, ds = conv.conv_bwd_collapsed(cp, x, y, s, snd, rcv, dm)
    lhs = float((dm.astype(np.float64) * got).sum())
    assert abs(lhs - float((dx * x64).sum())) < 1e-10 * abs(lhs)
    assert abs(lhs - float((dy * y64).sum())) < 1e-10 * abs(lhs)
    assert abs(lhs - float((ds * s64).sum())) < 1e-10 * abs(lhs)
    # one path per irrep: nothing to collapse
    cp1 = conv.Coupling("2x0e", 2)
    R1, _ = conv.collapse_matrix(cp1)
    assert np.array_equal(R1, np.eye(cp1.D))


def test_double_backward_is_the_derivative_of_the_backward():
    """Phi = <ux, dx> + <uy, dy> + <us, ds> with (dx, dy, ds) = conv_bwd(x, y, s, dm) is linear in each of
    x, y, s, dm, so central differences of Phi give its gradient up to rounding; the double backward must
    return exactly that gradient."""
    rng = np.random.default_rng(31)
    cp = conv.Coupling("2x0e+2x1o", 2)
    n, e = 4, 7
    snd = rng.integers(0, n, e).astype(np.int32); rcv = np.sort(rng.integers(0, n, e)).astype(np.int32)
    x, y, s = _random_inputs(rng, cp, n, e)
    dm = rng.standard_normal((n, cp.D, cp.nq)).astype(np.float32)
    ux, uy, us = _random_inputs(rng, cp, n, e)
    # inputs on a binary grid, so that adding the step is exact in float32 (the oracle takes float32 inputs)
    x, y, s, dm = [np.round(a * 256.0) / 256.0 for a in (x, y, s, dm)]
    x, y, s, dm = [a.astype(np.float32) for a in (x, y, s, dm)]
    got = conv.conv_bwd_bwd(cp, x, y, s, snd, rcv, dm, ux, uy, us)

    def phi(x_, y_, s_, dm_):
        dx, dy, ds = conv.conv_bwd(cp, x_, y_, s_, snd, rcv, dm_)
        return float((ux * dx).sum() + (uy * dy).sum() + (us * ds).sum())

    args = [x, y, s, dm]
    h = 0.25   # exactly representable; Phi is linear in every argument
    for which, grad in zip((3, 0, 1, 2), got):
        base = args[which]
        flat_idx = rng.choice(base.size, size=min(12, base.size), replace=False)
        for fi in flat_idx:
            idx = np.unravel_index(fi, base.shape)
            plus = [a.copy() for a in args]; minus = [a.copy() for a in args]
            plus[which][idx] += h; minus[which][idx] -= h
            fd = (phi(*plus) - phi(*minus)) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-9 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])


def test_conv_from_edge_vectors_backward_matches_a_directional_difference():
    """conv_vec_bwd's dvec against central differences of sum(g * conv_vec_fwd) along a random direction; the
    vectors sit on a binary grid so that vec +- h * delta is exact in float32 (the rounding of y to float32 inside
    the forward leaves noise of about 1e-4 of the derivative)."""
    rng = np.random.default_rng(21)
    cp = conv.Coupling("4x0e+4x1o", 2)
    n, e = 5, 14
    snd = rng.integers(0, n, size=e).astype(np.int32)
    rcv = np.sort(rng.integers(0, n, size=e)).astype(np.int32)
    x = rng.standard_normal((n, cp.d, cp.nq)).astype(np.float32)
    s = rng.standard_normal((e, cp.P, cp.nq)).astype(np.float32)
    g = rng.standard_normal((n, cp.D, cp.nq)).astype(np.float32)
    vec = (np.round(rng.uniform(-2, 2, size=(e, 3)) * 64) / 64).astype(np.float32)
    vec[np.abs(vec).sum(axis=1) < 0.5] += 1.0
    delta = rng.choice([-1.0, 1.0], size=(e, 3)).astype(np.float32)
    h = 2.0 ** -8
    phi = lambda v: float(np.sum(g.astype(np.float64) * conv.conv_vec_fwd(cp, x, v, s, snd, rcv)))
    fd = (phi(vec + h * delta) - phi(vec - h * delta)) / (2 * h)
    dx, dvec, ds = conv.conv_vec_bwd(cp, x, vec, s, snd, rcv, g)
    assert abs(fd - float(np.sum(dvec * delta))) < 2e-3 * max(1.0, np.abs(dvec).sum())
    # the other two cotangents are those of the convolution with the same harmonics
    y = sh.real_sh_all_of_vectors(2, vec.astype(np.float64)).astype(np.float32)
    dx2, _, ds2 = conv.conv_bwd(cp, x, y, s, snd, rcv, g)
    assert np.array_equal(dx, dx2) and np.array_equal(ds, ds2)
    # a vector's length does not matter to the forward
    assert np.allclose(conv.conv_vec_fwd(cp, x, 2 * vec, s, snd, rcv), conv.conv_vec_fwd(cp, x, vec, s, snd, rcv),
                       atol=1e-5)
