"""Pins for the oracle's convolution with edge scalars taken from the radial network's last layer (CPU only).

The radial functions are the convolution of test_oracle_conv.py fed s = h W.  They are pinned against things
that do not go through their own matrix product: an explicit triple loop on tiny inputs whose products are
exact in float32, one-hot and constant hidden activations (closed forms), the exact adjoint identities of a
map that is linear in h and in W, and central differences that are exact on a binary grid.
"""
import numpy as np
import pytest

from oracle import conv


def _graph(rng, n, e):
    rcv = np.sort(rng.integers(0, n, size=e)).astype(np.int32)
    snd = rng.integers(0, n, size=e).astype(np.int32)
    return snd, rcv


def _grid(rng, shape, lo=-4, hi=5, step=2.0):
    """Small dyadic values: sums of a few products of them are exact in float32 and float64."""
    return (rng.integers(lo, hi, size=shape) / step).astype(np.float32)


def _case(seed, irreps="3x0e+3x1o", lmax=2, irreps_out="0e+1o+1e+2e+2o", n=7, e=23, H=5, grid=False):
    rng = np.random.default_rng(seed)
    cp = conv.Coupling(irreps, lmax, irreps_out)
    snd, rcv = _graph(rng, n, e)
    draw = (lambda s: _grid(rng, s)) if grid else (lambda s: rng.standard_normal(s).astype(np.float32))
    x, y = draw((n, cp.d, cp.nq)), draw((e, cp.dp))
    h, W = draw((e, H)), draw((H, cp.P * cp.nq))
    dm = draw((n, cp.D, cp.nq))
    return rng, cp, snd, rcv, x, y, h, W, dm


def test_radial_forward_equals_the_convolution_of_the_product_written_as_loops():
    rng, cp, snd, rcv, x, y, h, W, dm = _case(1, grid=True)
    e, H = h.shape
    s = np.zeros((e, cp.P, cp.nq), np.float32)
    for edge in range(e):
        for k in range(cp.P):
            for q in range(cp.nq):
                acc = 0.0
                for j in range(H):
                    acc += float(h[edge, j]) * float(W[j, k * cp.nq + q])
                s[edge, k, q] = acc            # exact: dyadic inputs, |acc| small
                assert float(s[edge, k, q]) == acc
    want = conv.conv_fwd(cp, x, y, s, snd, rcv)
    got = conv.conv_radial_fwd(cp, x, y, h, W, snd, rcv)
    assert np.array_equal(got, want)           # same doubles go into the same sums
    dx0, dy0, ds0 = conv.conv_bwd(cp, x, y, s, snd, rcv, dm)
    dx, dy, dh, dW = conv.conv_radial_bwd(cp, x, y, h, W, snd, rcv, dm)
    assert np.array_equal(dx, dx0) and np.array_equal(dy, dy0)
    # chain rule through the product, again as loops
    for edge in rng.choice(e, size=5, replace=False):
        for j in range(H):
            want_h = sum(ds0[edge, k, q] * float(W[j, k * cp.nq + q]) for k in range(cp.P) for q in range(cp.nq))
            assert dh[edge, j] == pytest.approx(want_h, abs=1e-9)
    for j in range(H):
        for col in rng.choice(cp.P * cp.nq, size=6, replace=False):
            k, q = divmod(int(col), cp.nq)
            want_w = sum(float(h[edge, j]) * ds0[edge, k, q] for edge in range(e))
            assert dW[j, col] == pytest.approx(want_w, abs=1e-9)


def test_one_hot_hidden_activations_select_one_row_of_the_layer():
    rng, cp, snd, rcv, x, y, h, W, dm = _case(2)
    e, H = h.shape
    pick = rng.integers(0, H, size=e)
    h1 = np.zeros_like(h)
    h1[np.arange(e), pick] = 1.0
    s = W[pick].reshape(e, cp.P, cp.nq)        # float32 values, no arithmetic
    assert np.array_equal(conv.conv_radial_fwd(cp, x, y, h1, W, snd, rcv), conv.conv_fwd(cp, x, y, s, snd, rcv))


def test_constant_hidden_activation_scales_the_output():
    rng, cp, snd, rcv, x, y, h, W, dm = _case(3, H=1)
    ones = np.ones_like(h)
    base = conv.conv_radial_fwd(cp, x, y, ones, W, snd, rcv)
    s = np.broadcast_to(W.reshape(1, cp.P, cp.nq), (len(snd), cp.P, cp.nq))
    assert np.array_equal(base, conv.conv_fwd(cp, x, y, s, snd, rcv))
    # doubling every hidden activation doubles every message (exact in binary floating point)
    assert np.array_equal(conv.conv_radial_fwd(cp, x, y, 2 * ones, W, snd, rcv), 2 * base)


def test_radial_backward_is_the_exact_adjoint_in_h_and_W():
    rng, cp, snd, rcv, x, y, h, W, dm = _case(4, n=9, e=40, H=6)
    dx, dy, dh, dW = conv.conv_radial_bwd(cp, x, y, h, W, snd, rcv, dm)
    dm64 = dm.astype(np.float64)
    f = lambda hh, ww: conv.conv_radial_fwd(cp, x, y, hh, ww, snd, rcv)
    ref = np.vdot(dm64, f(h, W))
    assert abs(ref - np.vdot(dh, h.astype(np.float64))) <= 1e-12 * abs(ref)
    assert abs(ref - np.vdot(dW, W.astype(np.float64))) <= 1e-12 * abs(ref)
    v = rng.standard_normal(h.shape).astype(np.float32)
    V = rng.standard_normal(W.shape).astype(np.float32)
    assert abs(np.vdot(dm64, f(v, W)) - np.vdot(dh, v.astype(np.float64))) <= 1e-11 * abs(ref)
    assert abs(np.vdot(dm64, f(h, V)) - np.vdot(dW, V.astype(np.float64))) <= 1e-11 * abs(ref)
    # x and y: the same identities as for the plain convolution, through the radial entry points
    u = rng.standard_normal(x.shape).astype(np.float32)
    t = rng.standard_normal(y.shape).astype(np.float32)
    assert abs(np.vdot(dm64, conv.conv_radial_fwd(cp, u, y, h, W, snd, rcv)) - np.vdot(dx, u.astype(np.float64))) <= 1e-11 * abs(ref)
    assert abs(np.vdot(dm64, conv.conv_radial_fwd(cp, x, t, h, W, snd, rcv)) - np.vdot(dy, t.astype(np.float64))) <= 1e-11 * abs(ref)


def test_radial_backward_matches_central_differences():
    rng, cp, snd, rcv, x, y, h, W, dm = _case(5, irreps="2x0e+2x1o", lmax=1, irreps_out=None, n=4, e=9, H=3, grid=True)
    cp = conv.Coupling("2x0e+2x1o", 1, None, 2)
    W = _grid(rng, (3, cp.P * cp.nq)); dm = _grid(rng, (4, cp.D, cp.nq))
    dx, dy, dh, dW = conv.conv_radial_bwd(cp, x, y, h, W, snd, rcv, dm)
    step = np.float32(0.5)
    loss = lambda: float(np.vdot(dm.astype(np.float64), conv.conv_radial_fwd(cp, x, y, h, W, snd, rcv)))
    for arr, grad in ((h, dh), (W, dW), (x, dx), (y, dy)):
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, size=min(10, flat.size), replace=False):
            old = flat[idx]
            flat[idx] = old + step; up = loss()
            flat[idx] = old - step; dn = loss()
            flat[idx] = old
            assert (up - dn) / (2 * float(step)) == pytest.approx(grad.reshape(-1)[idx], abs=1e-9)


def test_radial_product_is_not_rounded_to_float32():
    """s = h W keeps its float64 value: a product that float32 cannot hold still reaches the output."""
    cp = conv.Coupling("1x0e", 0, None, 0)     # out[b] = sum_e s[e] x[snd] y[e], one scalar path, C = 1
    x = np.ones((1, 1, 1), np.float32); y = np.ones((1, 1), np.float32)
    h = np.array([[1.0, 2.0 ** -30]], np.float32); W = np.array([[1.0], [1.0]], np.float32)
    snd = rcv = np.zeros(1, np.int32)
    out = conv.conv_radial_fwd(cp, x, y, h, W, snd, rcv)
    assert out[0, 0, 0] == 1.0 + 2.0 ** -30
