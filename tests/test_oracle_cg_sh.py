"""Pins for the oracle's coefficient and harmonics code (CPU only).

The paper prints no numerical coefficient, so every pin is a textbook value, an
identity of angular-momentum algebra, or a cross-check between two independent
constructions.
"""
import math
import os

import numpy as np
import pytest

from oracle import cg, sh

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "su2_cg_textbook.txt")


def test_complex_cg_textbook_values():
    n = 0
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        l1, m1, l2, m2, L, M, sg, nu, de = map(int, line.split())
        assert cg.su2_cg(l1, m1, l2, m2, L, M) == pytest.approx(sg * math.sqrt(nu / de), abs=1e-14)
        n += 1
    assert n >= 20


@pytest.mark.parametrize("l1,l2", [(a, b) for a in range(5) for b in range(5)])
def test_complex_cg_orthogonality_completeness_symmetry(l1, l2):
    blocks = {L: cg.complex_cg_block(l1, l2, L) for L in range(abs(l1 - l2), l1 + l2 + 1)}
    for L, C in blocks.items():
        # orthonormal rows: sum_{m1 m2} C^{LM} C^{LM'} = delta
        G = np.einsum("Mab,Nab->MN", C, C)
        assert np.allclose(G, np.eye(2 * L + 1), atol=1e-14)
        # exchange symmetry C(l2,l1) = (-1)^{l1+l2-L} C(l1,l2)
        Cs = cg.complex_cg_block(l2, l1, L)
        assert np.allclose(Cs, (-1) ** (l1 + l2 - L) * np.transpose(C, (0, 2, 1)), atol=1e-14)
    # completeness: sum_{L M} C C = delta delta
    tot = sum(np.einsum("Mab,Mcd->abcd", C, C) for C in blocks.values())
    n1, n2 = 2 * l1 + 1, 2 * l2 + 1
    assert np.allclose(tot.reshape(n1 * n2, n1 * n2), np.eye(n1 * n2), atol=1e-13)


@pytest.mark.parametrize("l", range(5))
def test_coupling_with_scalar_is_identity(l):
    assert np.allclose(cg.complex_cg_block(l, 0, l)[:, :, 0], np.eye(2 * l + 1), atol=1e-15)
    assert np.allclose(cg.real_cg_block(l, 0, l)[:, :, 0], np.eye(2 * l + 1), atol=1e-15)
    assert np.allclose(cg.real_cg_block(0, l, l)[:, 0, :], np.eye(2 * l + 1), atol=1e-15)


def test_real_basis_is_unitary():
    for l in range(6):
        U = cg.real_basis(l)
        assert np.allclose(U @ U.conj().T, np.eye(2 * l + 1), atol=1e-15)


def test_vector_couplings_closed_forms():
    # 1 x 1 -> 0 is +dot/sqrt(3)
    assert np.allclose(cg.real_cg_block(1, 1, 0)[0], np.eye(3) / math.sqrt(3), atol=1e-15)
    # 1 x 1 -> 1 is +cross/sqrt(2) with components ordered (y, z, x)
    T = cg.real_cg_block(1, 1, 1)
    perm = [2, 0, 1]  # position of x, y, z inside the (y, z, x) ordering
    rng = np.random.default_rng(0)
    for _ in range(5):
        a, b = rng.standard_normal(3), rng.standard_normal(3)
        a_yzx, b_yzx = a[[1, 2, 0]], b[[1, 2, 0]]
        got = np.einsum("Mab,a,b->M", T, a_yzx, b_yzx)
        want = np.cross(a, b)[[1, 2, 0]] / math.sqrt(2)
        assert np.allclose(got, want, atol=1e-14)
    assert perm == [2, 0, 1]


@pytest.mark.parametrize("l1,l2", [(a, b) for a in range(4) for b in range(4)])
def test_real_cg_orthogonal_and_sparse(l1, l2):
    for L in range(abs(l1 - l2), l1 + l2 + 1):
        T = cg.real_cg_block(l1, l2, L)
        G = np.einsum("Mab,Nab->MN", T, T)
        assert np.allclose(G, np.eye(2 * L + 1), atol=1e-14)
        for M in range(-L, L + 1):
            for m1 in range(-l1, l1 + 1):
                for m2 in range(-l2, l2 + 1):
                    if T[M + L, m1 + l1, m2 + l2] != 0.0:
                        assert abs(M) in (abs(m1) + abs(m2), abs(abs(m1) - abs(m2)))
        nz = T.ravel()[np.flatnonzero(T.ravel())]
        assert nz[0] > 0  # canonical sign


def test_table_sizes_of_the_five_configurations():
    cases = [
        (("8x0e+8x1o", 2, "0e+1o+1e+2e+2o", None), (9, 29, 59, 55)),
        (("128x0e+128x1o", 3, None, 3), (13, 55, 134, 116)),
        (("128x0e+128x1o", 3, "0e+1o+2e+3o", None), (10, 40, 86, 76)),
        (("64x0e+64x1o+64x2e+64x3o", 3, None, 3), (34, 156, 611, 541)),
        (("128x0e+128x1o+128x2e", 3, None, 3), (24, 106, 351, 303)),
    ]
    for args, (P, D, nnz, pairs) in cases:
        C, i3, paths, nq = cg.dense_coupling(*args)
        assert (len(paths), C.shape[0], np.count_nonzero(C)) == (P, D, nnz)
        assert np.count_nonzero(np.abs(C).sum(axis=2)) == pairs
        assert list(i3) == sorted(i3)  # blocks are contiguous and ordered
        # independent count of allowed (l1, l2, L, parity) triples
        ins = cg.parse_irreps(args[0])
        wanted = cg.default_output_order(args[3]) if args[2] is None else \
            [(l, p) for _, l, p in cg.parse_irreps(args[2])]
        cnt = sum(1 for _, l1, p1 in ins for l2 in range(args[1] + 1)
                  for L in range(abs(l1 - l2), l1 + l2 + 1) if (L, p1 * (-1) ** l2) in wanted)
        assert cnt == P


def test_path_order_rule():
    nq, d, dp, D, paths = cg.enumerate_paths("8x0e+8x1o", 2, "0e+1o+1e+2e+2o")
    got = [(p.L, p.p, p.in_index, p.l2) for p in paths]
    want = [(0, 1, 0, 0), (0, 1, 1, 1), (1, -1, 0, 1), (1, -1, 1, 0), (1, -1, 1, 2), (1, 1, 1, 1),
            (2, 1, 0, 2), (2, 1, 1, 1), (2, -1, 1, 2)]
    assert got == want
    assert (nq, d, dp, D) == (8, 4, 9, 29)


# ------------------------------------------------------------------ harmonics
def _unit(n, seed=0):
    v = np.random.default_rng(seed).standard_normal((n, 3))
    return v / np.linalg.norm(v, axis=1, keepdims=True)


@pytest.mark.parametrize("l", range(6))
def test_sh_addition_theorem(l):
    u, v = _unit(40, 1), _unit(40, 2)
    lhs = np.einsum("nm,nm->n", sh.real_sh(l, u), sh.real_sh(l, v))
    cosg = np.einsum("ni,ni->n", u, v)
    Pl = np.polynomial.legendre.Legendre.basis(l)(cosg)
    assert np.allclose(lhs, (2 * l + 1) * Pl, atol=1e-12)


def test_sh_low_degree_closed_forms():
    u = _unit(30, 3)
    assert np.allclose(sh.real_sh(0, u), 1.0)
    assert np.allclose(sh.real_sh(1, u), math.sqrt(3) * u[:, [1, 2, 0]], atol=1e-14)
    x, y, z = u.T
    assert np.allclose(sh.real_sh(2, u)[:, 2], math.sqrt(5) / 2 * (3 * z * z - 1), atol=1e-14)
    assert np.allclose(sh.real_sh(2, u)[:, 4], math.sqrt(15) / 2 * (x * x - y * y), atol=1e-14)


@pytest.mark.parametrize("l", range(1, 5))
def test_sh_is_harmonic_and_homogeneous(l):
    """r^l Y_l(r/|r|) must satisfy Laplace's equation (finite differences)."""
    def solid(p):
        r = np.linalg.norm(p, axis=1, keepdims=True)
        return r ** l * sh.real_sh(l, p / r)
    p0 = np.random.default_rng(4).uniform(0.5, 1.5, size=(6, 3))
    h = 1e-3
    lap = -6 * solid(p0)
    for ax in range(3):
        e = np.zeros(3); e[ax] = h
        lap = lap + solid(p0 + e) + solid(p0 - e)
    lap /= h * h
    # exact Laplacian is 0; the stencil's own error is O(h^2) times a 4th derivative
    assert np.abs(lap).max() < 2e-4 * max(1.0, np.abs(solid(p0)).max())


@pytest.mark.parametrize("l1,l2", [(a, b) for a in range(4) for b in range(4)])
def test_gaunt_relation_ties_real_cg_to_real_sh(l1, l2):
    """(Y_l1(r) x Y_l2(r))_L = sqrt((2l1+1)(2l2+1)/(2L+1)) <l1 0 l2 0|L 0> Y_L(r), up to the path sign."""
    u = _unit(25, 5)
    for L in range(abs(l1 - l2), l1 + l2 + 1):
        T = cg.real_cg_block(l1, l2, L)
        got = np.einsum("Mab,na,nb->nM", T, sh.real_sh(l1, u), sh.real_sh(l2, u))
        fac = math.sqrt((2 * l1 + 1) * (2 * l2 + 1) / (2 * L + 1)) * cg.su2_cg(l1, 0, l2, 0, L, 0)
        want = fac * sh.real_sh(L, u)
        if (l1 + l2 + L) % 2 == 1:
            assert np.abs(got).max() < 1e-13
        else:
            assert np.allclose(got, want, atol=1e-13) or np.allclose(got, -want, atol=1e-13)
            assert abs(fac) > 1e-3


def test_workload_harmonics_match_the_oracle():
    from paper_2609_35099_b200 import workloads
    u = _unit(200, 6)
    for lmax in range(4):
        assert np.allclose(workloads.spherical_harmonics(lmax, u), sh.real_sh_all(lmax, u), atol=1e-14)


# ------------------------------------------------------------------ harmonics of edge vectors and their gradient
def _vectors(n, seed):
    rng = np.random.default_rng(seed)
    return _unit(n, seed) * rng.uniform(0.7, 5.0, size=(n, 1))


def test_sh_of_vectors_ignores_the_length():
    v = _vectors(50, 7)
    u = v / np.linalg.norm(v, axis=1, keepdims=True)
    assert np.allclose(sh.real_sh_all_of_vectors(3, v), sh.real_sh_all(3, u), atol=1e-14)
    assert np.allclose(sh.real_sh_all_of_vectors(3, 3.7 * v), sh.real_sh_all(3, u), atol=1e-13)
    with pytest.raises(ValueError):
        sh.real_sh_all_of_vectors(2, np.zeros((1, 3)))


def test_sh_vjp_closed_forms_for_l1_and_l2():
    """d/dv of sqrt(3) (y, z, x) / r and of sqrt(5)/2 (3 z^2 / r^2 - 1), written out by hand."""
    v = _vectors(40, 8)
    x, y, z = v.T
    r = np.linalg.norm(v, axis=1)
    g = np.random.default_rng(9).standard_normal((40, 9))
    got = sh.real_sh_all_vjp(2, v, g)
    # l = 1: Y = sqrt(3) (y, z, x) / r  ->  dY_a/dv_b = sqrt(3) (delta_ab / r - v_a v_b / r^3)
    g1 = g[:, 1:4]                         # cotangents of (y, z, x) components
    gv = np.stack([g1[:, 2], g1[:, 0], g1[:, 1]], axis=1)   # reordered to (x, y, z)
    want = math.sqrt(3) * (gv / r[:, None] - v * np.einsum("ni,ni->n", gv, v)[:, None] / r[:, None] ** 3)
    # l = 2, m = 0: Y = sqrt(5)/2 (3 z^2 / r^2 - 1)  ->  grad = sqrt(5)/2 * 3 * (2 z e_z / r^2 - 2 z^2 v / r^4)
    ez = np.zeros_like(v); ez[:, 2] = 1.0
    want += (g[:, 6] * math.sqrt(5) / 2 * 3)[:, None] * (2 * z[:, None] * ez / r[:, None] ** 2
                                                          - 2 * (z ** 2)[:, None] * v / r[:, None] ** 4)
    only = np.zeros_like(g); only[:, 1:4] = g[:, 1:4]; only[:, 6] = g[:, 6]
    assert np.allclose(sh.real_sh_all_vjp(2, v, only), want, atol=1e-8)
    # the other components contribute too: the full product differs from the partial one
    assert np.abs(got - want).max() > 1e-3


def test_sh_vjp_is_tangential_and_scales_inversely_with_the_length():
    """Y depends on the direction only: v . grad = 0, and grad(c v) = grad(v) / c."""
    v = _vectors(30, 10)
    g = np.random.default_rng(11).standard_normal((30, 16))
    gv = sh.real_sh_all_vjp(3, v, g)
    assert np.abs(np.einsum("ni,ni->n", gv, v)).max() < 1e-7
    assert np.allclose(sh.real_sh_all_vjp(3, 2.5 * v, g), gv / 2.5, atol=1e-8)
    # Y_0 is constant
    g0 = np.zeros_like(g); g0[:, 0] = 1.0
    assert np.abs(sh.real_sh_all_vjp(3, v, g0)).max() < 1e-9


def test_sh_vjp_agrees_with_the_rotation_generators():
    """An infinitesimal rotation of v about axis a changes Y_l by the action of the real generator: checked through
    the invariance of sum_m Y_lm(v) Y_lm(w) under a joint rotation, i.e. grad_v[Y(v).Y(w)] x v + grad_w[...] x w = 0."""
    v, w = _vectors(20, 12), _vectors(20, 13)
    for l in (1, 2, 3):
        sl = slice(l * l, (l + 1) * (l + 1))
        Yv, Yw = sh.real_sh_all_of_vectors(3, v), sh.real_sh_all_of_vectors(3, w)
        gv_in, gw_in = np.zeros_like(Yv), np.zeros_like(Yw)
        gv_in[:, sl], gw_in[:, sl] = Yw[:, sl], Yv[:, sl]
        gv = sh.real_sh_all_vjp(3, v, gv_in)
        gw = sh.real_sh_all_vjp(3, w, gw_in)
        torque = np.cross(v, gv) + np.cross(w, gw)
        assert np.abs(torque).max() < 1e-6
