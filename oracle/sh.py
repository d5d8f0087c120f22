"""Oracle: real spherical harmonics of unit vectors (test infrastructure only).

The paper's harmonic embedding stacks Y_l(r) = [Y_lm(r) | m = -l..l] for
l = 0..l_max ("Key Operations in Scope", harmonics item) and builds the
complex Y_l^m from Y_l^{+-l} = c_l (x +- i y)^l with z the polar axis
("Reconstruction of harmonic polynomials").  The normalisation factor c_l is
left open there; the reading taken here is "component" normalisation,
sum_m Y_lm(r)^2 = 2l+1 on the unit sphere (so Y_0 = 1), and the real basis of
oracle.cg.real_basis.

Computed from the textbook complex definition
    Y_l^m = (-1)^m N_lm (x + i y)^m  d^m P_l(z)/dz^m          (m >= 0)
    Y_l^{-m} = (-1)^m conj(Y_l^m)
with N_lm = sqrt((2l+1)/(4 pi) (l-m)!/(l+m)!), for any degree, in float64.
"""
from __future__ import annotations

import math

import numpy as np
from numpy.polynomial import legendre as npleg

from .cg import real_basis


def complex_sh(l: int, xyz: np.ndarray) -> np.ndarray:
    """Orthonormal complex Y_l^m of unit vectors, shape [n, 2l+1], index m+l."""
    xyz = np.asarray(xyz, dtype=np.float64)
    x, y, z = xyz[:, 0], xyz[:, 1], xyz[:, 2]
    out = np.zeros((xyz.shape[0], 2 * l + 1), dtype=complex)
    basis = npleg.Legendre.basis(l)
    for m in range(0, l + 1):
        dP = basis.deriv(m)(z) if m > 0 else basis(z)
        N = math.sqrt((2 * l + 1) / (4 * math.pi) * math.factorial(l - m) / math.factorial(l + m))
        Ylm = (-1) ** m * N * (x + 1j * y) ** m * dP
        out[:, l + m] = Ylm
        if m > 0:
            out[:, l - m] = (-1) ** m * np.conj(Ylm)
    return out


def real_sh(l: int, xyz: np.ndarray, normalization: str = "component") -> np.ndarray:
    """Real Y_lm of unit vectors, [n, 2l+1], m = -l..l."""
    Yc = complex_sh(l, xyz)
    Yr = Yc @ real_basis(l).T
    assert np.abs(Yr.imag).max(initial=0.0) < 1e-12
    Yr = Yr.real
    if normalization == "component":
        Yr = Yr * math.sqrt(4 * math.pi)
    elif normalization != "orthonormal":
        raise ValueError(normalization)
    return Yr


def real_sh_all(lmax: int, xyz: np.ndarray, normalization: str = "component") -> np.ndarray:
    """Concatenation over l = 0..lmax, shape [n, (lmax+1)^2]."""
    return np.concatenate([real_sh(l, xyz, normalization) for l in range(lmax + 1)], axis=1)
