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


def real_sh_all_of_vectors(lmax: int, vec: np.ndarray, normalization: str = "component") -> np.ndarray:
    """Harmonic embedding of edge vectors: Y(vec / |vec|), [n, (lmax+1)^2] (the paper's "Key Operations in Scope":
    the harmonics are functions of the edge direction).  A zero vector has no direction: rejected here."""
    vec = np.asarray(vec, dtype=np.float64)
    r = np.linalg.norm(vec, axis=1, keepdims=True)
    if np.any(r == 0):
        raise ValueError("zero-length edge vector")
    return real_sh_all(lmax, vec / r, normalization)


def real_sh_all_vjp(lmax: int, vec: np.ndarray, grad_sh: np.ndarray, step: float = 1e-6) -> np.ndarray:
    """grad_vec[n, 3] = sum_i grad_sh[n, i] d Y_i(vec / |vec|) / d vec, by the definition of the derivative:
    central differences in float64 with a step relative to |vec| (truncation error ~ step^2 = 1e-12 relative,
    rounding ~ 1e-16 / step = 1e-10: far below the float32 kernels this is compared with)."""
    vec = np.asarray(vec, dtype=np.float64)
    grad_sh = np.asarray(grad_sh, dtype=np.float64)
    r = np.linalg.norm(vec, axis=1)
    out = np.zeros_like(vec)
    for axis in range(3):
        d = np.zeros_like(vec)
        d[:, axis] = step * r
        plus = real_sh_all_of_vectors(lmax, vec + d)
        minus = real_sh_all_of_vectors(lmax, vec - d)
        out[:, axis] = np.einsum("ni,ni->n", grad_sh, plus - minus) / (2 * step * r)
    return out
