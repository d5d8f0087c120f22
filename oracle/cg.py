"""Oracle: real Clebsch-Gordan coupling tensors (test infrastructure only).

What the paper fixes: the tensor product couples x (degree l) and y (degree l')
into every output degree L = |l-l'| .. l+l' with "the Clebsch-Gordan
coefficients" (section "Key Operations in Scope", tensor-product equation), the
components of a degree-l block are ordered m = -l .. l (harmonics equation of
the same section), output multiplicities are kept (one output block per path,
"Notation": m_b "does not have the same feature dimension as x as
multiplicities arise"), and the index i3(i0) sends an output coordinate to its
irreducible block, which selects the edge scalar (edge-scalar-weighting
equation).

What the paper leaves open, and the reading taken here:
  * normalisation: unitary CG (sum over (m1,m2) of C^2 = 1 for each (L,M));
    no extra path or component weights.
  * complex coefficients: Racah's closed form, Condon-Shortley phase.
  * real basis: Y_{l,m>0} = sqrt2 (-1)^m Re Y_l^m, Y_{l,0} = Y_l^0,
    Y_{l,m<0} = sqrt2 (-1)^m Im Y_l^{|m|}.
  * sign of a real path: the whole path is flipped so that its first non-zero
    entry in lexicographic (M, m1, m2) order is positive.
  * path order: paths are sorted (stably) by the position of their output
    irrep (L,p) in the requested output list; the default list is
    0e,0o,1o,1e,2e,2o,3o,3e,... (natural parity first); ties keep the order
    (input irrep index, l2).

Everything is computed in exact rational arithmetic up to the final square
roots, then in float64.
"""
from __future__ import annotations

import math
import re
from dataclasses import dataclass
from fractions import Fraction
from functools import lru_cache

import numpy as np


# --------------------------------------------------------------------------
# complex SU(2) Clebsch-Gordan coefficients, Racah's closed form
# --------------------------------------------------------------------------
def _f(n: int) -> int:
    return math.factorial(n)


@lru_cache(maxsize=None)
def su2_cg(l1: int, m1: int, l2: int, m2: int, L: int, M: int) -> float:
    """<l1 m1 l2 m2 | L M> for integer degrees (Racah formula, CS phase)."""
    if M != m1 + m2 or not (abs(l1 - l2) <= L <= l1 + l2):
        return 0.0
    if abs(m1) > l1 or abs(m2) > l2 or abs(M) > L:
        return 0.0
    pref2 = Fraction(
        (2 * L + 1) * _f(L + l1 - l2) * _f(L - l1 + l2) * _f(l1 + l2 - L),
        _f(l1 + l2 + L + 1),
    )
    pref2 *= _f(L + M) * _f(L - M) * _f(l1 - m1) * _f(l1 + m1) * _f(l2 - m2) * _f(l2 + m2)
    total = Fraction(0)
    for k in range(0, l1 + l2 - L + 1):
        args = (
            k,
            l1 + l2 - L - k,
            l1 - m1 - k,
            l2 + m2 - k,
            L - l2 + m1 + k,
            L - l1 - m2 + k,
        )
        if min(args) < 0:
            continue
        den = 1
        for a in args:
            den *= _f(a)
        total += Fraction((-1) ** k, den)
    # sign(total) * sqrt(pref2 * total^2), evaluated in float64
    val = math.sqrt(float(pref2 * total * total))
    return val if total >= 0 else -val


def complex_cg_block(l1: int, l2: int, L: int) -> np.ndarray:
    """Array [2L+1, 2l1+1, 2l2+1] of <l1 m1 l2 m2|L M>, indices m+l."""
    out = np.zeros((2 * L + 1, 2 * l1 + 1, 2 * l2 + 1))
    for M in range(-L, L + 1):
        for m1 in range(-l1, l1 + 1):
            m2 = M - m1
            if abs(m2) <= l2:
                out[M + L, m1 + l1, m2 + l2] = su2_cg(l1, m1, l2, m2, L, M)
    return out


# --------------------------------------------------------------------------
# complex -> real change of basis
# --------------------------------------------------------------------------
def real_basis(l: int) -> np.ndarray:
    """Unitary U_l with  Y_real[m] = sum_m' U_l[m, m'] Y_complex[m']  (m+l indexing)."""
    U = np.zeros((2 * l + 1, 2 * l + 1), dtype=complex)
    r = 1.0 / math.sqrt(2.0)
    U[l, l] = 1.0
    for m in range(1, l + 1):
        s = (-1) ** m
        # m > 0 :  sqrt2 (-1)^m Re Y_l^m = ((-1)^m Y_l^m + Y_l^{-m}) / sqrt2
        U[l + m, l + m] = s * r
        U[l + m, l - m] = r
        # m < 0 :  sqrt2 (-1)^m Im Y_l^{|m|} = ((-1)^m Y_l^{|m|} - Y_l^{-|m|}) / (i sqrt2)
        U[l - m, l + m] = -1j * s * r
        U[l - m, l - m] = 1j * r
    return U


@lru_cache(maxsize=None)
def _real_cg_block_cached(l1: int, l2: int, L: int) -> tuple:
    C = complex_cg_block(l1, l2, L).astype(complex)
    U1, U2, UL = real_basis(l1), real_basis(l2), real_basis(L)
    # z_real = U_L CG (U_1^H x_real) (U_2^H y_real)
    T = np.einsum("Mk,kab,ia,jb->Mij", UL, C, U1.conj(), U2.conj())
    if (l1 + l2 + L) % 2 == 0:
        R, rest = T.real, T.imag
    else:
        R, rest = T.imag, T.real
    assert np.abs(rest).max() < 1e-14, "real CG block is neither real nor imaginary"
    R = np.where(np.abs(R) < 1e-14, 0.0, R)
    nz = np.flatnonzero(R.ravel())
    if nz.size and R.ravel()[nz[0]] < 0:
        R = -R
    R = R + 0.0  # normalise -0.0
    return R.shape, R.tobytes()


def real_cg_block(l1: int, l2: int, L: int) -> np.ndarray:
    """Real coupling tensor T[M, m1, m2] of one path, canonical sign, unitary norm."""
    shape, buf = _real_cg_block_cached(l1, l2, L)
    return np.frombuffer(buf, dtype=np.float64).reshape(shape).copy()


# --------------------------------------------------------------------------
# irreps descriptors and path enumeration
# --------------------------------------------------------------------------
_IRREP = re.compile(r"^\s*(?:(\d+)\s*x\s*)?(\d+)([eo])\s*$")


def parse_irreps(text: str) -> list[tuple[int, int, int]]:
    """'128x0e+128x1o' -> [(128,0,+1),(128,1,-1)]; parity +1 = even."""
    out = []
    for tok in text.split("+"):
        m = _IRREP.match(tok)
        if not m:
            raise ValueError(f"bad irrep token {tok!r}")
        mul = int(m.group(1)) if m.group(1) else 1
        out.append((mul, int(m.group(2)), 1 if m.group(3) == "e" else -1))
    return out


def default_output_order(out_lmax: int) -> list[tuple[int, int]]:
    order = []
    for L in range(out_lmax + 1):
        nat = 1 if L % 2 == 0 else -1
        order += [(L, nat), (L, -nat)]
    return order


@dataclass(frozen=True)
class Path:
    k: int          # block index = weight block = i3 value
    in_index: int   # which input irrep
    l1: int
    p1: int
    l2: int
    L: int
    p: int
    x_off: int      # first i1 coordinate
    y_off: int      # first i2 coordinate (= l2^2)
    out_off: int    # first i0 coordinate


def enumerate_paths(irreps_in: str, sh_lmax: int, irreps_out: str | None = None,
                    out_lmax: int | None = None) -> tuple[int, int, int, int, list[Path]]:
    """Returns (N_q, d, d', D, paths)."""
    ins = parse_irreps(irreps_in)
    muls = {m for m, _, _ in ins}
    if len(muls) != 1:
        raise ValueError("input multiplicity must be uniform")
    nq = muls.pop()
    if irreps_out is None:
        if out_lmax is None:
            out_lmax = max(l for _, l, _ in ins) + sh_lmax
        wanted = default_output_order(out_lmax)
    else:
        wanted = [(l, p) for _, l, p in parse_irreps(irreps_out)]
    raw = []
    x_off = 0
    for idx, (_, l1, p1) in enumerate(ins):
        for l2 in range(sh_lmax + 1):
            p2 = 1 if l2 % 2 == 0 else -1
            for L in range(abs(l1 - l2), l1 + l2 + 1):
                p = p1 * p2
                if (L, p) in wanted:
                    raw.append((wanted.index((L, p)), idx, l2, l1, p1, L, p, x_off))
        x_off += 2 * l1 + 1
    d = x_off
    raw.sort(key=lambda t: (t[0], t[1], t[2]))
    paths, off = [], 0
    for k, (_, idx, l2, l1, p1, L, p, xo) in enumerate(raw):
        paths.append(Path(k, idx, l1, p1, l2, L, p, xo, l2 * l2, off))
        off += 2 * L + 1
    return nq, d, (sh_lmax + 1) ** 2, off, paths


def dense_coupling(irreps_in: str, sh_lmax: int, irreps_out: str | None = None,
                   out_lmax: int | None = None):
    """Dense C[D, d, d'] (float64), i3[D] (int32) and the path list."""
    nq, d, dp, D, paths = enumerate_paths(irreps_in, sh_lmax, irreps_out, out_lmax)
    C = np.zeros((D, d, dp))
    i3 = np.zeros(D, dtype=np.int32)
    for pth in paths:
        blk = real_cg_block(pth.l1, pth.l2, pth.L)
        C[pth.out_off:pth.out_off + 2 * pth.L + 1,
          pth.x_off:pth.x_off + 2 * pth.l1 + 1,
          pth.y_off:pth.y_off + 2 * pth.l2 + 1] = blk
        i3[pth.out_off:pth.out_off + 2 * pth.L + 1] = pth.k
    return C, i3, paths, nq
