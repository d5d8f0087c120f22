"""Oracle: convolution / tensor-product entry points (test infrastructure only).

conv_fwd / conv_bwd call the plain C loops of conv_naive.c (float64 sums of the
paper's message-passing-convolution and message-passing-backward equations).
tp_fwd / tp_bwd are the tensor-product formula followed by the edge-scalar
weighting ("Mathematical operations") and the tensor-product backward rule
("Differentiation"), written as dense numpy contractions in float64.

The C file is compiled on first use with gcc (and by the repository build
step); nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

from . import cg

_HERE = Path(__file__).resolve().parent
_SO = _HERE / "libe3j_oracle.so"
_SRC = _HERE / "conv_naive.c"
_lib = None


def build(force: bool = False) -> Path:
    """Compile conv_naive.c into libe3j_oracle.so next to it."""
    if force or not _SO.exists() or _SO.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _SO.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", str(tmp), str(_SRC)])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_SO))
        i64, i32 = ctypes.c_int64, ctypes.c_int
        ptr = ctypes.c_void_p
        lib.e3j_oracle_conv_fwd.argtypes = [i64, i64, i32, i32, i32, i32, i32] + [ptr] * 8
        lib.e3j_oracle_conv_fwd.restype = i32
        lib.e3j_oracle_conv_bwd.argtypes = [i64, i64, i32, i32, i32, i32, i32] + [ptr] * 11
        lib.e3j_oracle_conv_bwd.restype = i32
        lib.e3j_oracle_conv_fwd_sd.argtypes = lib.e3j_oracle_conv_fwd.argtypes
        lib.e3j_oracle_conv_fwd_sd.restype = i32
        lib.e3j_oracle_conv_bwd_sd.argtypes = lib.e3j_oracle_conv_bwd.argtypes
        lib.e3j_oracle_conv_bwd_sd.restype = i32
        lib.e3j_oracle_threads.restype = i32
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the C loops will use."""
    return int(_load().e3j_oracle_threads())


class Coupling:
    """Dense coupling tensor and shapes of one (irreps_in, sh_lmax, irreps_out) signature."""

    def __init__(self, irreps_in: str, sh_lmax: int, irreps_out: str | None = None,
                 out_lmax: int | None = None):
        self.C, self.i3, self.paths, self.nq = cg.dense_coupling(irreps_in, sh_lmax, irreps_out, out_lmax)
        self.D, self.d, self.dp = self.C.shape
        self.P = len(self.paths)
        self.C = np.ascontiguousarray(self.C)
        self.i3 = np.ascontiguousarray(self.i3, dtype=np.int32)

    @property
    def nnz(self) -> int:
        return int(np.count_nonzero(self.C))


def _f32(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _i32(a, n):
    a = np.ascontiguousarray(a, dtype=np.int32)
    assert a.shape == (n,)
    return a


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def conv_fwd(cp: Coupling, x, y, s, senders, receivers) -> np.ndarray:
    """m[N, D, N_q] in float64."""
    n, e = x.shape[0], len(senders)
    x = _f32(x, (n, cp.d, cp.nq)); y = _f32(y, (e, cp.dp)); s = _f32(s, (e, cp.P, cp.nq))
    senders, receivers = _i32(senders, e), _i32(receivers, e)
    out = np.zeros((n, cp.D, cp.nq))
    rc = _load().e3j_oracle_conv_fwd(n, e, cp.d, cp.dp, cp.P, cp.D, cp.nq, _p(cp.C), _p(cp.i3),
                                     _p(x), _p(y), _p(s), _p(senders), _p(receivers), _p(out))
    if rc != 0:
        raise ValueError("oracle: receivers not sorted or index out of range")
    return out


def conv_bwd(cp: Coupling, x, y, s, senders, receivers, dm):
    """(dx[N,d,N_q], dy[E,d'], ds[E,P,N_q]) in float64."""
    n, e = x.shape[0], len(senders)
    x = _f32(x, (n, cp.d, cp.nq)); y = _f32(y, (e, cp.dp)); s = _f32(s, (e, cp.P, cp.nq))
    dm = _f32(dm, (n, cp.D, cp.nq))
    senders, receivers = _i32(senders, e), _i32(receivers, e)
    dx = np.zeros((n, cp.d, cp.nq)); dy = np.zeros((e, cp.dp)); ds = np.zeros((e, cp.P, cp.nq))
    rc = _load().e3j_oracle_conv_bwd(n, e, cp.d, cp.dp, cp.P, cp.D, cp.nq, _p(cp.C), _p(cp.i3),
                                     _p(x), _p(y), _p(s), _p(senders), _p(receivers), _p(dm),
                                     _p(dx), _p(dy), _p(ds))
    if rc != 0:
        raise ValueError("oracle: receivers not sorted or index out of range")
    return dx, dy, ds


def tp_fwd(cp: Coupling, x1, x2, w) -> np.ndarray:
    """z[r,i0,q] = w[r,i3(i0),q] * sum_{i1,i2} C[i0,i1,i2] x1[r,i1,q] x2[r,i2]  (float64)."""
    x1 = np.asarray(x1, dtype=np.float64); x2 = np.asarray(x2, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    z = np.einsum("ijk,rjq,rk->riq", cp.C, x1, x2)
    return z * w[:, cp.i3, :]


def tp_bwd(cp: Coupling, x1, x2, w, dz):
    """(dx1, dx2, dw) of tp_fwd for the output cotangent dz, float64."""
    x1 = np.asarray(x1, dtype=np.float64); x2 = np.asarray(x2, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64); dz = np.asarray(dz, dtype=np.float64)
    wdz = dz * w[:, cp.i3, :]
    dx1 = np.einsum("ijk,rk,riq->rjq", cp.C, x2, wdz)
    dx2 = np.einsum("ijk,rjq,riq->rk", cp.C, x1, wdz)
    z = np.einsum("ijk,rjq,rk->riq", cp.C, x1, x2)
    dw = np.zeros_like(w)
    np.add.at(dw, (slice(None), cp.i3, slice(None)), z * dz)
    return dx1, dx2, dw


# ---------------------------------------------------------------------------------------------
# Padded edge lists.  The paper keeps the neighbour list of its molecular-dynamics runs at a fixed
# padded size and flags the padding edges, without saying how; the reading taken here: an edge
# whose receiver id is >= the number of nodes is padding.  A padding edge takes no part in any
# sum, nothing of it is looked at, and its rows of the edge-local cotangents are zero.
def conv_fwd_padded(cp: Coupling, x, y, s, senders, receivers) -> np.ndarray:
    """The forward sum over the real edges only."""
    real = np.asarray(receivers) < x.shape[0]
    return conv_fwd(cp, x, np.asarray(y)[real], np.asarray(s)[real], np.asarray(senders)[real],
                    np.asarray(receivers)[real])


def conv_bwd_padded(cp: Coupling, x, y, s, senders, receivers, dm):
    """(dx, dy, ds): dx from the real edges; dy, ds rows of padding edges are zero."""
    real = np.asarray(receivers) < x.shape[0]
    dx, dy_r, ds_r = conv_bwd(cp, x, np.asarray(y)[real], np.asarray(s)[real], np.asarray(senders)[real],
                              np.asarray(receivers)[real], dm)
    e = len(receivers)
    dy = np.zeros((e, cp.dp)); ds = np.zeros((e, cp.P, cp.nq))
    dy[real] = dy_r; ds[real] = ds_r
    return dx, dy, ds


# ---------------------------------------------------------------------------------------------
# Collapsed output multiplicities.  The paper evaluates its kernels also with a coefficient set
# (appendix on the comparison with the SO(2) convolution) in which the copies of one irreducible
# output space produced by different paths are added: every path that lands on the same
# (L, parity) adds into one shared output block.  Written out here from
# the uncollapsed definition: out_c = R out, with R the 0/1 matrix that maps row M of every
# path's block to row M of the shared block of its (L, parity); the backward is the chain rule
# through that sum (dm = R^T dm_c).  Blocks are ordered as their first path is.
def collapse_matrix(cp: Coupling) -> np.ndarray:
    """(R [D_collapsed, D], block offset of every path)."""
    block_off, offsets, d_c = {}, [], 0
    for p in cp.paths:
        key = (p.L, p.p)
        if key not in block_off:
            block_off[key] = d_c
            d_c += 2 * p.L + 1
        offsets.append(block_off[key])
    R = np.zeros((d_c, cp.D))
    for p, off in zip(cp.paths, offsets):
        for m in range(2 * p.L + 1):
            R[off + m, p.out_off + m] = 1.0
    return R, offsets


def conv_fwd_collapsed(cp: Coupling, x, y, s, senders, receivers) -> np.ndarray:
    R, _ = collapse_matrix(cp)
    return np.einsum("ci,niq->ncq", R, conv_fwd(cp, x, y, s, senders, receivers))


def conv_bwd_collapsed(cp: Coupling, x, y, s, senders, receivers, dm_c):
    R, _ = collapse_matrix(cp)
    dm = np.einsum("ci,ncq->niq", R, np.asarray(dm_c, dtype=np.float64)).astype(np.float32)
    return conv_bwd(cp, x, y, s, senders, receivers, dm)


# ---------------------------------------------------------------------------------------------
# Double backward (paper, "Differentiation", message-passing double backward): with (ux, uy, us) the
# cotangents of the backward's results (dx, dy, ds), the cotangents of the backward's inputs are
#   d(dm) = conv(ux, y, s) + conv(x, uy, s) + conv(x, y, us)
#   dx = dx[conv_bwd(x, uy, s, dm)] + dx[conv_bwd(x, y, us, dm)]         and cyclically for y and s.
def conv_bwd_bwd(cp: Coupling, x, y, s, senders, receivers, dm, ux, uy, us):
    """(g_dm, g_x, g_y, g_s) in float64."""
    g_dm = (conv_fwd(cp, ux, y, s, senders, receivers) + conv_fwd(cp, x, uy, s, senders, receivers) +
            conv_fwd(cp, x, y, us, senders, receivers))
    _, y_from_x, s_from_x = conv_bwd(cp, ux, y, s, senders, receivers, dm)
    x_from_y, _, s_from_y = conv_bwd(cp, x, uy, s, senders, receivers, dm)
    x_from_s, y_from_s, _ = conv_bwd(cp, x, y, us, senders, receivers, dm)
    return g_dm, x_from_y + x_from_s, y_from_x + y_from_s, s_from_x + s_from_y


# ---------------------------------------------------------------------------------------------
# Edge scalars from the radial network (paper, "Key operations in scope": the scalars s_ab of the
# message-passing layer depend on the interatomic distance through a radial-basis embedding followed by a
# multi-layer perceptron, and such scalar mixings are named as candidates for fusion into the message
# passing).  What is taken inside the convolution here is the perceptron's last, purely linear layer:
#   s[e, k, q] = sum_j h[e, j] * W[j, k * N_q + q]
# with h [E, H] the last hidden activations of the edge and W [H, P * N_q] the layer's matrix (no bias;
# the paper does not state the layer sizes, H is free).  The product is formed in float64 and is never
# rounded to float32; the convolution is then the defining sum.  Backward: the chain rule through the
# product, dh = ds W^T and dW = h^T ds, with ds the edge-scalar cotangent of the convolution.
def radial_weights(h, W, n_paths: int, nq: int) -> np.ndarray:
    """s[E, P, N_q] = h W in float64."""
    h = np.asarray(h, dtype=np.float64); W = np.asarray(W, dtype=np.float64)
    assert h.ndim == 2 and W.shape == (h.shape[1], n_paths * nq), (h.shape, W.shape)
    return (h @ W).reshape(h.shape[0], n_paths, nq)


def _conv_fwd_sd(cp: Coupling, x, y, s, senders, receivers) -> np.ndarray:
    n, e = x.shape[0], len(senders)
    x = _f32(x, (n, cp.d, cp.nq)); y = _f32(y, (e, cp.dp))
    s = np.ascontiguousarray(s, dtype=np.float64); assert s.shape == (e, cp.P, cp.nq)
    senders, receivers = _i32(senders, e), _i32(receivers, e)
    out = np.zeros((n, cp.D, cp.nq))
    rc = _load().e3j_oracle_conv_fwd_sd(n, e, cp.d, cp.dp, cp.P, cp.D, cp.nq, _p(cp.C), _p(cp.i3),
                                        _p(x), _p(y), _p(s), _p(senders), _p(receivers), _p(out))
    if rc != 0:
        raise ValueError("oracle: receivers not sorted or index out of range")
    return out


def _conv_bwd_sd(cp: Coupling, x, y, s, senders, receivers, dm):
    n, e = x.shape[0], len(senders)
    x = _f32(x, (n, cp.d, cp.nq)); y = _f32(y, (e, cp.dp)); dm = _f32(dm, (n, cp.D, cp.nq))
    s = np.ascontiguousarray(s, dtype=np.float64); assert s.shape == (e, cp.P, cp.nq)
    senders, receivers = _i32(senders, e), _i32(receivers, e)
    dx = np.zeros((n, cp.d, cp.nq)); dy = np.zeros((e, cp.dp)); ds = np.zeros((e, cp.P, cp.nq))
    rc = _load().e3j_oracle_conv_bwd_sd(n, e, cp.d, cp.dp, cp.P, cp.D, cp.nq, _p(cp.C), _p(cp.i3),
                                        _p(x), _p(y), _p(s), _p(senders), _p(receivers), _p(dm),
                                        _p(dx), _p(dy), _p(ds))
    if rc != 0:
        raise ValueError("oracle: receivers not sorted or index out of range")
    return dx, dy, ds


def conv_radial_fwd(cp: Coupling, x, y, h, W, senders, receivers) -> np.ndarray:
    """m[N, D, N_q] with the edge scalars s = h W formed in float64."""
    return _conv_fwd_sd(cp, x, y, radial_weights(h, W, cp.P, cp.nq), senders, receivers)


def conv_radial_bwd(cp: Coupling, x, y, h, W, senders, receivers, dm):
    """(dx[N,d,N_q], dy[E,d'], dh[E,H], dW[H,P*N_q]) in float64."""
    s = radial_weights(h, W, cp.P, cp.nq)
    dx, dy, ds = _conv_bwd_sd(cp, x, y, s, senders, receivers, dm)
    ds2 = ds.reshape(ds.shape[0], cp.P * cp.nq)
    dh = ds2 @ np.asarray(W, dtype=np.float64).T
    dW = np.asarray(h, dtype=np.float64).T @ ds2
    return dx, dy, dh, dW


# ---------------------------------------------------------------------------------------------
# Harmonics taken from the edge vectors.  The paper lists the harmonic embedding Y(r_ab / |r_ab|) of the
# edge direction among the operations in scope and feeds it to the convolution as y; here the two are
# composed: y is evaluated in float64 from the float32 vectors and rounded to float32, the precision it has
# as an input of the convolution, and the backward continues the chain rule into the vectors.
def _sh_lmax(cp: Coupling) -> int:
    lmax = int(round(cp.dp ** 0.5)) - 1
    assert (lmax + 1) ** 2 == cp.dp
    return lmax


def conv_vec_fwd(cp: Coupling, x, vec, s, senders, receivers) -> np.ndarray:
    from . import sh
    vec = np.ascontiguousarray(vec, dtype=np.float32)
    y = sh.real_sh_all_of_vectors(_sh_lmax(cp), vec.astype(np.float64)).astype(np.float32)
    return conv_fwd(cp, x, y, s, senders, receivers)


def conv_vec_bwd(cp: Coupling, x, vec, s, senders, receivers, dm):
    """(dx[N,d,N_q], dvec[E,3], ds[E,P,N_q]) in float64."""
    from . import sh
    vec = np.ascontiguousarray(vec, dtype=np.float32)
    y = sh.real_sh_all_of_vectors(_sh_lmax(cp), vec.astype(np.float64)).astype(np.float32)
    dx, dy, ds = conv_bwd(cp, x, y, s, senders, receivers, dm)
    return dx, sh.real_sh_all_vjp(_sh_lmax(cp), vec.astype(np.float64), dy), ds
