"""Shared helpers of the GPU parity tests: build a seeded case, run the oracle, compare per irrep block."""
from __future__ import annotations

import numpy as np

TOL = 1e-5  # max abs error <= TOL * max|oracle| per irrep block (fp32 kernel vs fp64 oracle)


def blocks_of_paths(paths, kind):
    """Coordinate ranges of the irreducible blocks of each tensor kind."""
    if kind == "out":
        return [(p.out_off, p.out_off + 2 * p.L + 1) for p in paths]
    if kind == "w":
        return [(p.k, p.k + 1) for p in paths]
    if kind == "x":
        seen = {}
        for p in paths:
            seen[p.x_off] = (p.x_off, p.x_off + 2 * p.l1 + 1)
        return sorted(seen.values())
    if kind == "sh":
        seen = {}
        for p in paths:
            seen[p.y_off] = (p.y_off, p.y_off + 2 * p.l2 + 1)
        return sorted(seen.values())
    raise ValueError(kind)


def assert_blockwise_close(got, want, blocks, axis=1, tol=TOL, what=""):
    """got: float32 array from the GPU, want: float64 oracle array; blocks along `axis`."""
    got = np.asarray(got, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), what
    worst = 0.0
    for lo, hi in blocks:
        sl = [slice(None)] * want.ndim
        sl[axis] = slice(lo, hi)
        g, w = got[tuple(sl)], want[tuple(sl)]
        if w.size == 0:
            continue
        scale = np.abs(w).max()
        err = np.abs(g - w).max()
        if scale == 0.0:
            assert err == 0.0, f"{what} block {lo}:{hi}: oracle is zero but got {err}"
            continue
        worst = max(worst, err / scale)
        assert err <= tol * scale, f"{what} block {lo}:{hi}: err {err:.3e} > {tol} * {scale:.3e}"
    return worst
