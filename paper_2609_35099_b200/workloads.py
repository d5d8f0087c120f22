"""Seeded synthetic workloads shaped like the paper's benchmarks.

This module only manufactures INPUTS (graphs, feature arrays, weights,
cotangents).  It contains none of the convolution's arithmetic, imports neither
the CUDA binding nor the CPU oracle, and is the one piece both sides share: the
same arrays are handed to the CUDA path and to the oracle.

The shapes follow the paper's unit benchmarks (5 Angstrom cutoff, about 45-50
neighbours per atom, 128 channels, l_max 3; table "Maximal convolution
throughput" and the MACE hyper-parameter table) and the five named
configurations of this repository:

  1  tiny        64 atoms, 6 A periodic cube, 3 A cutoff, 8x0e+8x1o, sh l<=2
  2  water3000   1000 rigid water molecules in a 31.04 A cube, 128x0e+128x1o, sh l<=3
  3  highorder   1500 atoms, 24.64 A cube, 64x(0e+1o+2e+3o), sh l<=3
  4  tp          row-wise tensor product, 128x(0e+1o+2e) (x) (0e+1o+2e+3o)
  5  large       100k atoms, 105 A cube, 10 % of the molecules at twice the density

Spherical harmonics of the edge directions are an *input* of the convolution;
they are evaluated here from written-out Cartesian polynomials (l <= 3,
component normalisation: sum_m Y_lm^2 = 2l+1, components m = -l..l, so that
l = 1 is sqrt(3) (y, z, x)).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

# --------------------------------------------------------------------------
# configuration table
# --------------------------------------------------------------------------
CONFIGS = {
    1: dict(name="tiny", irreps_in="8x0e+8x1o", sh_lmax=2, irreps_out="0e+1o+1e+2e+2o", out_lmax=2, seed=1),
    2: dict(name="water3000", irreps_in="128x0e+128x1o", sh_lmax=3, irreps_out=None, out_lmax=3, seed=2),
    3: dict(name="highorder", irreps_in="64x0e+64x1o+64x2e+64x3o", sh_lmax=3, irreps_out=None, out_lmax=3, seed=3),
    4: dict(name="tp", irreps_in="128x0e+128x1o+128x2e", sh_lmax=3, irreps_out=None, out_lmax=3, seed=4),
    5: dict(name="large", irreps_in="128x0e+128x1o", sh_lmax=3, irreps_out=None, out_lmax=3, seed=5),
}
# config 2 restricted to the natural-parity outputs a MACE layer without
# pseudotensors keeps (secondary, labelled variant)
NATURAL_PARITY_OUT = "0e+1o+2e+3o"


# --------------------------------------------------------------------------
# real spherical harmonics, l <= 3, Cartesian closed forms
# --------------------------------------------------------------------------
def spherical_harmonics(lmax: int, unit: np.ndarray) -> np.ndarray:
    """[n, (lmax+1)^2] float64 component-normalised real harmonics of unit vectors."""
    if not 0 <= lmax <= 3:
        raise ValueError("closed forms are written out for l <= 3 only")
    x, y, z = unit[:, 0], unit[:, 1], unit[:, 2]
    cols = [np.ones_like(x)]
    if lmax >= 1:
        r3 = math.sqrt(3.0)
        cols += [r3 * y, r3 * z, r3 * x]
    if lmax >= 2:
        r15, r5 = math.sqrt(15.0), math.sqrt(5.0)
        cols += [r15 * x * y, r15 * y * z, 0.5 * r5 * (3 * z * z - 1.0), r15 * x * z,
                 0.5 * r15 * (x * x - y * y)]
    if lmax >= 3:
        a, b, c = math.sqrt(35.0 / 8.0), math.sqrt(105.0), math.sqrt(21.0 / 8.0)
        cols += [a * y * (3 * x * x - y * y), b * x * y * z, c * y * (5 * z * z - 1.0),
                 0.5 * math.sqrt(7.0) * (5 * z ** 3 - 3 * z), c * x * (5 * z * z - 1.0),
                 0.5 * b * (x * x - y * y) * z, a * x * (x * x - 3 * y * y)]
    return np.stack(cols, axis=1)


# --------------------------------------------------------------------------
# periodic neighbour lists
# --------------------------------------------------------------------------
def periodic_edges(pos: np.ndarray, box: float, cutoff: float):
    """All ordered pairs (a -> b), a != b, with minimum-image distance < cutoff.

    Returns senders, receivers (int32, sorted by receiver then sender) and the
    edge vectors r_b - r_a (float64).  Needs box > 2 * cutoff.
    """
    from scipy.spatial import cKDTree

    assert box > 2 * cutoff
    p = np.mod(pos, box)
    p[p >= box] = 0.0  # guard against mod returning box itself
    tree = cKDTree(p, boxsize=box)
    pairs = tree.query_pairs(cutoff, output_type="ndarray")
    a = np.concatenate([pairs[:, 0], pairs[:, 1]])
    b = np.concatenate([pairs[:, 1], pairs[:, 0]])
    vec = p[b] - p[a]
    vec -= box * np.round(vec / box)
    r = np.linalg.norm(vec, axis=1)
    keep = (r > 0) & (r < cutoff)
    a, b, vec = a[keep], b[keep], vec[keep]
    order = np.lexsort((a, b))
    return a[order].astype(np.int32), b[order].astype(np.int32), vec[order]


def _random_rotations(rng: np.random.Generator, n: int) -> np.ndarray:
    """n rotation matrices from uniformly distributed unit quaternions."""
    q = rng.standard_normal((n, 4))
    q /= np.linalg.norm(q, axis=1, keepdims=True)
    w, x, y, z = q.T
    return np.stack([
        np.stack([1 - 2 * (y * y + z * z), 2 * (x * y - z * w), 2 * (x * z + y * w)], axis=1),
        np.stack([2 * (x * y + z * w), 1 - 2 * (x * x + z * z), 2 * (y * z - x * w)], axis=1),
        np.stack([2 * (x * z - y * w), 2 * (y * z + x * w), 1 - 2 * (x * x + y * y)], axis=1),
    ], axis=1)


def _water_molecules(rng: np.random.Generator, oxygen: np.ndarray) -> np.ndarray:
    """O,H,H positions for rigid molecules (O-H 0.96 A, H-O-H 104.5 deg), random orientation."""
    n = oxygen.shape[0]
    half = math.radians(104.5) / 2
    h_local = 0.96 * np.array([[math.sin(half), 0.0, math.cos(half)],
                               [-math.sin(half), 0.0, math.cos(half)]])
    R = _random_rotations(rng, n)
    h = oxygen[:, None, :] + np.einsum("nij,kj->nki", R, h_local)
    return np.concatenate([oxygen[:, None, :], h], axis=1).reshape(3 * n, 3)


def water_box(rng: np.random.Generator, grid: int, spacing: float, jitter: float = 0.5):
    """grid^3 water molecules on a jittered cubic lattice; returns positions, box length."""
    g = np.arange(grid)
    ox = np.stack(np.meshgrid(g, g, g, indexing="ij"), axis=-1).reshape(-1, 3) * spacing
    ox = ox + rng.uniform(-jitter, jitter, size=ox.shape)
    return _water_molecules(rng, ox), grid * spacing


def sequential_insertion(rng: np.random.Generator, n: int, box: float, min_sep: float) -> np.ndarray:
    """n points uniform in a periodic cube, rejected while closer than min_sep to an earlier one."""
    cell = max(min_sep, box / 64)
    ncell = int(box // cell)
    cell = box / ncell
    grid: dict[tuple[int, int, int], list[int]] = {}
    pts = np.zeros((n, 3))
    count = 0
    while count < n:
        p = rng.uniform(0, box, size=3)
        c = tuple((p // cell).astype(int) % ncell)
        ok = True
        for dx in (-1, 0, 1):
            for dy in (-1, 0, 1):
                for dz in (-1, 0, 1):
                    for j in grid.get(((c[0] + dx) % ncell, (c[1] + dy) % ncell, (c[2] + dz) % ncell), ()):
                        v = pts[j] - p
                        v -= box * np.round(v / box)
                        if v @ v < min_sep * min_sep:
                            ok = False
        if ok:
            pts[count] = p
            grid.setdefault(c, []).append(count)
            count += 1
    return pts


def sort_by_cell(pos: np.ndarray, box: float, cell: float) -> np.ndarray:
    """Reorder points by the index of the cubic cell they fall in (spatial locality)."""
    n = int(math.ceil(box / cell))
    c = np.minimum((np.mod(pos, box) // cell).astype(np.int64), n - 1)
    key = (c[:, 0] * n + c[:, 1]) * n + c[:, 2]
    return pos[np.argsort(key, kind="stable")]


def skewed_water(rng: np.random.Generator, n_atoms: int, box: float, dense_frac: float = 0.10):
    """Water molecules with dense_frac of them in a sub-cube at twice the base density."""
    n_mol = (n_atoms + 2) // 3
    n_dense = int(round(dense_frac * n_mol))
    n_base = n_mol - n_dense
    # volumes: V_sub * 2 rho + (V - V_sub) * rho = n_mol  and  V_sub * 2 rho = n_dense
    vol = box ** 3
    rho = (n_mol - n_dense / 2.0) / vol
    sub = (n_dense / (2 * rho)) ** (1.0 / 3.0)

    def lattice(count: int, lo: float, hi: float, exclude=None):
        span = hi - lo
        m = 1
        while True:
            g = (np.arange(m) + 0.5) * (span / m) + lo
            pts = np.stack(np.meshgrid(g, g, g, indexing="ij"), axis=-1).reshape(-1, 3)
            if exclude is not None:
                inside = np.all((pts >= exclude[0]) & (pts < exclude[1]), axis=1)
                pts = pts[~inside]
            if pts.shape[0] >= count:
                sel = np.sort(rng.choice(pts.shape[0], size=count, replace=False))
                return pts[sel], span / m
            m += 1

    dense, hd = lattice(n_dense, 0.0, sub)
    base, hb = lattice(n_base, 0.0, box, exclude=(0.0, sub))
    dense = dense + rng.uniform(-0.2 * hd, 0.2 * hd, size=dense.shape)
    base = base + rng.uniform(-0.2 * hb, 0.2 * hb, size=base.shape)
    ox = np.concatenate([dense, base], axis=0)
    atoms = _water_molecules(rng, ox)[:n_atoms]
    return atoms


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------
@dataclass
class Workload:
    config: int
    name: str
    irreps_in: str
    sh_lmax: int
    irreps_out: str | None
    out_lmax: int
    n_nodes: int
    n_edges: int
    senders: np.ndarray | None = None      # int32 [E]
    receivers: np.ndarray | None = None    # int32 [E], non-decreasing
    vectors: np.ndarray | None = None      # float64 [E,3]  r_b - r_a
    positions: np.ndarray | None = None
    box: float = 0.0
    cutoff: float = 0.0
    meta: dict = field(default_factory=dict)


def feature_dims(irreps_in: str, sh_lmax: int):
    """(N_q, d, d') from the descriptor strings; no path logic here."""
    mul, d = None, 0
    for tok in irreps_in.split("+"):
        m, ir = tok.strip().split("x")
        mul = int(m)
        d += 2 * int(ir[:-1]) + 1
    return mul, d, (sh_lmax + 1) ** 2


def make_graph(config: int, n_atoms: int | None = None) -> Workload:
    """Graph and descriptors of one configuration (no feature arrays yet)."""
    c = CONFIGS[config]
    rng = np.random.Generator(np.random.PCG64(c["seed"]))
    common = dict(config=config, name=c["name"], irreps_in=c["irreps_in"], sh_lmax=c["sh_lmax"],
                  irreps_out=c["irreps_out"], out_lmax=c["out_lmax"])
    if config == 1:
        n = n_atoms or 64
        pos, box, cut = rng.uniform(0, 6.0, size=(n, 3)), 6.0, 3.0
        # 6 A box with a 3 A cutoff: box == 2*cutoff, so enumerate images directly
        a, b = np.meshgrid(np.arange(n), np.arange(n), indexing="ij")
        a, b = a.ravel(), b.ravel()
        vec = pos[b] - pos[a]
        vec -= box * np.round(vec / box)
        r = np.linalg.norm(vec, axis=1)
        keep = (a != b) & (r > 0) & (r < cut)
        a, b, vec = a[keep], b[keep], vec[keep]
        order = np.lexsort((a, b))
        snd, rcv, vec = a[order].astype(np.int32), b[order].astype(np.int32), vec[order]
    elif config == 2:
        grid = 10 if n_atoms is None else max(2, round((n_atoms / 3) ** (1 / 3)))
        if grid * 3.104 <= 10.0:
            raise ValueError("box too small for the 5 A cutoff")
        pos, box = water_box(rng, grid, 3.104)
        cut = 5.0
        snd, rcv, vec = periodic_edges(pos, box, cut)
    elif config == 3:
        n = n_atoms or 1500
        box = max(24.64 * (n / 1500.0) ** (1 / 3), 10.5)  # keep box > 2 * cutoff on reduced sizes
        cut = 5.0
        pos = sort_by_cell(sequential_insertion(rng, n, box, 0.8), box, 4.0)
        snd, rcv, vec = periodic_edges(pos, box, cut)
    elif config == 5:
        n = n_atoms or 100_000
        box = max(105.0 * (n / 100_000.0) ** (1 / 3), 10.5)
        cut = 5.0
        pos = sort_by_cell(skewed_water(rng, n, box), box, 5.0)
        snd, rcv, vec = periodic_edges(pos, box, cut)
    else:
        raise ValueError("config 4 has no graph; use make_tp_rows")
    return Workload(n_nodes=pos.shape[0], n_edges=len(snd), senders=snd, receivers=rcv, vectors=vec,
                    positions=pos, box=box, cutoff=cut, **common)


def edge_harmonics(wl: Workload) -> np.ndarray:
    """y[E, d'] float32: harmonics of the unit edge vectors."""
    unit = wl.vectors / np.linalg.norm(wl.vectors, axis=1, keepdims=True)
    return spherical_harmonics(wl.sh_lmax, unit).astype(np.float32)


def make_features(wl: Workload, n_paths: int, n_out: int, with_weights: bool = True):
    """x, y, (w), grad_out as float32 arrays, N(0,1), drawn in this fixed order."""
    c = CONFIGS[wl.config]
    rng = np.random.Generator(np.random.PCG64([c["seed"], 1]))
    nq, d, dp = feature_dims(wl.irreps_in, wl.sh_lmax)
    x = rng.standard_normal((wl.n_nodes, d, nq), dtype=np.float32)
    grad_out = rng.standard_normal((wl.n_nodes, n_out, nq), dtype=np.float32)
    y = edge_harmonics(wl)
    w = rng.standard_normal((wl.n_edges, n_paths, nq), dtype=np.float32) if with_weights else None
    return x, y, w, grad_out


def make_radial(wl: Workload, n_paths: int, hidden: int = 64):
    """Stand-ins for the radial network's last layer: hidden activations h[E, hidden] ~ N(0,1) and the layer
    matrix W[hidden, P * N_q] ~ N(0, 1/hidden), float32 (so that h W has the unit scale of the stand-in weights
    of make_features).  The paper gives num_rbf = 8 and no layer sizes; 64 is the usual width of MACE's radial
    perceptron."""
    c = CONFIGS[wl.config]
    rng = np.random.Generator(np.random.PCG64([c["seed"], 2]))
    nq, _, _ = feature_dims(wl.irreps_in, wl.sh_lmax)
    h = rng.standard_normal((wl.n_edges, hidden), dtype=np.float32)
    W = rng.standard_normal((hidden, n_paths * nq), dtype=np.float32) * np.float32(1.0 / np.sqrt(hidden))
    return h, W


def make_tp_rows(rows: int, n_paths: int, n_out: int, seed: int = 4):
    """Config 4: x1[B,9,128], x2[B,16], w[B,P,128], grad_out[B,D,128], N(0,1) float32."""
    c = CONFIGS[4]
    nq, d, dp = feature_dims(c["irreps_in"], c["sh_lmax"])
    rng = np.random.Generator(np.random.PCG64([seed, 1]))
    x1 = rng.standard_normal((rows, d, nq), dtype=np.float32)
    x2 = rng.standard_normal((rows, dp), dtype=np.float32)
    w = rng.standard_normal((rows, n_paths, nq), dtype=np.float32)
    g = rng.standard_normal((rows, n_out, nq), dtype=np.float32)
    return x1, x2, w, g


def shard_receivers(wl_rowptr: np.ndarray, rank: int, world: int):
    """Contiguous receiver range [lo, hi) of this rank, balanced by edge count.

    Every edge-local tensor and every output row lives with its receiver, so a
    rank's shard is the rows lo..hi-1 and the edges rowptr[lo]..rowptr[hi]-1.
    """
    e_total = int(wl_rowptr[-1])
    n = len(wl_rowptr) - 1
    cuts = [int(np.searchsorted(wl_rowptr, (e_total * r) // world, side="left")) for r in range(world + 1)]
    cuts[0], cuts[-1] = 0, n
    cuts = [min(max(c, 0), n) for c in cuts]
    for i in range(1, world + 1):
        cuts[i] = max(cuts[i], cuts[i - 1])
    return cuts[rank], cuts[rank + 1]
