#!/usr/bin/env python
"""Generator of the signature-specialised kernel sources under csrc/fast/.

    python paper_2609_35099_b200/csrc/gen_fast.py [--check]

For every entry of fast/signatures.json this script asks the library's own plan builder
(e3j_plan_create / e3j_plan_records of an already built libe3j.so) for the coefficient records of
that signature and writes fast/sig_<name>.cu: a struct of compile-time constants, the record
tables, and fully unrolled per-edge bodies in which every (i0,i1) pair is a straight-line FMA on
registers (the counterpart of the paper's trace-time specialisation of the coefficient loop).
fast/registry_entries.inc lists the generated entries.  The generated files are committed, so a
clean checkout builds without running this script; --check verifies that they are current.
"""
from __future__ import annotations

import argparse
import json
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
sys.path.insert(0, str(HERE.parent.parent))


def load_records(sig):
    import paper_2609_35099_b200 as e3j
    flags = e3j.E3J_PLAN_GENERIC_ONLY | (e3j.E3J_PLAN_COLLAPSE_OUTPUTS if sig.get("collapse") else 0)
    plan = e3j.e3j_plan_create(sig["irreps_in"], sig["sh_lmax"], sig.get("irreps_out"),
                               sig.get("out_lmax", -1), flags)
    info = e3j.e3j_plan_info(plan)
    paths = e3j.e3j_plan_paths(plan)
    i0, i1, i2, i3, val = e3j.e3j_plan_records(plan)
    recs = [(int(a), int(b), int(c), int(k), float(v)) for a, b, c, k, v in zip(i0, i1, i2, i3, val)]
    signature = e3j.e3j_plan_signature(plan)
    return info, paths, recs, signature


def partition_rows(costs, n_groups, weights=None):
    """Contiguous partition of rows into n_groups minimising the largest group cost (DP); weights[g] scales
    the cost of group g (a group whose warp shares its scheduler with a producer warp should get less)."""
    n = len(costs)
    n_groups = min(n_groups, n)
    weights = list(weights or []) + [1.0] * n_groups
    pre = [0]
    for c in costs:
        pre.append(pre[-1] + c)
    INF = float("inf")
    best = [[INF] * (n + 1) for _ in range(n_groups + 1)]
    cut = [[0] * (n + 1) for _ in range(n_groups + 1)]
    best[0][0] = 0
    for g in range(1, n_groups + 1):
        for j in range(g, n + 1):
            for i in range(g - 1, j):
                v = max(best[g - 1][i], (pre[j] - pre[i]) * weights[g - 1])
                if v < best[g][j]:
                    best[g][j], cut[g][j] = v, i
    bounds = [n]
    j = n
    for g in range(n_groups, 0, -1):
        j = cut[g][j]
        bounds.append(j)
    return list(reversed(bounds))


def fmt_float(v: float) -> str:
    """Shortest decimal literal that round-trips the float32 value."""
    import numpy as np
    f = float(np.float32(v))
    s = f"{f:.9g}"
    if "." not in s and "e" not in s:
        s += ".0"
    return s + "f"


def auto_params(sig, info):
    """Tile parameters for a signature that gives none ("auto": 1, or an overlay entry): channels per lane from the
    channel count, row groups from the number of coefficient pairs, tile sizes from what fits in shared memory
    (the formulas of FwdSmem / BwdSmem / Bwd1Smem) and CTAs per SM from the registers the bodies need.  The
    hand-tuned entries of signatures.json were found by measurement; these are the starting point such a search
    would begin from."""
    NQ, DIN, DSH, P, D = info["n_channels"], info["d_in"], info["d_sh"], info["n_paths"], info["d_out"]
    apad = info["n_pairs"] + 16
    if NQ % 32:
        raise ValueError("generated kernels need a multiple of 32 channels")
    V = 4 if NQ % 128 == 0 else 2 if NQ % 64 == 0 else 1
    CH = NQ // (32 * V)
    smem = 227 * 1024
    up = lambda v, a: (v + a - 1) // a * a
    need = {4: 168, 2: 104, 1: 72}[V]
    out = {"V": V, "FW": 4 if info["n_pairs"] <= 300 else 2, "FS": 2, "BV": V, "BW": 4, "BS": 2, "EV": V, "ES": 2}
    # forward: CTAs per SM by registers, then the largest tile that fits
    threads = (out["FW"] * CH + 2) * 32
    FC = 2 if 65536 // (2 * threads) >= need else 1
    edge = 4 * (P * NQ + DIN * NQ + apad + DSH)
    while True:
        T = min(12, ((smem // FC - 1024 - 256) // out["FS"] - 256) // edge)
        if T >= 3 or FC == 1:
            break
        FC = 1
    if T < 1:
        raise ValueError("one edge does not fit the forward stage ring")
    out.update(FT=T, FC=FC)
    # path-group backward (the fallback; always compiled)
    fixed = 256 + 4 * 2 * out["BW"] * DIN * NQ + 4 * 2 * out["BW"] * CH * 16
    BC = FC
    while True:
        BT = min(8, ((smem // BC - 1024 - fixed) // out["BS"] - 256) // edge)
        if BT >= 2 or BC == 1:
            break
        BC = 1
    if BT < 1:
        raise ValueError("one edge does not fit the backward stage ring")
    out.update(BT=BT, BC=BC)
    # edge-wise backward: one CTA per SM, T edges x CH warps per edge.  When shared memory allows only a few edges
    # per tile, halving the channels per lane doubles the warps (measured on 128x(0e+1o+2e+3o), l <= 2: 4 -> 8
    # consumer warps, 1.77 -> 1.08 ms)
    def edgewise(EV):
        CHe = NQ // (32 * EV)
        warps = 65536 // (32 * {4: 224, 2: 128, 1: 96}[EV]) - 1
        fixed = 2048 + 4 * 2 * 32 * DSH + 4 * out["ES"] * D * NQ
        return min(warps // CHe, 16, ((smem - 1024 - fixed) // out["ES"] - 256) // (edge + 4 * CHe * 16)), CHe
    EV = V
    ET, CHe = edgewise(EV)
    if ET * CHe < 6 and EV > 1:
        EV //= 2
        ET, CHe = edgewise(EV)
    if ET >= 2:
        out.update(ET=ET, EV=EV)
    return out


class Sig:
    def __init__(self, sig):
        self.name = sig["name"]
        self.info, self.paths, self.recs, self.signature = load_records(sig)
        if "V" not in sig:   # no (or only some) tile parameters given: derive the rest
            sig = {**auto_params(sig, self.info), **sig}
        self.cfg = sig
        self.NQ, self.DIN, self.DSH = self.info["n_channels"], self.info["d_in"], self.info["d_sh"]
        self.P, self.D, self.NNZ = self.info["n_paths"], self.info["d_out"], self.info["nnz"]
        self.V = sig["V"]
        assert self.NQ % (32 * self.V) == 0, "channels must fill whole warps"
        # pairs in (i0, path, i1) order with their records (a collapsed plan has several paths per output row)
        self.pairs = []  # (i0, i1, k, [(i2, val)])
        for i0, i1, i2, k, v in self.recs:
            if self.pairs and self.pairs[-1][0] == i0 and self.pairs[-1][1] == i1 and self.pairs[-1][2] == k:
                self.pairs[-1][3].append((i2, v))
            else:
                self.pairs.append((i0, i1, k, [(i2, v)]))
        assert len(self.pairs) == self.info["n_pairs"]
        self.row_pairs = [[] for _ in range(self.D)]   # all pairs of an output row
        self.rp = {}                                   # (row, path) -> pairs
        self.row_paths = [[] for _ in range(self.D)]   # paths that reach an output row, in path order
        for pi, (i0, i1, k, rl) in enumerate(self.pairs):
            self.row_pairs[i0].append(pi)
            self.rp.setdefault((i0, k), []).append(pi)
            if k not in self.row_paths[i0]:
                self.row_paths[i0].append(k)

    # Bodies whose multiplies and fused multiply-adds are emitted in the packed two-channel form (pfma / pmul of
    # fast_common.cuh).  Measured on the 128-channel water signature: the forward-shaped bodies and the double
    # backward gain (fewer issue slots), the first backward's edge body loses (more registers, it is bound by
    # memory), so it stays scalar unless the signature's "PK" list names it.
    PACKED_DEFAULT = ("fwd", "fwd2", "rfwd", "bwd2")

    def ops(self, kind):
        packed = kind in self.cfg.get("PK", self.PACKED_DEFAULT)
        return ("pfma", "pmul") if packed else ("vfma", "vmul")

    def path_rows(self, k):
        p = self.paths[k]
        return range(p["out_off"], p["out_off"] + 2 * p["L"] + 1)

    def pairs_of(self, row, k):
        return self.rp.get((row, k), [])

    # ---------------------------------------------------------------- forward
    def fwd_layout(self, FW=None):
        """Row groups of the forward bodies.  FW given: the layout of the forward that forms its edge scalars in
        the kernel (its own number of row groups, balanced by the estimate alone)."""
        radial = FW is not None
        FW = FW or self.cfg["FW"]
        costs = []
        for row in range(self.D):
            starts = sum((2 * self.paths[k]["l1"] + 1) * 1.0 + 0.5 for k in self.row_paths[row]
                         if row == self.paths[k]["out_off"])
            costs.append(len(self.row_pairs[row]) * 1.0 + starts + 0.3)
        bounds = partition_rows(costs, FW, None if radial else self.cfg.get("F_BIAS"))
        # Measured group sizes override the estimate: consumer warp 1 shares its scheduler with the table
        # producer warp (and warp 0 with the copy warp), so an even split leaves the other two waiting for it.
        if self.cfg.get("F_ROWS") and not radial:
            bounds = [0]
            for r in self.cfg["F_ROWS"]:
                bounds.append(bounds[-1] + r)
            assert bounds[-1] == self.D and len(bounds) == FW + 1
        while len(bounds) < FW + 1:
            bounds.append(bounds[-1])
        a0, slots = [0], []  # slot -> pair index or None
        for g in range(FW):
            for row in range(bounds[g], bounds[g + 1]):
                slots += self.row_pairs[row]
            while len(slots) % 4:
                slots.append(None)
            a0.append(len(slots))
        return bounds, a0, slots

    # ---------------------------------------------------------------- backward
    def bwd_layout(self):
        """Groups of whole paths (any subset, not only contiguous ones), balanced by estimated
        instruction count: longest-processing-time assignment, paths inside a group in path order.
        Optional signature keys: B_SLACK_PCT (how far above the best balance a smaller row cap may be,
        default 3) and B_CAPS (how many row caps are tried, default 6)."""
        BW = self.cfg["BW"]
        V = self.cfg.get("BV", self.V)
        costs = []
        for k, p in enumerate(self.paths):
            rows = self.path_rows(k)
            npairs = sum(len(self.pairs_of(r, k)) for r in rows)
            nrec = sum(len(self.pairs[pi][3]) for r in rows for pi in self.pairs_of(r, k))
            combos = len({self.pairs[pi][1] for r in rows for pi in self.pairs_of(r, k)})
            # per pair: u += A dm and the lane dot product; per record one scalar FMA; per (path, i1): s*x,
            # the grad_w and grad_x FMAs; per path the weight load and the grad_w store
            costs.append(2.0 * V * npairs + nrec + 3.0 * V * combos + npairs / 4.0 + 2.0)
        nrows = [2 * p["L"] + 1 for p in self.paths]

        def assign(cap, order):
            bins = [[0.0, 0, []] for _ in range(BW)]
            for k in order:
                ok = [i for i in range(BW) if bins[i][1] + nrows[k] <= cap]
                if not ok:
                    return None
                tgt = min(ok, key=lambda i: (bins[i][0], i))
                bins[tgt][0] += costs[k]
                bins[tgt][1] += nrows[k]
                bins[tgt][2].append(k)
            return bins

        # The rows of a group live in registers, so the largest group's row count is capped: take the
        # smallest cap whose best assignment found is within 3 % of the best over all caps.
        import random
        rng = random.Random(1234)
        lpt = sorted(range(self.P), key=lambda k: (-costs[k], k))
        found = {}
        for cap in range(-(-self.D // BW), self.D + 1):
            best = None
            for trial in range(400):
                order = list(lpt)
                if trial:
                    for _ in range(1 + trial % 4):  # a few swaps of neighbours in the LPT order
                        i = rng.randrange(len(order) - 1)
                        order[i], order[i + 1] = order[i + 1], order[i]
                bins = assign(cap, order)
                if bins is not None and (best is None or max(b[0] for b in bins) < max(b[0] for b in best)):
                    best = bins
            if best is not None:
                found[cap] = best
            if len(found) >= self.cfg.get("B_CAPS", 6):
                break
        floor_cost = min(max(b[0] for b in bins) for bins in found.values())
        slack = 1.0 + self.cfg.get("B_SLACK_PCT", 3) / 100.0
        cap = min(c for c, bins in found.items() if max(b[0] for b in bins) <= slack * floor_cost)
        bins = [[b[0], b[2]] for b in found[cap]]
        groups = sorted((sorted(b[1]) for b in bins), key=lambda g: (g[0] if g else self.P))
        rows_of = []   # distinct output rows of every group (paths of a collapsed plan may share rows)
        for g in groups:
            rows = []
            for k in g:
                rows += [r for r in self.path_rows(k) if r not in rows]
            rows_of.append(rows)
        a0, slots = [0], []
        for g in groups:
            for k in g:
                for row in self.path_rows(k):
                    slots += self.pairs_of(row, k)
            while len(slots) % 4:
                slots.append(None)
            a0.append(len(slots))
        return groups, rows_of, a0, slots

    def emit_bwd(self):
        if "BW" not in self.cfg:
            return []
        V, NQ = self.cfg.get("BV", self.V), self.NQ
        assert NQ % (32 * V) == 0
        bvec = {1: "float", 2: "float2", 4: "float4"}[V]
        BW, BT, BS, BC = self.cfg["BW"], self.cfg["BT"], self.cfg["BS"], self.cfg["BC"]
        groups, rows_of, a0, slots = self.bwd_layout()
        slot_of_pair = {pi: s for s, pi in enumerate(slots) if pi is not None}
        rmax = max(len(r) for r in rows_of)
        rec_val, rec_i2, pair_tab = [], [], []
        for pi in slots:
            if pi is None:
                pair_tab.append((len(rec_val), 0)); continue
            rl = self.pairs[pi][3]
            pair_tab.append((len(rec_val), len(rl)))
            for i2, v in rl:
                rec_val.append(v); rec_i2.append(i2)
        row_tab = [rows + [rows[-1] if rows else 0] * (rmax - len(rows)) for rows in rows_of]
        self.bwd_tables = (pair_tab, rec_val, rec_i2, row_tab)
        o = []
        o.append(f"    // ---- backward: path groups {groups}")
        o.append(f"    static constexpr int BV = {V};  // channels per lane in the backward")
        o.append(f"    using BVec = {bvec};")
        o.append(f"    static constexpr int BW = {BW}, BT = {BT}, BS = {BS}, BC = {BC}, B_RMAX = {rmax}, B_APAD = {len(slots)}, "
                 f"B_NREC = {max(c for _, c in pair_tab)};")
        o.append(f"    // edge-wise backward (one warp per edge, grad_out rows read from shared memory): edges per tile "
                 f"(0 = not generated), ring stages")
        EV = self.cfg.get("EV", V)
        o.append(f"    static constexpr int ET = {self.cfg.get('ET', 0)}, ES = {self.cfg.get('ES', 2)}, EV = {EV};")
        o.append(f"    // the same for the standalone tensor product: rows per ring slot (0 = not generated), ring slots")
        o.append(f"    static constexpr int ETR = {self.cfg.get('ETR', 0)}, ESR = {self.cfg.get('ESR', 3)};")
        o.append(f"    // fused double backward (edge outputs): edges per tile (0 = not generated), ring stages")
        DV = self.cfg.get("DV", EV)
        o.append(f"    static constexpr int DT = {self.cfg.get('DT', 0)}, DS = {self.cfg.get('DS', 2)}, DV = {DV};")
        o.append(f"    using DVec = {{1: 'float', 2: 'float2', 4: 'float4'}}[DV];".replace("{1: 'float', 2: 'float2', 4: 'float4'}[DV]", {1: "float", 2: "float2", 4: "float4"}[DV]))
        o.append(f"    using EVec = {{1: 'float', 2: 'float2', 4: 'float4'}}[EV];".replace("{1: 'float', 2: 'float2', 4: 'float4'}[EV]", {1: "float", 2: "float2", 4: "float4"}[EV]))
        o.append(f"    __device__ static __forceinline__ PairRec b_pair_rec(int i) {{ return kBPair_{self.name}[i]; }}")
        o.append(f"    __device__ static __forceinline__ float b_rec_val(int i) {{ return kBVal_{self.name}[i]; }}")
        o.append(f"    __device__ static __forceinline__ unsigned char b_rec_i2(int i) {{ return kBI2_{self.name}[i]; }}")
        o.append(f"    // output rows of path group g: b_nrow(g) of them, the r-th is b_row(g, r)")
        o.append(f"    __device__ static __forceinline__ int b_row(int g, int r) {{ return kBRow_{self.name}[g * B_RMAX + r]; }}")
        o.append(f"    static constexpr int b_nrow(int g) {{")
        o.append("        switch (g) {")
        for i, rows in enumerate(rows_of):
            o.append(f"            case {i}: return {len(rows)};")
        o.append(f"            default: return 0;")
        o.append("        }\n    }")
        o.append(f"    __device__ static __forceinline__ void bwd_edge(const int G, const BVec (&dm)[B_RMAX], const BVec* __restrict__ xs, "
                 f"const BVec* __restrict__ ss, const float* __restrict__ As, BVec (&dxp)[DIN], float (&dyl)[16], "
                 f"BVec* __restrict__ gw) {{")
        o.append(f"        constexpr int NQV = NQ / BV;")
        o.append("        switch (G) {")
        for g in range(BW):
            o.append(f"        case {g}: {{")
            rows = rows_of[g]
            local = {row: i for i, row in enumerate(rows)}
            need_x = sorted({self.pairs[pi][1] for k in groups[g] for row in self.path_rows(k)
                             for pi in self.pairs_of(row, k)})
            for i1 in need_x:
                o.append(f"            const BVec x{i1} = xs[{i1} * NQV];")
            loaded_a = set()
            dx_touched, dy_touched = set(), set()   # first contribution assigns, later ones accumulate
            for k in groups[g]:
                p = self.paths[k]
                prow = list(self.path_rows(k))
                used = sorted({self.pairs[pi][1] for r2 in prow for pi in self.pairs_of(r2, k)})
                o.append(f"            const BVec s{k} = ss[{k} * NQV];  // path {k}: l1={p['l1']} l2={p['l2']} -> L={p['L']}")
                for i1 in used:
                    F, M = self.ops("bwd"); o.append(f"            const BVec sx{k}_{i1} = {M}(s{k}, x{i1});")
                    o.append(f"            BVec u{k}_{i1}; vzero(u{k}_{i1});")
                depth = max(len(self.pairs_of(r2, k)) for r2 in prow)
                for j in range(depth):
                    for row in prow:
                        if j >= len(self.pairs_of(row, k)):
                            continue
                        pi = self.pairs_of(row, k)[j]
                        slot = slot_of_pair[pi]
                        q, lane = slot // 4, "xyzw"[slot % 4]
                        if q not in loaded_a:
                            loaded_a.add(q)
                            o.append(f"            const float4 a{q} = *reinterpret_cast<const float4*>(As + {4 * q});")
                        i1 = self.pairs[pi][1]
                        r = local[row]
                        F, M = self.ops("bwd"); o.append(f"            {F}(u{k}_{i1}, a{q}.{lane}, dm[{r}]);")
                        o.append(f"            {{ const float t = vdot(sx{k}_{i1}, dm[{r}]);")
                        for i2, c in self.pairs[pi][3]:
                            if i2 in dy_touched:
                                o.append(f"              dyl[{i2}] = fmaf({fmt_float(c)}, t, dyl[{i2}]);")
                            else:
                                dy_touched.add(i2)
                                o.append(f"              dyl[{i2}] = {fmt_float(c)} * t;")
                        o.append("            }")
                first = used[0]
                F, M = self.ops("bwd"); o.append(f"            BVec ds{k} = {M}(x{first}, u{k}_{first});")
                for i1 in used[1:]:
                    F, M = self.ops("bwd"); o.append(f"            {F}(ds{k}, x{i1}, u{k}_{i1});")
                o.append(f"            if (gw) gw[{k} * NQV] = ds{k};")
                for i1 in used:
                    if i1 in dx_touched:
                        F, M = self.ops("bwd"); o.append(f"            {F}(dxp[{i1}], s{k}, u{k}_{i1});")
                    else:
                        dx_touched.add(i1)
                        F, M = self.ops("bwd"); o.append(f"            dxp[{i1}] = {M}(s{k}, u{k}_{i1});")
            # entries this group never touches
            for i1 in range(self.DIN):
                if i1 not in dx_touched:
                    o.append(f"            vzero(dxp[{i1}]);")
            for i2 in range(16):
                if i2 not in dy_touched:
                    o.append(f"            dyl[{i2}] = 0.f;")
            o.append("        } break;")
        o.append("        default: {")
        o.append("#pragma unroll")
        o.append("            for (int i = 0; i < DIN; ++i) vzero(dxp[i]);")
        o.append("#pragma unroll")
        o.append("            for (int i = 0; i < 16; ++i) dyl[i] = 0.f;")
        o.append("        } break;")
        o.append("        }")
        o.append("    }")
        if self.cfg.get("ET", 0) or self.cfg.get("ETR", 0):
            o += self.emit_bwd_edgewise(slot_of_pair)
        if self.cfg.get("DT", 0):
            o += self.emit_bwd2_edgewise(slot_of_pair)
        return o

    def emit_bwd_edgewise(self, slot_of_pair):
        """The whole backward of one edge in one warp: every path in turn, the rows of grad_out[receiver]
        loaded from shared memory (dms) where they are used, no partial sums to exchange."""
        o = []
        o.append(f"    __device__ static __forceinline__ void bwd_edge_all(const EVec* __restrict__ dms, const EVec* __restrict__ xs, "
                 f"const EVec* __restrict__ ss, const float* __restrict__ As, EVec (&dxp)[DIN], float (&dyl)[16], "
                 f"EVec* __restrict__ gw) {{")
        o.append(f"        constexpr int NQV = NQ / EV;")
        for i1 in range(self.DIN):
            o.append(f"        const EVec x{i1} = xs[{i1} * NQV];")
        loaded_a, dx_touched, dy_touched = set(), set(), set()
        for k in range(self.P):
            p = self.paths[k]
            prow = list(self.path_rows(k))
            used = sorted({self.pairs[pi][1] for r2 in prow for pi in self.pairs_of(r2, k)})
            o.append(f"        const EVec s{k} = ss[{k} * NQV];  // path {k}: l1={p['l1']} l2={p['l2']} -> L={p['L']}")
            for i1 in used:
                F, M = self.ops("bwd"); o.append(f"        const EVec sx{k}_{i1} = {M}(s{k}, x{i1});")
                o.append(f"        EVec u{k}_{i1}; vzero(u{k}_{i1});")
            depth = max(len(self.pairs_of(r2, k)) for r2 in prow)
            have = set()
            for j in range(depth):
                for row in prow:
                    if j >= len(self.pairs_of(row, k)):
                        continue
                    if row not in have:
                        have.add(row)
                        o.append(f"        const EVec d{k}_{row} = dms[{row} * NQV];")
                    pi = self.pairs_of(row, k)[j]
                    slot = slot_of_pair[pi]
                    q, lane = slot // 4, "xyzw"[slot % 4]
                    if q not in loaded_a:
                        loaded_a.add(q)
                        o.append(f"        const float4 a{q} = *reinterpret_cast<const float4*>(As + {4 * q});")
                    i1 = self.pairs[pi][1]
                    F, M = self.ops("bwd"); o.append(f"        {F}(u{k}_{i1}, a{q}.{lane}, d{k}_{row});")
                    o.append(f"        {{ const float t = vdot(sx{k}_{i1}, d{k}_{row});")
                    for i2, c in self.pairs[pi][3]:
                        if i2 in dy_touched:
                            o.append(f"          dyl[{i2}] = fmaf({fmt_float(c)}, t, dyl[{i2}]);")
                        else:
                            dy_touched.add(i2)
                            o.append(f"          dyl[{i2}] = {fmt_float(c)} * t;")
                    o.append("        }")
            first = used[0]
            F, M = self.ops("bwd"); o.append(f"        EVec ds{k} = {M}(x{first}, u{k}_{first});")
            for i1 in used[1:]:
                F, M = self.ops("bwd"); o.append(f"        {F}(ds{k}, x{i1}, u{k}_{i1});")
            o.append(f"        if (gw) gw[{k} * NQV] = ds{k};")
            for i1 in used:
                if i1 in dx_touched:
                    F, M = self.ops("bwd"); o.append(f"        {F}(dxp[{i1}], s{k}, u{k}_{i1});")
                else:
                    dx_touched.add(i1)
                    F, M = self.ops("bwd"); o.append(f"        dxp[{i1}] = {M}(s{k}, u{k}_{i1});")
        for i1 in range(self.DIN):
            if i1 not in dx_touched:
                o.append(f"        vzero(dxp[{i1}]);")
        for i2 in range(16):
            if i2 not in dy_touched:
                o.append(f"        dyl[{i2}] = 0.f;")
        o.append("    }")
        return o

    def emit_bwd2_edgewise(self, slot_of_pair):
        """Edge outputs of the double backward in one sweep, one warp per edge.  With the cotangents (ux, uy, us)
        of (grad_x, grad_sh, grad_w), A = C y, B = C uy, g = grad_out[receiver]:
          v[k,i1] = sum_i0 A g[i0],  v2[k,i1] = sum_i0 B g[i0],  sxu[k,i1] = s[k] ux[i1] + us[k] x[i1]
          d_s[k]  = sum_i1 ux[i1] v + x[i1] v2;   d_x[i1] = sum_k us[k] v + s[k] v2;
          d_y[i2] = sum C g[i0] sxu[k,i1]."""
        o = []
        o.append(f"    __device__ static __forceinline__ void bwd2_edge_all(const DVec* __restrict__ dms, const DVec* __restrict__ xs, "
                 f"const DVec* __restrict__ uxs, const DVec* __restrict__ ss, const DVec* __restrict__ uss, "
                 f"const float* __restrict__ As, const float* __restrict__ Bs, DVec (&dxp)[DIN], float (&dyl)[16], "
                 f"DVec* __restrict__ gw) {{")
        o.append(f"        constexpr int NQV = NQ / DV;")
        for i1 in range(self.DIN):
            o.append(f"        const DVec x{i1} = xs[{i1} * NQV];")
            o.append(f"        const DVec ux{i1} = uxs[{i1} * NQV];")
        loaded_a, dx_touched, dy_touched = set(), set(), set()
        for k in range(self.P):
            p = self.paths[k]
            prow = list(self.path_rows(k))
            used = sorted({self.pairs[pi][1] for r2 in prow for pi in self.pairs_of(r2, k)})
            o.append(f"        const DVec s{k} = ss[{k} * NQV];  // path {k}: l1={p['l1']} l2={p['l2']} -> L={p['L']}")
            o.append(f"        const DVec us{k} = uss[{k} * NQV];")
            for i1 in used:
                F, M = self.ops("bwd2"); o.append(f"        DVec sxu{k}_{i1} = {M}(s{k}, ux{i1}); {F}(sxu{k}_{i1}, us{k}, x{i1});")
                o.append(f"        DVec v{k}_{i1}; vzero(v{k}_{i1});")
                o.append(f"        DVec w{k}_{i1}; vzero(w{k}_{i1});")
            depth = max(len(self.pairs_of(r2, k)) for r2 in prow)
            have = set()
            for j in range(depth):
                for row in prow:
                    if j >= len(self.pairs_of(row, k)):
                        continue
                    if row not in have:
                        have.add(row)
                        o.append(f"        const DVec d{k}_{row} = dms[{row} * NQV];")
                    pi = self.pairs_of(row, k)[j]
                    slot = slot_of_pair[pi]
                    q, lane = slot // 4, "xyzw"[slot % 4]
                    if q not in loaded_a:
                        loaded_a.add(q)
                        o.append(f"        const float4 a{q} = *reinterpret_cast<const float4*>(As + {4 * q});")
                        o.append(f"        const float4 b{q} = *reinterpret_cast<const float4*>(Bs + {4 * q});")
                    i1 = self.pairs[pi][1]
                    F, M = self.ops("bwd2"); o.append(f"        {F}(v{k}_{i1}, a{q}.{lane}, d{k}_{row});")
                    F, M = self.ops("bwd2"); o.append(f"        {F}(w{k}_{i1}, b{q}.{lane}, d{k}_{row});")
                    o.append(f"        {{ const float t = vdot(sxu{k}_{i1}, d{k}_{row});")
                    for i2, c in self.pairs[pi][3]:
                        if i2 in dy_touched:
                            o.append(f"          dyl[{i2}] = fmaf({fmt_float(c)}, t, dyl[{i2}]);")
                        else:
                            dy_touched.add(i2)
                            o.append(f"          dyl[{i2}] = {fmt_float(c)} * t;")
                    o.append("        }")
            first = used[0]
            F, M = self.ops("bwd2"); o.append(f"        DVec ds{k} = {M}(ux{first}, v{k}_{first}); {F}(ds{k}, x{first}, w{k}_{first});")
            for i1 in used[1:]:
                F, M = self.ops("bwd2"); o.append(f"        {F}(ds{k}, ux{i1}, v{k}_{i1}); {F}(ds{k}, x{i1}, w{k}_{i1});")
            o.append(f"        if (gw) gw[{k} * NQV] = ds{k};")
            for i1 in used:
                if i1 in dx_touched:
                    F, M = self.ops("bwd2"); o.append(f"        {F}(dxp[{i1}], us{k}, v{k}_{i1}); {F}(dxp[{i1}], s{k}, w{k}_{i1});")
                else:
                    dx_touched.add(i1)
                    F, M = self.ops("bwd2"); o.append(f"        dxp[{i1}] = {M}(us{k}, v{k}_{i1}); {F}(dxp[{i1}], s{k}, w{k}_{i1});")
        for i1 in range(self.DIN):
            if i1 not in dx_touched:
                o.append(f"        vzero(dxp[{i1}]);")
        for i2 in range(16):
            if i2 not in dy_touched:
                o.append(f"        dyl[{i2}] = 0.f;")
        o.append("    }")
        return o

    def emit_radial(self):
        """Bodies of the forward that forms its edge scalars in the kernel: RF row groups (one consumer warp each),
        their own A-slot order, and the A entries of one edge computed from harmonics held in registers."""
        RW = self.cfg["RF"]
        bounds, a0, slots = self.fwd_layout(RW)
        slot_of_pair = {pi: s for s, pi in enumerate(slots) if pi is not None}
        rmax = max(bounds[g + 1] - bounds[g] for g in range(RW))
        o = []
        o.append(f"    // ---- forward with in-kernel edge scalars (fast_radial.cuh): {RW} row groups")
        o.append(f"    static constexpr int R_FW = {RW}, R_RMAX = {rmax}, R_APAD = {len(slots)};")
        o.append(f"    static constexpr int r_row0(int g) {{")
        o.append("        switch (g) {")
        for i, v in enumerate(bounds):
            o.append(f"            case {i}: return {v};")
        o.append(f"            default: return {bounds[-1]};")
        o.append("        }\n    }")
        o.append(f"    template <int G>")
        o.append(f"    __device__ static __forceinline__ void rfwd_edge(Vec (&acc)[R_RMAX], "
                 f"const Vec* __restrict__ xs, const Vec* __restrict__ ss, const float* __restrict__ As) {{")
        o.append(f"        constexpr int NQV = NQ / V;")
        for g in range(RW):
            o.append(f"        if constexpr (G == {g}) {{")
            rows = range(bounds[g], bounds[g + 1])
            need_x = sorted({self.pairs[pi][1] for row in rows for pi in self.row_pairs[row]})
            for i1 in need_x:
                o.append(f"            const Vec x{i1} = xs[{i1} * NQV];")
            loaded_a = set()
            paths_here = []
            for row in rows:
                for k in self.row_paths[row]:
                    if k not in paths_here:
                        paths_here.append(k)
            for k in paths_here:
                prow = [r2 for r2 in rows if self.pairs_of(r2, k)]
                o.append(f"            const Vec s{k} = ss[{k} * NQV];")
                used = sorted({self.pairs[pi][1] for r2 in prow for pi in self.pairs_of(r2, k)})
                for i1 in used:
                    F, M = self.ops("rfwd"); o.append(f"            const Vec sx{k}_{i1} = {M}(s{k}, x{i1});")
                depth = max(len(self.pairs_of(r2, k)) for r2 in prow)
                for j in range(depth):
                    for row in prow:
                        if j >= len(self.pairs_of(row, k)):
                            continue
                        pi = self.pairs_of(row, k)[j]
                        slot = slot_of_pair[pi]
                        q, lane = slot // 4, "xyzw"[slot % 4]
                        if q not in loaded_a:
                            loaded_a.add(q)
                            o.append(f"            const float4 a{q} = *reinterpret_cast<const float4*>(As + {4 * q});")
                        i1 = self.pairs[pi][1]
                        F, M = self.ops("rfwd"); o.append(f"            {F}(acc[{row - bounds[g]}], a{q}.{lane}, sx{k}_{i1});")
            o.append("        }")
        o.append("    }")
        o.append(f"    template <int G, class VecT>")
        o.append(f"    __device__ static __forceinline__ void rfwd_store(const VecT (&acc)[R_RMAX], VecT* __restrict__ dst, const int stride) {{")
        for g in range(RW):
            o.append(f"        if constexpr (G == {g}) {{")
            for row in range(bounds[g], bounds[g + 1]):
                o.append(f"            dst[{row - bounds[g]} * stride] = acc[{row - bounds[g]}];")
            o.append("        }")
        o.append("    }")
        assert len(slots) % 4 == 0
        o.append(f"    // A[slot] = sum over the slot's records of c * y[i2], four slots per store")
        o.append(f"    __device__ static __forceinline__ void a_entries(const float (&y)[DSH], float4* __restrict__ dst) {{")
        for q in range(len(slots) // 4):
            terms = []
            for s_i in range(4 * q, 4 * q + 4):
                pi = slots[s_i]
                if pi is None:
                    terms.append("0.f")
                else:
                    terms.append(" + ".join(f"{fmt_float(v)} * y[{i2}]" for i2, v in self.pairs[pi][3]))
            o.append(f"        dst[{q}] = make_float4({', '.join(terms)});")
        o.append("    }")
        return o

    def emit(self) -> str:
        V, NQ = self.V, self.NQ
        FW, FT, FS, FC = self.cfg["FW"], self.cfg["FT"], self.cfg["FS"], self.cfg["FC"]
        bounds, a0, slots = self.fwd_layout()
        slot_of_pair = {pi: s for s, pi in enumerate(slots) if pi is not None}
        rmax = max(bounds[g + 1] - bounds[g] for g in range(FW))
        vec = {1: "float", 2: "float2", 4: "float4"}[V]
        # record tables in slot order
        rec_val, rec_i2, pair_tab = [], [], []
        for pi in slots:
            if pi is None:
                pair_tab.append((len(rec_val), 0))
                continue
            rl = self.pairs[pi][3]
            pair_tab.append((len(rec_val), len(rl)))
            for i2, v in rl:
                rec_val.append(v); rec_i2.append(i2)
        assert len(rec_val) == self.NNZ
        S = f"Sig_{self.name}"
        o = []
        o.append(f"// GENERATED by csrc/gen_fast.py from fast/signatures.json -- do not edit.")
        o.append(f"// signature: {self.signature}")
        o.append(f"// {self.cfg['irreps_in']} (x) harmonics l<={self.cfg['sh_lmax']}: P={self.P} D={self.D} "
                 f"nnz={self.NNZ} pairs={len(self.pairs)}")
        o.append('#include "fast_fwd.cuh"')
        o.append('#include "fast_bwd.cuh"')
        o.append('#include "fast_launch.cuh"')
        if self.cfg.get("SB", 0):
            o.append('#include "fast_bwd1s.cuh"')
        if self.cfg.get("RF", 0):
            o.append('#include "fast_radial.cuh"')
        o.append("")
        o.append("namespace e3j {\nnamespace fast {\nnamespace {")
        o.append(f"__device__ const PairRec kPair_{self.name}[{len(pair_tab)}] = {{")
        o.append("    " + ", ".join(f"{{{s},{c}}}" for s, c in pair_tab) + "};")
        o.append(f"__device__ const float kVal_{self.name}[{self.NNZ}] = {{")
        o.append("    " + ", ".join(fmt_float(v) for v in rec_val) + "};")
        o.append(f"__device__ const unsigned char kI2_{self.name}[{self.NNZ}] = {{")
        o.append("    " + ", ".join(str(i) for i in rec_i2) + "};")
        bwd_lines = self.emit_bwd()
        if bwd_lines:
            bpair, bval, bi2, brow = self.bwd_tables
            o.append(f"__device__ const PairRec kBPair_{self.name}[{len(bpair)}] = {{")
            o.append("    " + ", ".join(f"{{{s_},{c_}}}" for s_, c_ in bpair) + "};")
            o.append(f"__device__ const float kBVal_{self.name}[{len(bval)}] = {{")
            o.append("    " + ", ".join(fmt_float(v) for v in bval) + "};")
            o.append(f"__device__ const unsigned char kBI2_{self.name}[{len(bi2)}] = {{")
            o.append("    " + ", ".join(str(i) for i in bi2) + "};")
            o.append(f"__device__ const unsigned char kBRow_{self.name}[{len(brow) * len(brow[0])}] = {{")
            o.append("    " + ", ".join(str(i) for rows in brow for i in rows) + "};")
        o.append("")
        o.append(f"struct {S} {{")
        o.append(f"    static constexpr int NQ = {NQ}, DIN = {self.DIN}, DSH = {self.DSH}, P = {self.P}, D = {self.D};")
        o.append(f"    static constexpr int NNZ = {self.NNZ}, NPAIR = {len(self.pairs)}, V = {V};")
        o.append(f"    static constexpr int FW = {FW}, FT = {FT}, FS = {FS}, FC = {FC}, F_RMAX = {rmax}, F_APAD = {len(slots)}, F_NREC = {max(c for _, c in pair_tab)}, F_NPMAX = {max(a0[g + 1] - a0[g] for g in range(FW))}, F_MAXREG = {self.cfg.get("F_MAXREG", 255)};")
        o.append(f"    // fused double backward (cotangent of grad_out): tile, stages, CTAs per SM (DFT = 0: not generated)")
        DFV = self.cfg.get("DFV", V)
        dfvec = {1: "float", 2: "float2", 4: "float4"}[DFV]
        o.append(f"    static constexpr int DFT = {self.cfg.get('DFT', 0)}, DFS = {self.cfg.get('DFS', 2)}, DFC = {self.cfg.get('DFC', 1)}, DFV = {DFV};")
        o.append(f"    using DFVec = {dfvec};")
        o.append(f"    using Vec = {vec};")
        o.append(f"    __device__ static __forceinline__ PairRec pair_rec(int i) {{ return kPair_{self.name}[i]; }}")
        o.append(f"    __device__ static __forceinline__ float rec_val(int i) {{ return kVal_{self.name}[i]; }}")
        o.append(f"    __device__ static __forceinline__ unsigned char rec_i2(int i) {{ return kI2_{self.name}[i]; }}")

        def table_fn(fname, values):
            o.append(f"    static constexpr int {fname}(int g) {{")
            o.append("        switch (g) {")
            for i, v in enumerate(values):
                o.append(f"            case {i}: return {v};")
            o.append(f"            default: return {values[-1]};")
            o.append("        }\n    }")

        table_fn("f_row0", bounds)
        table_fn("f_a0", a0)

        # ---- fwd_edge
        o.append(f"    template <int G>")
        o.append(f"    __device__ static __forceinline__ void fwd_edge(Vec (&acc)[F_RMAX], "
                 f"const Vec* __restrict__ xs, const Vec* __restrict__ ss, const float* __restrict__ As) {{")
        o.append(f"        constexpr int NQV = NQ / V;")
        for g in range(FW):
            o.append(f"        if constexpr (G == {g}) {{")
            rows = range(bounds[g], bounds[g + 1])
            need_x = sorted({self.pairs[pi][1] for row in rows for pi in self.row_pairs[row]})
            for i1 in need_x:
                o.append(f"            const Vec x{i1} = xs[{i1} * NQV];")
            loaded_a = set()
            paths_here = []
            for row in rows:
                for k in self.row_paths[row]:
                    if k not in paths_here:
                        paths_here.append(k)
            for k in paths_here:
                p = self.paths[k]
                prow = [r2 for r2 in rows if self.pairs_of(r2, k)]
                o.append(f"            const Vec s{k} = ss[{k} * NQV];  // path {k}: l1={p['l1']} l2={p['l2']} -> L={p['L']}")
                used = sorted({self.pairs[pi][1] for r2 in prow for pi in self.pairs_of(r2, k)})
                for i1 in used:
                    F, M = self.ops("fwd"); o.append(f"            const Vec sx{k}_{i1} = {M}(s{k}, x{i1});")
                # round-robin over the rows of the path so that consecutive FMAs hit different accumulators
                depth = max(len(self.pairs_of(r2, k)) for r2 in prow)
                for j in range(depth):
                    for row in prow:
                        if j >= len(self.pairs_of(row, k)):
                            continue
                        pi = self.pairs_of(row, k)[j]
                        slot = slot_of_pair[pi]
                        q, lane = slot // 4, "xyzw"[slot % 4]
                        if q not in loaded_a:
                            loaded_a.add(q)
                            o.append(f"            const float4 a{q} = *reinterpret_cast<const float4*>(As + {4 * q});")
                        i1 = self.pairs[pi][1]
                        F, M = self.ops("fwd"); o.append(f"            {F}(acc[{row - bounds[g]}], a{q}.{lane}, sx{k}_{i1});")
            o.append("        }")
        o.append("    }")

        # ---- fwd2_edge: cotangent of grad_out in the double backward,
        # acc[i0] += A[i0,i1] (s ux[i1] + us x[i1]) + B[i0,i1] (s x[i1]),  A = C y, B = C uy
        if self.cfg.get("DFT", 0):
            o.append(f"    template <int G>")
            o.append(f"    __device__ static __forceinline__ void fwd2_edge(DFVec (&acc)[F_RMAX], "
                     f"const DFVec* __restrict__ xs, const DFVec* __restrict__ uxs, const DFVec* __restrict__ ss, "
                     f"const DFVec* __restrict__ uss, const float* __restrict__ As, const float* __restrict__ Bs) {{")
            o.append(f"        constexpr int NQV = NQ / DFV;")
            for g in range(FW):
                o.append(f"        if constexpr (G == {g}) {{")
                rows = range(bounds[g], bounds[g + 1])
                need_x = sorted({self.pairs[pi][1] for row in rows for pi in self.row_pairs[row]})
                for i1 in need_x:
                    o.append(f"            const DFVec x{i1} = xs[{i1} * NQV];")
                    o.append(f"            const DFVec ux{i1} = uxs[{i1} * NQV];")
                loaded_a = set()
                paths_here = []
                for row in rows:
                    for k in self.row_paths[row]:
                        if k not in paths_here:
                            paths_here.append(k)
                for k in paths_here:
                    prow = [r2 for r2 in rows if self.pairs_of(r2, k)]
                    o.append(f"            const DFVec s{k} = ss[{k} * NQV];")
                    o.append(f"            const DFVec us{k} = uss[{k} * NQV];")
                    used = sorted({self.pairs[pi][1] for r2 in prow for pi in self.pairs_of(r2, k)})
                    for i1 in used:
                        F, M = self.ops("fwd2"); o.append(f"            const DFVec sx{k}_{i1} = {M}(s{k}, x{i1});")
                        F, M = self.ops("fwd2"); o.append(f"            DFVec sxu{k}_{i1} = {M}(s{k}, ux{i1}); {F}(sxu{k}_{i1}, us{k}, x{i1});")
                    depth = max(len(self.pairs_of(r2, k)) for r2 in prow)
                    for j in range(depth):
                        for row in prow:
                            if j >= len(self.pairs_of(row, k)):
                                continue
                            pi = self.pairs_of(row, k)[j]
                            slot = slot_of_pair[pi]
                            q, lane = slot // 4, "xyzw"[slot % 4]
                            if q not in loaded_a:
                                loaded_a.add(q)
                                o.append(f"            const float4 a{q} = *reinterpret_cast<const float4*>(As + {4 * q});")
                                o.append(f"            const float4 b{q} = *reinterpret_cast<const float4*>(Bs + {4 * q});")
                            i1 = self.pairs[pi][1]
                            F, M = self.ops("fwd2"); o.append(f"            {F}(acc[{row - bounds[g]}], a{q}.{lane}, sxu{k}_{i1});")
                            F, M = self.ops("fwd2"); o.append(f"            {F}(acc[{row - bounds[g]}], b{q}.{lane}, sx{k}_{i1});")
                o.append("        }")
            o.append("    }")

        # ---- fwd_store
        o.append(f"    // writes the group's rows to dst[r * stride] (dst already offset by the lane and the first row)")
        o.append(f"    template <int G, class VecT>")
        o.append(f"    __device__ static __forceinline__ void fwd_store(const VecT (&acc)[F_RMAX], VecT* __restrict__ dst, const int stride) {{")
        for g in range(FW):
            o.append(f"        if constexpr (G == {g}) {{")
            for row in range(bounds[g], bounds[g + 1]):
                o.append(f"            dst[{row - bounds[g]} * stride] = acc[{row - bounds[g]}];")
            o.append("        }")
        o.append("    }")
        if self.cfg.get("RF", 0):
            o += self.emit_radial()
        o += bwd_lines
        o.append("};")
        o.append("}  // namespace")
        o.append("}  // namespace fast")
        o.append("")
        o.append(f"extern const FastKernels kFast_{self.name};")
        o.append(f"const FastKernels kFast_{self.name} = {{")
        o.append(f'    "{self.signature}",')
        if bwd_lines:
            o.append(f"    &fast::fwd_scratch_bytes<fast::{S}>, &fast::bwd_scratch_bytes<fast::{S}>, "
                     f"&fast::launch_fwd<fast::{S}>, &fast::launch_bwd<fast::{S}>, &fast::launch_tp_fwd<fast::{S}>, "
                     f"&fast::launch_tp_bwd<fast::{S}>,")
            dbl_e = f"&fast::launch_dbl_edges<fast::{S}>" if self.cfg.get("DT", 0) else "nullptr"
            dbl_o = f"&fast::launch_dbl_out<fast::{S}>" if self.cfg.get("DFT", 0) else "nullptr"
            rf = f"&fast::launch_radial_fwd<fast::{S}>" if self.cfg.get("RF", 0) else "nullptr"
            sb = (f"&fast::launch_bwd_sched<fast::{S}>, {self.cfg['ET']}" if self.cfg.get("SB", 0) else "nullptr, 0")
            o.append(f"    {dbl_e}, {dbl_o}, {rf}, {sb}}};")
        else:
            o.append(f"    &fast::fwd_scratch_bytes<fast::{S}>, nullptr, &fast::launch_fwd<fast::{S}>, nullptr, nullptr, nullptr, "
                     f"nullptr, nullptr}};")
        o.append("}  // namespace e3j")
        return "\n".join(o) + "\n"


def generate(extra=None):
    """{file name: text} for the committed signatures plus, if given, the entries of an overlay list."""
    sigs = json.loads((HERE / "fast" / "signatures.json").read_text())
    if extra:
        have = {s["name"] for s in sigs}
        for s in extra:
            if s["name"] in have:
                raise ValueError(f"overlay signature {s['name']} already exists")
        sigs = sigs + list(extra)
    files = {}
    for sig in sigs:
        files[f"sig_{sig['name']}.cu"] = Sig(sig).emit()
    entries = "// GENERATED by csrc/gen_fast.py -- one E3J_FAST_ENTRY(name) per specialised signature\n"
    entries += "".join(f"E3J_FAST_ENTRY(kFast_{sig['name']})\n" for sig in sigs)
    files["registry_entries.inc"] = entries
    return files


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--check", action="store_true", help="exit 1 if a generated file is out of date")
    args = ap.parse_args()
    files = generate()
    stale = []
    for name, text in files.items():
        path = HERE / "fast" / name
        if not path.exists() or path.read_text() != text:
            stale.append(name)
            if not args.check:
                path.write_text(text)
    if args.check and stale:
        print("stale generated files:", ", ".join(stale))
        sys.exit(1)
    print("generated" if not args.check else "up to date", ", ".join(files))


if __name__ == "__main__":
    main()
