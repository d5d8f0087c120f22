"""The processing order of the scheduled backward (host builder, no GPU): every edge once, runs of one sender in one
column, every run's row written once, grad_out rows resident when used and never overwritten while in use."""
import ctypes

import numpy as np
import pytest

import paper_2609_35099_b200 as e3j
from paper_2609_35099_b200 import workloads

NSLOT, NSTAGE, WINDOW = 3, 2, 2


def build(T, n_ranges, n_nodes, snd, rcv):
    lib = e3j._load()
    fn = lib.e3j_bwd_schedule_build_host
    fn.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                   ctypes.c_void_p, ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
    fn.restype = ctypes.c_int
    snd = np.ascontiguousarray(snd, dtype=np.int32); rcv = np.ascontiguousarray(rcv, dtype=np.int32)
    need = ctypes.c_size_t(0)
    rc = fn(T, n_ranges, n_nodes, len(snd), snd.ctypes.data, rcv.ctypes.data, None, 0, ctypes.byref(need))
    if rc == -1:
        return None
    assert rc == -2
    words = np.zeros(need.value, dtype=np.int32)
    assert fn(T, n_ranges, n_nodes, len(snd), snd.ctypes.data, rcv.ctypes.data, words.ctypes.data, len(words),
              ctypes.byref(need)) == 0
    return words


def check(words, T, n_ranges, n_nodes, snd, rcv):
    E = len(snd)
    magic, t_, nslot, nr, n_tiles, n_rows, ne, nn, off_tp, off_rp, off_t = (int(v) for v in words[:11])
    assert (magic, t_, nslot, nr, ne, nn) == (0x53434844, T, NSLOT, n_ranges, E, n_nodes)
    assert off_t % 4 == 0
    tile_ptr = words[off_tp:off_tp + n_ranges + 1]
    row_ptr = words[off_rp:off_rp + n_nodes + 1]
    assert tile_ptr[0] == 0 and tile_ptr[-1] == n_tiles and np.all(np.diff(tile_ptr) >= 0)
    assert row_ptr[0] == 0 and row_ptr[-1] == n_rows and np.all(np.diff(row_ptr) >= 0)
    tiles = words[off_t:off_t + n_tiles * (T + 1) * 4].reshape(n_tiles, T + 1, 4)
    chunk = max(1, -(-E // n_ranges))
    seen_edge = np.zeros(E, dtype=np.int32)
    seen_row = np.zeros(n_rows, dtype=np.int32)
    for c in range(n_ranges):
        occupant = [-1] * NSLOT
        last_use = [-(10 ** 9)] * NSLOT
        open_sender = [-1] * T
        for t in range(tile_ptr[c], tile_ptr[c + 1]):
            lt = t - tile_ptr[c]
            for u in range(NSLOT):
                q = int(tiles[t, T, u])
                if q >= 0:
                    assert q % NSLOT == u
                    assert last_use[u] <= lt - NSTAGE, "row overwritten while a tile in flight may read it"
                    occupant[u] = q
            for j in range(T):
                e, s, row, slot = (int(v) for v in tiles[t, j])
                if e < 0:
                    continue
                assert e // chunk == c and s == snd[e] and slot == rcv[e] % NSLOT
                assert occupant[slot] == rcv[e], "grad_out row not resident"
                last_use[slot] = lt
                seen_edge[e] += 1
                assert open_sender[j] in (-1, s), "a run mixes senders"
                if row >= 0:
                    assert row_ptr[s] <= row < row_ptr[s + 1]
                    seen_row[row] += 1
                    open_sender[j] = -1
                else:
                    open_sender[j] = s
        assert open_sender == [-1] * T, "a run is left open at the end of a range"
    assert np.all(seen_edge == 1) and np.all(seen_row == 1)
    return n_tiles, n_rows


@pytest.mark.parametrize("T,n_ranges", [(7, 148), (5, 148), (7, 3), (10, 1)])
def test_schedule_invariants_on_the_water_box(T, n_ranges):
    wl = workloads.make_graph(2, 648)
    words = build(T, n_ranges, wl.n_nodes, wl.senders, wl.receivers)
    n_tiles, n_rows = check(words, T, n_ranges, wl.n_nodes, wl.senders, wl.receivers)
    assert n_rows < wl.n_edges          # runs longer than one edge exist
    assert n_tiles * T < 1.6 * wl.n_edges + 4 * T * n_ranges


def test_schedule_of_the_bench_graph_merges_shares_and_fills_its_tiles():
    wl = workloads.make_graph(2)
    words = build(7, 148, wl.n_nodes, wl.senders, wl.receivers)
    n_tiles, n_rows = check(words, 7, 148, wl.n_nodes, wl.senders, wl.receivers)
    assert wl.n_edges / n_rows > 1.55           # simulated: 1.64 edges per written row
    assert wl.n_edges / (n_tiles * 7) > 0.90    # slot use; the plain kernel's tiles reach 0.94


def test_schedule_edge_cases():
    # no edges; one edge; duplicate edges; a sender whose receivers are more than the window apart; isolated nodes
    assert check(build(7, 4, 5, [], []), 7, 4, 5, np.zeros(0, np.int32), np.zeros(0, np.int32)) == (0, 0)
    snd = np.array([2], np.int32); rcv = np.array([0], np.int32)
    assert check(build(7, 4, 3, snd, rcv), 7, 4, 3, snd, rcv)[1] == 1
    snd = np.array([1, 1, 1, 0, 1, 1], np.int32); rcv = np.array([0, 0, 1, 2, 4, 9], np.int32)
    n_tiles, n_rows = check(build(3, 1, 10, snd, rcv), 3, 1, 10, snd, rcv)
    assert n_rows == 4     # sender 1: {0,0,1}, {4}, {9}; sender 0: {2}
    rng = np.random.default_rng(0)
    for _ in range(20):
        n = int(rng.integers(1, 40)); e = int(rng.integers(0, 400))
        snd = rng.integers(0, n, size=e).astype(np.int32)
        rcv = np.sort(rng.integers(0, n, size=e)).astype(np.int32)
        T = int(rng.integers(1, 12)); g = int(rng.integers(1, 9))
        check(build(T, g, n, snd, rcv), T, g, n, snd, rcv)


def test_schedule_rejects_bad_graphs():
    assert build(7, 2, 4, [0, 1], [2, 1]) is None      # receivers not sorted
    assert build(7, 2, 4, [0, 9], [1, 2]) is None      # sender out of range
    assert build(7, 2, 4, [0, 1], [1, 4]) is None      # receiver out of range
