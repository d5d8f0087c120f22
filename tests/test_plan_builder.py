"""Host logic of libe3j (CPU only): the library loads, exports every declared symbol, and its
plan builder (ladder-operator coefficients) agrees with the oracle (Racah closed form)."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2609_35099_b200 as e3j
from oracle import cg


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2609_35099_b200 import build
    build.build()


def test_library_exports_every_declared_symbol(repo_root):
    header = open(os.path.join(repo_root, "include", "e3j.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(e3j_[a-z0-9_]+)\s*\(", header))
    assert {"e3j_plan_create", "e3j_conv_fwd", "e3j_conv_bwd", "e3j_plan_destroy", "e3j_tp_fwd",
            "e3j_tp_bwd", "e3j_graph_prepare"} <= names
    lib = ctypes.CDLL(str(e3j.library_path()))
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} declared in e3j.h but not exported"


SIGNATURES = [
    ("8x0e+8x1o", 2, "0e+1o+1e+2e+2o", -1),
    ("128x0e+128x1o", 3, None, 3),
    ("128x0e+128x1o", 3, "0e+1o+2e+3o", -1),
    ("64x0e+64x1o+64x2e+64x3o", 3, None, 3),
    ("128x0e+128x1o+128x2e", 3, None, 3),
    ("4x0e+4x0o+4x1o+4x1e+4x2e+4x2o", 2, None, 4),
    ("2x3o+2x4e", 2, None, -1),
]


@pytest.mark.parametrize("sig", SIGNATURES)
def test_ladder_coefficients_equal_racah_coefficients(sig):
    irreps_in, lmax, irreps_out, out_lmax = sig
    plan = e3j.e3j_plan_create(irreps_in, lmax, irreps_out, out_lmax)
    C, i3, paths, nq = cg.dense_coupling(irreps_in, lmax, irreps_out, None if out_lmax < 0 else out_lmax)
    info = e3j.e3j_plan_info(plan)
    assert (info["n_channels"], info["d_in"], info["d_sh"], info["n_paths"], info["d_out"]) == \
        (nq, C.shape[1], C.shape[2], len(paths), C.shape[0])
    assert info["nnz"] == np.count_nonzero(C)
    assert info["n_pairs"] == np.count_nonzero(np.abs(C).sum(axis=2))
    i0, i1, i2, k, val = e3j.e3j_plan_records(plan)
    dense = np.zeros_like(C)
    dense[i0, i1, i2] = val
    assert np.abs(dense - C).max() < 1e-13
    assert np.array_equal(k, i3[i0])
    order = np.lexsort((i2, i1, i0))
    assert np.array_equal(order, np.arange(len(i0)))  # sorted by (i0, i1, i2)
    for got, want in zip(e3j.e3j_plan_paths(plan), paths):
        assert (got["in_index"], got["l1"], got["p1"], got["l2"], got["L"], got["p"], got["x_off"],
                got["y_off"], got["out_off"]) == \
            (want.in_index, want.l1, want.p1, want.l2, want.L, want.p, want.x_off, want.y_off, want.out_off)


def test_high_degree_ladder_blocks_match_racah():
    lib = ctypes.CDLL(str(e3j.library_path()))  # noqa: F841  (loads the builder)
    for l1, l2, outs in [(5, 4, "1e+4e+9e"), (6, 6, "0e+6e+12e"), (8, 3, "5o+8o+11o")]:
        plan = e3j.e3j_plan_create(f"1x{l1}e", l2, outs, -1)
        i0, i1, i2, k, val = e3j.e3j_plan_records(plan)
        for p in e3j.e3j_plan_paths(plan):
            if p["l2"] != l2:
                continue
            blk = cg.real_cg_block(l1, l2, p["L"])
            sel = k == e3j.e3j_plan_paths(plan).index(p)
            dense = np.zeros_like(blk)
            dense[i0[sel] - p["out_off"], i1[sel], i2[sel] - p["y_off"]] = val[sel]
            assert np.abs(dense - blk).max() < 1e-12


@pytest.mark.parametrize("bad,status", [
    ("", -2), ("8x", -2), ("8x0z", -2), ("8x0e++8x1o", -2), ("8x0e+4x1o", -3), ("1x9e", -4)])
def test_bad_descriptors_return_status_codes(bad, status):
    with pytest.raises(e3j.E3JError) as err:
        e3j.e3j_plan_create(bad, 2)
    assert err.value.status == status


def test_no_coupling_path_is_an_error():
    with pytest.raises(e3j.E3JError) as err:
        e3j.e3j_plan_create("4x0e", 1, "3e")
    assert err.value.status == -4


def test_status_strings():
    assert e3j.e3j_status_string(0) == "ok"
    assert "workspace" in e3j.e3j_status_string(-5)


def test_compute_calls_fail_loudly_without_a_device():
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    plan = e3j.e3j_plan_create("4x0e+4x1o", 1)
    x = torch.zeros((2, 4, 4))
    with pytest.raises(TypeError):
        e3j.e3j_tp_fwd(plan, x, torch.zeros((2, 4)), torch.zeros((2, plan.n_paths, 4)))
    # straight through the C ABI with non-null dummy pointers: the CUDA error surfaces as a status
    lib = e3j._load()
    dummy = ctypes.c_void_p(256)
    st = lib.e3j_tp_fwd(plan.handle, 1, dummy, dummy, dummy, dummy, None)
    assert st == -6


@pytest.mark.parametrize("sig", [("8x0e+8x1o", 2, "0e+1o+1e+2e+2o", -1), ("128x0e+128x1o", 3, None, 3),
                                 ("64x0e+64x1o+64x2e+64x3o", 3, None, 3)])
def test_collapsed_plan_tables(sig):
    """E3J_PLAN_COLLAPSE_OUTPUTS: same paths, records and weights, output rows shared per (L, parity)."""
    from oracle import conv as oconv
    irreps_in, lmax, irreps_out, out_lmax = sig
    full = e3j.e3j_plan_create(irreps_in, lmax, irreps_out, out_lmax)
    plan = e3j.e3j_plan_create(irreps_in, lmax, irreps_out, out_lmax, e3j.E3J_PLAN_COLLAPSE_OUTPUTS)
    cp = oconv.Coupling(irreps_in, lmax, irreps_out, None if out_lmax < 0 else out_lmax)
    R, offs = oconv.collapse_matrix(cp)
    assert plan.n_paths == full.n_paths and plan.d_out == R.shape[0]
    # (only the 128-channel water-box signature has generated kernels for its collapsed form)
    assert plan.specialised == (irreps_in == "128x0e+128x1o" and irreps_out is None)
    assert [p["out_off"] for p in e3j.e3j_plan_paths(plan)] == offs
    i0, i1, i2, k, val = e3j.e3j_plan_records(plan)
    keys = list(zip(i0.tolist(), k.tolist(), i1.tolist(), i2.tolist()))
    assert keys == sorted(keys)   # sorted by (i0, path, i1, i2): the order the kernel generator relies on
    dense = np.zeros((R.shape[0], cp.d, cp.dp, cp.P))
    dense[i0, i1, i2, k] = val
    want = np.zeros_like(dense)
    for p, off in zip(cp.paths, offs):
        want[off:off + 2 * p.L + 1, :, :, p.k] = cp.C[p.out_off:p.out_off + 2 * p.L + 1]
    assert np.abs(dense - want).max() < 1e-13
    assert e3j.e3j_plan_signature(plan) != e3j.e3j_plan_signature(full)


def test_generated_kernel_sources_are_up_to_date(repo_root):
    """The specialised kernels are generated from signatures.json and the plan builder's records; the files in
    the tree must be what the generator writes today (a stale file would be compiled silently)."""
    import subprocess
    import sys
    gen = os.path.join(repo_root, "paper_2609_35099_b200", "csrc", "gen_fast.py")
    done = subprocess.run([sys.executable, gen, "--check"], capture_output=True, text=True, cwd=repo_root)
    assert done.returncode == 0, done.stdout + done.stderr


def test_every_generated_signature_is_picked_up_by_its_plan(repo_root):
    """A plan created from the descriptors of a signature in signatures.json selects the generated kernels."""
    import json
    path = os.path.join(repo_root, "paper_2609_35099_b200", "csrc", "fast", "signatures.json")
    for sig in json.load(open(path)):
        flags = e3j.E3J_PLAN_COLLAPSE_OUTPUTS if sig.get("collapse") else 0
        plan = e3j.e3j_plan_create(sig["irreps_in"], sig["sh_lmax"], sig["irreps_out"], sig["out_lmax"], flags)
        assert plan.specialised, sig["name"]
        generic = e3j.e3j_plan_create(sig["irreps_in"], sig["sh_lmax"], sig["irreps_out"], sig["out_lmax"],
                                      flags | e3j.E3J_PLAN_GENERIC_ONLY)
        assert not generic.specialised


def test_every_generated_signature_fits_the_allocation_free_scratch(repo_root):
    """e3j_conv_fwd_noalloc keeps the forward's boundary-row scratch in a 24 MiB static array: 8 KB of receiver ids
    plus two partial rows (D x N_q floats) per CTA, FC CTAs per SM.  Every signature in signatures.json must fit
    on a 148-SM device (the one closest to the limit is the 156-row config-3 signature)."""
    import json
    import sys
    sys.path.insert(0, os.path.join(repo_root, "paper_2609_35099_b200", "csrc"))
    import gen_fast
    sigs = json.load(open(os.path.join(repo_root, "paper_2609_35099_b200", "csrc", "fast", "signatures.json")))
    worst = 0
    for s in sigs:
        if "V" not in s:   # tile parameters chosen by the generator
            s = {**gen_fast.auto_params(s, gen_fast.load_records(s)[0]), **s}
        flags = e3j.E3J_PLAN_COLLAPSE_OUTPUTS if s.get("collapse") else 0
        plan = e3j.e3j_plan_create(s["irreps_in"], s["sh_lmax"], s["irreps_out"], s["out_lmax"], flags)
        need = 8192 + 4 * 2 * (148 * s["FC"]) * plan.d_out * plan.n_channels
        worst = max(worst, need)
        assert need <= 24 << 20, (s["name"], need)
    assert worst > 20 << 20   # the bound is tight: a new, larger signature must raise the array, not pass by luck


def test_overlay_build_generates_kernels_for_a_signature_outside_the_list(repo_root, tmp_path):
    """build.py --signatures: a signature that is not in signatures.json gets generated kernels (tile parameters
    chosen by the generator) in a library of its own; the committed library keeps using the table-driven ones."""
    import json
    import subprocess
    import sys
    sig = [{"name": "w32_l2", "irreps_in": "32x0e+32x1o", "sh_lmax": 2, "irreps_out": None, "out_lmax": 2}]
    (tmp_path / "extra.json").write_text(json.dumps(sig))
    out = tmp_path / "libe3j_overlay.so"
    subprocess.run([sys.executable, "-m", "paper_2609_35099_b200.build", "--signatures", str(tmp_path / "extra.json"),
                    "--out", str(out)], check=True, cwd=repo_root, capture_output=True)
    assert e3j.e3j_plan_create("32x0e+32x1o", 2, None, 2).specialised == 0
    probe = ("import pathlib, paper_2609_35099_b200 as e3j; e3j._LIB_PATH = pathlib.Path(r'%s'); "
             "print(e3j.e3j_plan_create('32x0e+32x1o', 2, None, 2).specialised, "
             "e3j.e3j_plan_create('128x0e+128x1o', 3, None, 3).specialised)" % out)
    done = subprocess.run([sys.executable, "-c", probe], check=True, cwd=repo_root, capture_output=True, text=True)
    assert done.stdout.split() == ["1", "1"]
