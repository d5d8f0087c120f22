"""The generated per-edge bodies of the specialised kernels, compiled for the host and run lane by lane on one
edge, against the oracle: a generator mistake (a wrong slot, a dropped pair, a transposed operand) shows up
without a GPU.  The runners in host_kernel_shim.hpp do what the kernels' warps do around the bodies."""
import ctypes
import json
import os
import subprocess

import numpy as np
import pytest

from oracle import conv as oconv

HERE = os.path.dirname(os.path.abspath(__file__))
FAST = os.path.join(os.path.dirname(HERE), "paper_2609_35099_b200", "csrc", "fast")
SIGS = json.load(open(os.path.join(FAST, "signatures.json")))


def _host_library(sig, tmp_path):
    text = open(os.path.join(FAST, f"sig_{sig['name']}.cu")).read()
    begin = text.index("namespace e3j {")
    end = text.index("}  // namespace\n}  // namespace fast")     # closes the anonymous namespace after the struct
    body = text[begin:end] + "}  // namespace\n}  // namespace fast\n}  // namespace e3j\n"
    name = f"e3j::fast::Sig_{sig['name']}"
    src = tmp_path / f"host_{sig['name']}.cpp"
    src.write_text(
        '#include "host_kernel_shim.hpp"\n' + body + '#define E3J_HOST_RUNNERS\n#include "host_kernel_shim.hpp"\n'
        f'using S = {name};\n'
        'extern "C" {\n'
        'void fwd(const float* x, const float* y, const float* s, float* out) { host_run::fwd<S>(x, y, s, out); }\n'
        'void bwd_groups(const float* x, const float* y, const float* s, const float* g, float* dx, float* dy, float* ds)'
        ' { host_run::bwd_groups<S>(x, y, s, g, dx, dy, ds); }\n'
        'void bwd_all(const float* x, const float* y, const float* s, const float* g, float* dx, float* dy, float* ds)'
        ' { host_run::bwd_all<S>(x, y, s, g, dx, dy, ds); }\n'
        'void dbl(const float* x, const float* y, const float* s, const float* g, const float* ux, const float* uy,'
        ' const float* us, float* gg, float* dx, float* dy, float* ds)'
        ' { host_run::dbl<S>(x, y, s, g, ux, uy, us, gg, dx, dy, ds); }\n'
        'int has_bwd_all() { return S::ET > 0 || S::ETR > 0; }\n'
        'int has_dbl() { return S::DT > 0 && S::DFT > 0; }\n'
        '}\n')
    lib = tmp_path / f"host_{sig['name']}.so"
    subprocess.run(["g++", "-std=c++17", "-O1", "-shared", "-fPIC", "-I", HERE, str(src), "-o", str(lib)], check=True)
    return ctypes.CDLL(str(lib))


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _close(got, want, what):
    scale = np.abs(want).max()
    assert scale > 0, what
    err = np.abs(got.astype(np.float64) - want).max() / scale
    assert err < 1e-5, (what, err)


@pytest.mark.parametrize("sig", SIGS, ids=[s["name"] for s in SIGS])
def test_generated_bodies_match_the_oracle_on_one_edge(sig, tmp_path):
    lib = _host_library(sig, tmp_path)
    olm = sig["out_lmax"] if sig["irreps_out"] is None else None
    cp = oconv.Coupling(sig["irreps_in"], sig["sh_lmax"], sig["irreps_out"], olm)
    collapsed = bool(sig.get("collapse"))
    rng = np.random.default_rng(5)
    mul = int(sig["irreps_in"].split("x")[0])
    d_in = sum(2 * int(t.split("x")[1][:-1]) + 1 for t in sig["irreps_in"].split("+"))
    d_sh = (sig["sh_lmax"] + 1) ** 2
    n_paths = len(cp.paths)
    x = rng.standard_normal((1, d_in, mul)).astype(np.float32)
    y = rng.standard_normal((1, d_sh)).astype(np.float32)
    s = rng.standard_normal((1, n_paths, mul)).astype(np.float32)
    zero = np.zeros(1, np.int32)
    ref_out = (oconv.conv_fwd_collapsed if collapsed else oconv.conv_fwd)(cp, x, y, s, zero, zero)
    d_out = ref_out.shape[1]
    g = rng.standard_normal((1, d_out, mul)).astype(np.float32)
    rx, ry, rs = (oconv.conv_bwd_collapsed if collapsed else oconv.conv_bwd)(cp, x, y, s, zero, zero, g)

    out = np.zeros((d_out, mul), np.float32)
    lib.fwd(_ptr(x), _ptr(y), _ptr(s), _ptr(out))
    _close(out, ref_out[0], "forward body")

    for entry in ("bwd_groups", "bwd_all"):
        if entry == "bwd_all" and not lib.has_bwd_all():
            continue
        dx, dy, ds = np.zeros((d_in, mul), np.float32), np.zeros(d_sh, np.float32), np.zeros((n_paths, mul), np.float32)
        getattr(lib, entry)(_ptr(x), _ptr(y), _ptr(s), _ptr(g), _ptr(dx), _ptr(dy), _ptr(ds))
        _close(dx, rx[0], entry + " grad_x share")
        _close(dy, ry[0], entry + " grad_sh")
        _close(ds, rs[0], entry + " grad_w")

    if lib.has_dbl() and not collapsed:
        ux = rng.standard_normal(x.shape).astype(np.float32)
        uy = rng.standard_normal(y.shape).astype(np.float32)
        us = rng.standard_normal(s.shape).astype(np.float32)
        want = oconv.conv_bwd_bwd(cp, x, y, s, zero, zero, g, ux, uy, us)
        gg = np.zeros((d_out, mul), np.float32)
        dx, dy, ds = np.zeros((d_in, mul), np.float32), np.zeros(d_sh, np.float32), np.zeros((n_paths, mul), np.float32)
        lib.dbl(_ptr(x), _ptr(y), _ptr(s), _ptr(g), _ptr(ux), _ptr(uy), _ptr(us), _ptr(gg), _ptr(dx), _ptr(dy), _ptr(ds))
        for got, ref, what in ((gg, want[0], "gg_out"), (dx, want[1], "g_x"), (dy, want[2], "g_sh"), (ds, want[3], "g_w")):
            _close(got, ref[0], "double backward " + what)
