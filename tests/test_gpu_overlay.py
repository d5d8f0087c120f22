"""A signature outside the committed list, built as an overlay (build.py --signatures), against the oracle (GPU)."""
import json
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

SCRIPT = r"""
import pathlib, sys, dataclasses
import numpy as np, torch
sys.path.insert(0, r'{root}'); sys.path.insert(0, r'{root}/tests')
import paper_2609_35099_b200 as e3j
e3j._LIB_PATH = pathlib.Path(r'{lib}')
from oracle import conv as oconv
from paper_2609_35099_b200 import workloads
from parity_util import assert_blockwise_close, blocks_of_paths
t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
# first: automatic parameters (edge-wise backward); second: the entry switches the edge-wise backward off, so its
# backward is the path-group kernel that signatures too large for the edge-wise layout fall back to
for irreps, lmax in (('32x0e+32x1o', 2), ('32x0e+32x1o+32x2e', 2)):
    wl = dataclasses.replace(workloads.make_graph(2, 300), irreps_in=irreps, sh_lmax=lmax, out_lmax=lmax)
    plan = e3j.e3j_plan_create(irreps, lmax, None, lmax)
    assert plan.specialised == 1
    cp = oconv.Coupling(irreps, lmax, None, lmax)
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    snd, rcv = t(wl.senders), t(wl.receivers)
    runs = []
    for _ in range(2):
        out = e3j.e3j_conv_fwd(plan, t(x), t(y), t(w), snd, rcv)
        runs.append((out, *e3j.e3j_conv_bwd(plan, t(x), t(y), t(w), snd, rcv, t(g))))
    torch.cuda.synchronize()
    assert e3j.e3j_plan_device_status(plan) == 0
    assert all(torch.equal(a, b) for a, b in zip(*runs)), 'results differ between two runs'
    out, gx, gy, gw = runs[0]
    ref = oconv.conv_fwd(cp, x, y, w, wl.senders, wl.receivers)
    rx, ry, rw = oconv.conv_bwd(cp, x, y, w, wl.senders, wl.receivers, g)
    for got, want, kind in ((out, ref, 'out'), (gx, rx, 'x'), (gy, ry, 'sh'), (gw, rw, 'w')):
        assert_blockwise_close(got.cpu().numpy(), want, blocks_of_paths(cp.paths, kind), what=kind)
print('overlay parity ok')
"""


def test_overlay_signature_matches_the_oracle(repo_root, tmp_path):
    sig = [{"name": "w32_l2", "irreps_in": "32x0e+32x1o", "sh_lmax": 2, "irreps_out": None, "out_lmax": 2},
           {"name": "t32_l2_pathgroups", "irreps_in": "32x0e+32x1o+32x2e", "sh_lmax": 2, "irreps_out": None,
            "out_lmax": 2, "ET": 0}]
    (tmp_path / "extra.json").write_text(json.dumps(sig))
    lib = tmp_path / "libe3j_overlay.so"
    subprocess.run([sys.executable, "-m", "paper_2609_35099_b200.build", "--signatures", str(tmp_path / "extra.json"),
                    "--out", str(lib)], check=True, cwd=repo_root, capture_output=True)
    done = subprocess.run([sys.executable, "-c", SCRIPT.format(root=repo_root, lib=lib)], cwd=repo_root,
                          capture_output=True, text=True)
    assert done.returncode == 0 and "overlay parity ok" in done.stdout, done.stdout + done.stderr
