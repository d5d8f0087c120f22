"""The allocation-free forward entry point against the workspace-taking one (GPU).

e3j_conv_fwd_noalloc serves callers that cannot obtain device memory at call time (engines that
reserve everything at start-up and forbid allocation in their step loop, plug-ins without an
allocator): its scratch is a static array inside the library.  This file is collected last so that
a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2609_35099_b200 as e3j
from oracle import conv as oconv
from paper_2609_35099_b200 import workloads
from parity_util import assert_blockwise_close, blocks_of_paths

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_noalloc_forward_matches_workspace_forward_twice():
    c = workloads.CONFIGS[2]
    wl = workloads.make_graph(2, n_atoms=648)  # 6^3 water molecules: several tiles and ragged range ends per CTA
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    assert plan.specialised == 1
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    x, y, w, _ = workloads.make_features(wl, plan.n_paths, plan.d_out)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    dx, dy, dw, snd, rcv = t(x), t(y), t(w), t(wl.senders), t(wl.receivers)
    want = e3j.e3j_conv_fwd(plan, dx, dy, dw, snd, rcv)
    blocks = blocks_of_paths(cp.paths, "out")
    out = torch.empty_like(want)
    for call in range(2):  # the shared scratch keeps the previous call's contents: the second call must not care
        out.fill_(float("nan"))
        e3j.e3j_conv_fwd_noalloc(plan, dx, dy, dw, snd, rcv, out)
        torch.cuda.synchronize()
        assert_blockwise_close(out.cpu().numpy(), want.cpu().numpy().astype(np.float64), blocks,
                               what=f"noalloc call {call}")
    assert e3j.e3j_noalloc_status() == 0   # no bounded wait gave up (the word is static, like the scratch)
    # and the reference entry point itself agrees with the oracle on this graph
    ref = oconv.conv_fwd(cp, x, y, w, wl.senders, wl.receivers)
    assert_blockwise_close(want.cpu().numpy(), ref, blocks, what="workspace forward")
    # a different graph right after: stale scratch from the larger problem must not leak in
    wl2 = workloads.make_graph(2, n_atoms=192)
    x2, y2, w2, _ = workloads.make_features(wl2, plan.n_paths, plan.d_out)
    a2 = [t(v) for v in (x2, y2, w2, wl2.senders, wl2.receivers)]
    want2 = e3j.e3j_conv_fwd(plan, *a2)
    out2 = torch.full_like(want2, float("nan"))
    e3j.e3j_conv_fwd_noalloc(plan, *a2, out2)
    assert_blockwise_close(out2.cpu().numpy(), want2.cpu().numpy().astype(np.float64), blocks, what="noalloc second graph")


def test_noalloc_forward_on_the_signature_closest_to_the_scratch_limit():
    """64x(0e+1o+2e+3o): 156 output rows, the largest need of the generated signatures (23.7 of the 24 MiB on
    148 SMs) and the one-channel-per-lane consumer layout."""
    c = workloads.CONFIGS[3]
    wl = workloads.make_graph(3, n_atoms=250)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    assert plan.specialised == 1
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], None, c["out_lmax"])
    x, y, w, _ = workloads.make_features(wl, plan.n_paths, plan.d_out)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    args = [t(v) for v in (x, y, w, wl.senders, wl.receivers)]
    want = e3j.e3j_conv_fwd(plan, *args)
    blocks = blocks_of_paths(cp.paths, "out")
    for call in range(2):
        out = torch.full_like(want, float("nan"))
        e3j.e3j_conv_fwd_noalloc(plan, *args, out)
        assert_blockwise_close(out.cpu().numpy(), want.cpu().numpy().astype(np.float64), blocks, what=f"noalloc call {call}")
    assert e3j.e3j_noalloc_status() == 0


def test_noalloc_rejects_plans_without_specialised_kernels_and_handles_empty_graphs():
    generic = e3j.e3j_plan_create("8x0e+8x1o", 2, "0e+1o+1e+2e+2o")
    x = torch.zeros((4, generic.d_in, generic.n_channels), device=DEV)
    e_i = torch.zeros(0, dtype=torch.int32, device=DEV)
    out = torch.ones((4, generic.d_out, generic.n_channels), device=DEV)
    with pytest.raises(e3j.E3JError) as err:
        e3j.e3j_conv_fwd_noalloc(generic, x, torch.zeros((0, generic.d_sh), device=DEV),
                                 torch.zeros((0, generic.n_paths, generic.n_channels), device=DEV), e_i, e_i, out)
    assert err.value.status == -4
    plan = e3j.e3j_plan_create("128x0e+128x1o", 3, None, 3)
    x = torch.zeros((4, plan.d_in, plan.n_channels), device=DEV)
    out = torch.ones((4, plan.d_out, plan.n_channels), device=DEV)
    e3j.e3j_conv_fwd_noalloc(plan, x, torch.zeros((0, plan.d_sh), device=DEV),
                             torch.zeros((0, plan.n_paths, plan.n_channels), device=DEV), e_i, e_i, out)
    assert torch.count_nonzero(out) == 0
