#!/usr/bin/env python
"""Benchmark of the fused equivariant convolution (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2|3|5]

One *step* is one pass of the whole hot path over one batch of synthetic input: e3j_conv_fwd
followed by e3j_conv_bwd (all three gradients) on the 3000-atom water box (128x0e+128x1o,
harmonics l<=3, 13 paths; about 161 k edges), graph already prepared.  `value` is edges per
second for that step with every input resident in HBM; `e2e` is the same metric with pinned HOST
buffers copied in and all results copied back inside the timed region.  Inputs (1.05 GB of
weights per step) exceed the 126 MB L2, so no explicit flush is needed between iterations.

With N > 1 (torchrun) every rank processes its own independent water box (no data-path
collective): weak scaling, value = total edges / max-over-ranks time.

--impl reference times the CPU oracle (plain fp64 loops, OpenMP) on a bounded sample of the same
workload; it is a deliberately slow program and only a reported baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6650 GB/s, earlier pool measurement)"


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per call from the ncu captures summarised in
# profiles/fast_fwd_kernel_water3000.txt, profiles/fast_bwd1_kernel_water3000.txt and the launch-list run
# (specialised kernels, workload water3000).  Other workloads / the generic kernels report null.
NCU_TRAFFIC = {
    ("water3000", "fwd"): 1.109735e9 + 0.085159e9 + 0.016343e9,          # fast_fwd_kernel + fwd_fixup_kernel
    ("water3000", "bwd"): 1.261320e9 + 1.362697e9 + 0.330463e9 + 0.0018e9,  # fast_bwd1_kernel + bwd_dx_reduce_kernel
}
# Where each term above is printed (file under profiles/, kernel, metric): tests/test_bench_traffic.py checks them.
NCU_TRAFFIC_SOURCE = {
    ("water3000", "fwd"): [("fast_fwd_kernel_water3000.txt", "fast_fwd_kernel", "dram__bytes_read.sum", 1.109735e9),
                           ("fast_fwd_kernel_water3000.txt", "fast_fwd_kernel", "dram__bytes_write.sum", 0.085159e9),
                           ("small_kernels_traffic_water3000.txt", "fwd_fixup_kernel", "total", 0.016343e9)],
    ("water3000", "bwd"): [("fast_bwd1_kernel_water3000.txt", "fast_bwd1_kernel", "dram__bytes_read.sum", 1.261320e9),
                           ("fast_bwd1_kernel_water3000.txt", "fast_bwd1_kernel", "dram__bytes_write.sum", 1.362697e9),
                           ("small_kernels_traffic_water3000.txt", "bwd_dx_reduce_kernel", "total", 0.330463e9 + 0.0018e9)],
}


def algorithmic_bytes(n, e, d, dp, P, D, nq):
    """Minimal bytes with the paper's accounting (inputs + outputs, no scratch, no residuals)."""
    x, y, s, idx = n * d * nq * 4, e * dp * 4, e * P * nq * 4, 2 * e * 4
    out = n * D * nq * 4
    fwd = x + y + s + idx + out
    bwd = (x + y + s + idx + out) + (x + y + s)  # primals + output cotangent read, three cotangents written
    return fwd, bwd


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons, power = [], [], set(), []
        for line in out.strip().splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "power_w_max": max(power), "samples": len(sm)}


def call_stats(ms):
    srt = sorted(ms)
    k = max(1, len(srt) // 5)
    return {"median": statistics.median(srt), "mean_fastest_20pct": statistics.mean(srt[:k]), "min": srt[0],
            "max": srt[-1], "mean": statistics.mean(srt)}


def oracle_sample(wl, cp, x, y, w, g, n_rows):
    """Sub-problem made of the first n_rows receivers (their edges are a prefix of the edge list)."""
    n_rows = min(n_rows, wl.n_nodes)
    e = int(np.searchsorted(wl.receivers, n_rows, side="left"))
    return dict(x=x, y=y[:e], w=w[:e], snd=wl.senders[:e], rcv=wl.receivers[:e], g=g, edges=e, rows=n_rows)


def time_oracle(cp, smp):
    from oracle import conv as oconv
    t0 = time.perf_counter()
    oconv.conv_fwd(cp, smp["x"], smp["y"], smp["w"], smp["snd"], smp["rcv"])
    t1 = time.perf_counter()
    oconv.conv_bwd(cp, smp["x"], smp["y"], smp["w"], smp["snd"], smp["rcv"], smp["g"])
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def build_workload(config):
    from paper_2609_35099_b200 import workloads
    c = workloads.CONFIGS[config]
    wl = workloads.make_graph(config)
    return c, wl


def run_reference(args, rank):
    """The oracle as it stands, timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    from oracle import conv as oconv
    from paper_2609_35099_b200 import workloads
    c, wl = build_workload(args.config)
    cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    x, y, w, g = workloads.make_features(wl, cp.P, cp.D)
    probe = oracle_sample(wl, cp, x, y, w, g, 64)
    tf, tb = time_oracle(cp, probe)
    per_edge = (tf + tb) / max(probe["edges"], 1)
    budget = 120.0 / max(args.steps + args.warmup, 1)  # whole run within a couple of minutes
    rows = int(min(wl.n_nodes, max(64, budget / per_edge / (wl.n_edges / wl.n_nodes))))
    smp = oracle_sample(wl, cp, x, y, w, g, rows)
    for _ in range(args.warmup):
        time_oracle(cp, smp)
    t0 = time.perf_counter()
    fwd_s = 0.0
    for _ in range(args.steps):
        a, b = time_oracle(cp, smp)
        fwd_s += a
    total = time.perf_counter() - t0
    value = smp["edges"] * args.steps / total
    sample = f"first {smp['rows']} receivers of {wl.name} ({smp['edges']} of {wl.n_edges} edges), fwd+bwd, fp64"
    line = {
        "impl": "reference", "metric": "conv_fwd_bwd_edges_per_s", "value": value, "unit": "edges/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{wl.name} (sample)", "sample": sample, "n_nodes": wl.n_nodes, "n_edges": wl.n_edges},
        "fwd_edges_per_s": smp["edges"] * args.steps / fwd_s,
        "cpu_baseline": {"value": value, "unit": "edges/s", "cores": oconv.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "edges/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_tp(args, e3j, workloads, torch, dev, rank, world, barrier):
    """Secondary workload: the standalone tensor product (rows are their own senders and receivers).

    The arrays are tens of GB at 2^20 rows, so they are drawn on the device with a seeded generator; there is
    no end-to-end or CPU leg for this workload (the headline workload carries those).
    """
    import torch.distributed as dist
    c = workloads.CONFIGS[4]
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"],
                               e3j.E3J_PLAN_GENERIC_ONLY if args.generic else 0)
    rows, nq = args.rows, plan.n_channels
    gen = torch.Generator(device=dev)
    gen.manual_seed(4 + rank)
    x1 = torch.randn((rows, plan.d_in, nq), device=dev, generator=gen)
    x2 = torch.randn((rows, plan.d_sh), device=dev, generator=gen)
    w = torch.randn((rows, plan.n_paths, nq), device=dev, generator=gen)
    g = torch.randn((rows, plan.d_out, nq), device=dev, generator=gen)
    out = torch.empty_like(g)
    g1, g2, gw = torch.empty_like(x1), torch.empty_like(x2), torch.empty_like(w)
    stream = torch.cuda.current_stream()
    fwd = lambda: e3j.e3j_tp_fwd(plan, x1, x2, w, out=out)
    bwd = lambda: e3j.e3j_tp_bwd(plan, x1, x2, w, g, grad_x1=g1, grad_x2=g2, grad_w=gw)
    for _ in range(args.warmup):
        fwd(); bwd()
    torch.cuda.synchronize()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    marks = [(ev(), ev(), ev()) for _ in range(args.steps)]
    sampler = ClockSampler(dev.index) if rank == 0 else None
    launches0 = e3j.e3j_launch_count()
    barrier(); torch.cuda.synchronize()
    for a, b, cc in marks:
        a.record(stream); fwd(); b.record(stream); bwd(); cc.record(stream)
    torch.cuda.synchronize(); barrier()
    launches = e3j.e3j_launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    total_ms = marks[0][0].elapsed_time(marks[-1][2])
    if world > 1:
        tm = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tm, op=dist.ReduceOp.MAX)
        total_ms = float(tm.item())
    if rank != 0:
        return
    f_ms = statistics.mean(a.elapsed_time(b) for a, b, _ in marks)
    b_ms = statistics.mean(b.elapsed_time(cc) for _, b, cc in marks)
    peak, peak_src = measured_peak()
    prim = 4 * rows * (plan.d_in * nq + plan.d_sh + plan.n_paths * nq)
    fb = prim + 4 * rows * plan.d_out * nq
    bb = fb + prim

    def roof(nbytes, ms, kernel):
        ach = nbytes / (ms * 1e-3) / 1e9
        return {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS, "peak_source": peak_src,
                "algorithmic_bytes_per_launch": nbytes, "avg_ms": ms, "traffic": None}

    roofs = {"fwd": roof(fb, f_ms, "e3j_tp_fwd call"), "bwd": roof(bb, b_ms, "e3j_tp_bwd call")}
    ms_per_step = total_ms / args.steps
    print(json.dumps({
        "metric": "tp_fwd_bwd_rows_per_s", "value": rows * world / (ms_per_step * 1e-3), "unit": "rows/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic (seeded device generator)",
        "config": {"workload": f"tp rows={rows} {c['irreps_in']} (x) l<={c['sh_lmax']}", "rows_per_gpu": rows,
                   "specialised_kernels": bool(plan.specialised), "l2": "inputs larger than L2"},
        "clocks": clocks, "e2e": None, "gpu_launches": launches, "fwd_ms": f_ms, "bwd_ms": b_ms,
        "roofline": roofs["bwd"] if b_ms >= f_ms else roofs["fwd"], "roofline_fwd": roofs["fwd"],
        "roofline_bwd": roofs["bwd"], "cpu_baseline": None}), flush=True)


def run_sharded(args, e3j, workloads, torch, dev, rank, world, barrier):
    """One system cut by receiver over the ranks: a step = all-gather of the owned x rows + halo row gather,
    e3j_conv_fwd and e3j_conv_bwd on the local problem, all-gather of the halo's grad_x shares + ordered adds."""
    import torch.distributed as dist
    from paper_2609_35099_b200 import sharding
    c, wl = build_workload(args.config)
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
    n, e = wl.n_nodes, wl.n_edges
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    ops = sharding.CudaOps(plan)
    rowptr_h = np.searchsorted(wl.receivers, np.arange(n + 1), side="left")
    if world == 1:   # the exchange needs a process group: a group of one
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1"); os.environ.setdefault("MASTER_PORT", "29517")
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    sh = sharding.make_shard(ops, rank, world, n, torch.from_numpy(wl.senders).to(dev), torch.from_numpy(wl.receivers).to(dev),
                             rowptr_h)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    x_owned, ys, ws_ = t(x[sh.lo:sh.hi]), t(y[sh.e_lo:sh.e_hi]), t(w[sh.e_lo:sh.e_hi])
    g_local = torch.zeros((sh.n_local, plan.d_out, plan.n_channels), device=dev)
    g_local[:sh.n_owned] = t(g[sh.lo:sh.hi])
    graph = ops.graph_prepare(sh.n_local, sh.senders, sh.receivers)
    e_loc = sh.e_hi - sh.e_lo
    out = torch.empty((sh.n_local, plan.d_out, plan.n_channels), device=dev)
    gxl = torch.empty((sh.n_local, plan.d_in, plan.n_channels), device=dev)
    gy, gw = torch.empty_like(ys), torch.empty_like(ws_)
    ws_f = torch.empty(max(e3j.e3j_conv_fwd_workspace_bytes(plan, sh.n_local, e_loc), 256), dtype=torch.uint8, device=dev)
    ws_b = torch.empty(max(e3j.e3j_conv_bwd_workspace_bytes(plan, sh.n_local, e_loc), 256), dtype=torch.uint8, device=dev)

    def step():
        x_local = sharding.gather_x(ops, sh, x_owned)
        ops.conv_fwd(x_local, ys, ws_, sh.senders, sh.receivers, graph, out=out, workspace=ws_f)
        ops.conv_bwd(x_local, ys, ws_, sh.senders, sh.receivers, g_local, graph, grad_x=gxl, grad_sh=gy, grad_w=gw,
                     workspace=ws_b)
        return sharding.reduce_grad_x(ops, sh, gxl)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(dev.index) if rank == 0 else None
    l0 = e3j.e3j_launch_count()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize()
    a.record(stream)
    for _ in range(args.steps):
        step()
    b.record(stream)
    torch.cuda.synchronize(); barrier()
    launches = e3j.e3j_launch_count() - l0
    clocks = sampler.stop() if sampler else None
    tm = torch.tensor([a.elapsed_time(b)], device=dev, dtype=torch.float64)
    dist.all_reduce(tm, op=dist.ReduceOp.MAX)
    ms_per_step = float(tm.item()) / args.steps
    if rank == 0:
        print(json.dumps({
            "metric": "conv_fwd_bwd_edges_per_s", "value": e / (ms_per_step * 1e-3), "unit": "edges/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name + " (receiver-sharded)", "n_nodes": n, "n_edges": e,
                       "parallelism": f"receivers cut into {world} ranges by edge count; x halo all-gather, grad_x shares added in rank order",
                       "halo_nodes_rank0": int(sh.halo_ids.numel()), "owned_nodes_rank0": sh.n_owned,
                       "l2": "inputs exceed the L2 at one rank; no explicit flush"},
            "clocks": clocks, "e2e": None, "gpu_launches": int(launches), "roofline": None, "cpu_baseline": None}), flush=True)
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[2, 3, 4, 5],
                    help="2 = headline workload; 3 / 5 = other convolution workloads; 4 = standalone tensor product rows")
    ap.add_argument("--rows", type=int, default=1 << 20, help="rows of the tensor-product workload (--config 4)")
    ap.add_argument("--generic", action="store_true", help="force the table-driven generic kernels")
    ap.add_argument("--collapse", action="store_true",
                    help="plan with collapsed output multiplicities (table-driven kernels; no CPU leg)")
    ap.add_argument("--pad", type=float, default=0.0,
                    help="append this fraction of padding edges and call the padded entry points (rates count real edges)")
    ap.add_argument("--double-backward", action="store_true", help="(default for configs 2 and 3; kept for old command lines)")
    ap.add_argument("--no-double-backward", action="store_true",
                    help="skip the timing of e3j_conv_bwd_bwd (after the steps, reported beside them; plain lists only)")
    ap.add_argument("--sustained-s", type=float, default=2.0,
                    help="length of the extra back-to-back loop whose means and clocks go into `sustained` (0 = skip)")
    ap.add_argument("--fused-radial", action="store_true",
                    help="also time the convolution that takes the radial network's last layer (h, W) instead of the "
                         "weights (after the steps, reported beside them); default for configs 2 and 3")
    ap.add_argument("--no-radial", action="store_true", help="skip the radial-layer timings")
    ap.add_argument("--hidden", type=int, default=64, help="width of the radial network's last hidden layer")
    ap.add_argument("--shard", action="store_true",
                    help="one system sharded by receiver over the ranks (halo exchange of x and grad_x inside the step) "
                         "instead of one system per rank; strong scaling")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist

    import paper_2609_35099_b200 as e3j
    from paper_2609_35099_b200 import workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()

    if args.config == 4:
        run_tp(args, e3j, workloads, torch, dev, rank, world, barrier)
        return
    if args.shard:
        run_sharded(args, e3j, workloads, torch, dev, rank, world, barrier)
        return

    c, wl = build_workload(args.config)
    t_plan = time.perf_counter()
    plan = e3j.e3j_plan_create(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"],
                               (e3j.E3J_PLAN_GENERIC_ONLY if args.generic else 0) |
                               (e3j.E3J_PLAN_COLLAPSE_OUTPUTS if args.collapse else 0))
    if args.collapse:
        args.no_cpu_baseline = True
    plan_build_ms = 1e3 * (time.perf_counter() - t_plan)   # host: paths, ladder-operator CG, record tables
    n, e = wl.n_nodes, wl.n_edges
    x, y, w, g = workloads.make_features(wl, plan.n_paths, plan.d_out)
    snd_h, rcv_h = wl.senders, wl.receivers
    n_pad = int(round(args.pad * e))
    if n_pad:
        # padding entries: receiver id = n_nodes (the padding mark), the rest arbitrary
        y = np.concatenate([y, np.zeros((n_pad, y.shape[1]), np.float32)])
        w = np.concatenate([w, np.zeros((n_pad,) + w.shape[1:], np.float32)])
        snd_h = np.concatenate([snd_h, np.zeros(n_pad, np.int32)])
        rcv_h = np.concatenate([rcv_h, np.full(n_pad, n, np.int32)])
    e_buf = e + n_pad
    host = dict(x=x, y=y, w=w, g=g, snd=snd_h, rcv=rcv_h)
    pinned = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in host.items()}
    d = {k: v.to(dev) for k, v in pinned.items()}
    stream = torch.cuda.current_stream()
    prepare = e3j.e3j_graph_prepare_padded if n_pad else e3j.e3j_graph_prepare
    conv_fwd = e3j.e3j_conv_fwd_padded if n_pad else e3j.e3j_conv_fwd
    conv_bwd = e3j.e3j_conv_bwd_padded if n_pad else e3j.e3j_conv_bwd
    rowptr, perm, colptr = prepare(n, d["snd"], d["rcv"])
    # graph preparation is once per neighbour list and not part of the step; timed on its own
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record(stream)
    for _ in range(5):
        prepare(n, d["snd"], d["rcv"])
    g1.record(stream)
    torch.cuda.synchronize()
    graph_prepare_ms = g0.elapsed_time(g1) / 5
    out = torch.empty((n, plan.d_out, plan.n_channels), device=dev)
    gx = torch.empty((n, plan.d_in, plan.n_channels), device=dev)
    gy = torch.empty((e_buf, plan.d_sh), device=dev)
    gw = torch.empty((e_buf, plan.n_paths, plan.n_channels), device=dev)
    ws_f = torch.empty(max(e3j.e3j_conv_fwd_workspace_bytes(plan, n, e_buf), 256), dtype=torch.uint8, device=dev)
    ws_b = torch.empty(max(e3j.e3j_conv_bwd_workspace_bytes(plan, n, e_buf), 256), dtype=torch.uint8, device=dev)

    def fwd(t):
        conv_fwd(plan, t["x"], t["y"], t["w"], t["snd"], t["rcv"], rowptr, out=out, workspace=ws_f)

    def bwd(t):
        conv_bwd(plan, t["x"], t["y"], t["w"], t["snd"], t["rcv"], t["g"], rowptr, perm, colptr,
                         grad_x=gx, grad_sh=gy, grad_w=gw, workspace=ws_b)

    for _ in range(args.warmup):
        fwd(d); bwd(d)
    torch.cuda.synchronize()

    # ---- device-resident timing: exactly K steps between two synchronisation points
    ev = lambda: torch.cuda.Event(enable_timing=True)
    marks = [(ev(), ev(), ev()) for _ in range(args.steps)]
    sampler = ClockSampler(local_rank) if rank == 0 else None
    launches0 = e3j.e3j_launch_count()
    barrier(); torch.cuda.synchronize()
    t_begin, t_end = ev(), ev()
    t_begin.record(stream)
    for a, b, cc in marks:
        a.record(stream); fwd(d); b.record(stream); bwd(d); cc.record(stream)
    t_end.record(stream)
    torch.cuda.synchronize(); barrier()
    launches = e3j.e3j_launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    total_ms = t_begin.elapsed_time(t_end)
    fwd_ms = [a.elapsed_time(b) for a, b, _ in marks]
    bwd_ms = [b.elapsed_time(cc) for _, b, cc in marks]
    if world > 1:
        tm = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tm, op=dist.ReduceOp.MAX)
        total_ms = float(tm.item())
    ms_per_step = total_ms / args.steps

    # ---- the same step back to back for at least two seconds: the forward is bound by instruction issue and follows
    # the SM clock, which the power cap lowers in long runs, so the clock dependence goes on the record whatever
    # --steps is
    sustained = None
    if args.sustained_s > 0 and world == 1:
        k_s = max(args.steps, int(args.sustained_s * 1e3 / max(ms_per_step, 1e-3)) + 1)
        marks_s = [(ev(), ev(), ev()) for _ in range(k_s)]
        samp = ClockSampler(local_rank)
        torch.cuda.synchronize()
        for a, b, cc in marks_s:
            a.record(stream); fwd(d); b.record(stream); bwd(d); cc.record(stream)
        torch.cuda.synchronize()
        clk = samp.stop()
        f_s = statistics.mean(a.elapsed_time(b) for a, b, _ in marks_s)
        b_s = statistics.mean(b.elapsed_time(cc) for _, b, cc in marks_s)
        mhz, mx = clk.get("sm_mhz"), clk.get("sm_max_mhz")
        sustained = {"steps": k_s, "seconds": marks_s[0][0].elapsed_time(marks_s[-1][2]) * 1e-3, "fwd_ms": f_s, "bwd_ms": b_s,
                     "clocks": clk,
                     "fwd_ms_at_max_clock": f_s * mhz / mx if mhz and mx else None,
                     "bwd_ms_at_max_clock": b_s * mhz / mx if mhz and mx else None}
        del marks_s

    # ---- the double backward of the same workload (not part of the step)
    dbl = None
    if not args.no_double_backward and not args.pad and not args.generic and not args.collapse and args.config in (2, 3):
        gen = torch.Generator(device=dev); gen.manual_seed(11)
        cts = [torch.randn(d[k].shape, generator=gen, device=dev) for k in ("x", "y", "w")]
        ws_d = torch.empty(max(e3j.e3j_conv_bwd_bwd_workspace_bytes(plan, n, e), 256), dtype=torch.uint8, device=dev)
        gg = torch.empty_like(out)

        def dbl_call():
            e3j.e3j_conv_bwd_bwd(plan, d["x"], d["y"], d["w"], d["snd"], d["rcv"], d["g"], rowptr, perm, colptr,
                                 cts[0], cts[1], cts[2], gg_out=gg, g_x=gx, g_sh=gy, g_w=gw, workspace=ws_d)

        for _ in range(3):
            dbl_call()
        k_dbl = max(3, min(args.steps, 50))
        l0 = e3j.e3j_launch_count()
        d0, d1 = ev(), ev()
        torch.cuda.synchronize()
        d0.record(stream)
        for _ in range(k_dbl):
            dbl_call()
        d1.record(stream)
        torch.cuda.synchronize()
        dbl = {"ms": d0.elapsed_time(d1) / k_dbl, "calls": k_dbl,
               "launches_per_call": (e3j.e3j_launch_count() - l0) // k_dbl,
               "note": "4 launches = fused sweeps (forward-shaped + fix-up, edge-wise + sender sum); "
                       "more = composition of forward and backward passes"}
        del ws_d, cts, gg

    # ---- the same convolution with the edge weights given as the radial network's last layer (h, W) instead of w:
    # the forward that forms them inside the kernel, beside the unfused form (tensor-core product into memory, then
    # the plain forward), and the backward (composed: product, convolution backward, two more products)
    radial = None
    want_radial = (args.fused_radial or args.config in (2, 3)) and not args.no_radial
    if want_radial and not args.pad and not args.collapse and not args.generic:
        H = args.hidden
        gen = torch.Generator(device=dev); gen.manual_seed(12)
        hh = torch.randn((e, H), generator=gen, device=dev)
        WW = torch.randn((H, plan.n_paths * plan.n_channels), generator=gen, device=dev) / (H ** 0.5)
        ws_rf = torch.empty(max(e3j.e3j_conv_radial_fwd_workspace_bytes(plan, n, e, H), 256), dtype=torch.uint8, device=dev)
        ws_rb = torch.empty(max(e3j.e3j_conv_radial_bwd_workspace_bytes(plan, n, e, H), 256), dtype=torch.uint8, device=dev)
        w_mat = torch.empty((e, plan.n_paths, plan.n_channels), device=dev)
        gh, gW = torch.empty_like(hh), torch.empty_like(WW)

        def timed(fn, k):
            for _ in range(3):
                fn()
            l0 = e3j.e3j_launch_count()
            a, b = ev(), ev()
            torch.cuda.synchronize()
            a.record(stream)
            for _ in range(k):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / k, (e3j.e3j_launch_count() - l0) // k

        k_r = max(3, min(args.steps, 50))
        rf_ms, rf_launches = timed(lambda: e3j.e3j_conv_radial_fwd(plan, d["x"], d["y"], hh, WW, d["snd"], d["rcv"], rowptr,
                                                                    out=out, workspace=ws_rf), k_r)
        gemm_ms, _ = timed(lambda: e3j.e3j_radial_weights(plan, hh, WW, out=w_mat), k_r)
        plain_ms, _ = timed(lambda: conv_fwd(plan, d["x"], d["y"], w_mat, d["snd"], d["rcv"], rowptr, out=out, workspace=ws_f), k_r)
        rb_ms, rb_launches = timed(lambda: e3j.e3j_conv_radial_bwd(plan, d["x"], d["y"], hh, WW, d["snd"], d["rcv"], d["g"], rowptr,
                                                                    perm, colptr, grad_x=gx, grad_sh=gy, grad_h=gh, grad_W=gW,
                                                                    workspace=ws_rb), max(3, k_r // 3))
        nq_, P_, D_ = plan.n_channels, plan.n_paths, plan.d_out
        bytes_fwd = 4 * (n * plan.d_in * nq_ + e * plan.d_sh + e * H + H * P_ * nq_ + 2 * e + n * D_ * nq_)
        fma_conv = e * (plan.n_pairs + sum(2 * p["l1"] + 1 for p in e3j.e3j_plan_paths(plan))) * nq_   # FP32 issue slots x 32 lanes
        flop_tensor = 3 * 2.0 * e * H * P_ * nq_                                                      # three TF32 products
        peak_hbm, _src = measured_peak()
        try:
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                bf16_peak = float(json.load(f)["bf16_tflops"])
        except Exception:
            bf16_peak = 1590.0
        fp32_peak = 148 * 128 * 1.965e9   # FMA lanes x max SM clock (nominal unit counts)
        radial = {
            "hidden": H, "fused_fwd_ms": rf_ms, "fused_fwd_launches": rf_launches,
            "unfused_fwd_ms": gemm_ms + plain_ms, "unfused_parts_ms": {"radial_weights": gemm_ms, "conv_fwd": plain_ms},
            "bwd_ms": rb_ms, "bwd_launches": rb_launches, "bwd_form": "composed (weights and their cotangent materialised)",
            "fwd_edges_per_s": e / (rf_ms * 1e-3),
            "roofline_fwd": {
                "minimal_bytes": bytes_fwd, "hbm_GBs": bytes_fwd / (rf_ms * 1e-3) / 1e9,
                "hbm_frac_of_measured": bytes_fwd / (rf_ms * 1e-3) / 1e9 / peak_hbm,
                "bound": "alu", "fp32_fma_per_s": fma_conv / (rf_ms * 1e-3), "fp32_peak_fma_per_s": fp32_peak,
                "fp32_issue_frac": fma_conv / (rf_ms * 1e-3) / fp32_peak,
                "tensor_tf32_TFLOPs": flop_tensor / (rf_ms * 1e-3) / 1e12,
                "tensor_frac_of_tf32_peak": flop_tensor / (rf_ms * 1e-3) / 1e12 / (0.5 * bf16_peak),
                "tensor_peak_note": "TF32 peak taken as half the measured bf16 peak (nominal ratio)"},
        }
        # The same two calls end to end from pinned host memory: with (h, W) in place of w a step moves a tenth of the
        # bytes over the bus, which is what bounds `e2e` of the headline calls.
        if not args.no_e2e and world == 1:
            keys_in = ("x", "y", "snd", "rcv", "g")
            host_in = {k: pinned[k] for k in keys_in}
            host_in["h"], host_in["W"] = hh.cpu().pin_memory(), WW.cpu().pin_memory()
            dev_res = dict(out=out, gx=gx, gy=gy, gh=gh, gW=gW)
            host_res = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in dev_res.items()}
            sets = [{k: torch.empty(v.shape, dtype=v.dtype, device=dev) for k, v in host_in.items()} for _ in range(2)]
            results = [{k: torch.empty_like(v) for k, v in dev_res.items()} for _ in range(2)]
            r_h2d = sum(v.numel() * v.element_size() for v in host_in.values())
            r_d2h = sum(v.numel() * v.element_size() for v in host_res.values())
            q_in, q_out = torch.cuda.Stream(), torch.cuda.Stream()
            done_c, done_o = [None, None], [None, None]

            def radial_step(i):
                b = i % 2
                s, r = sets[b], results[b]
                with torch.cuda.stream(q_in):
                    if done_c[b] is not None:
                        q_in.wait_event(done_c[b])
                    for k in s:
                        s[k].copy_(host_in[k], non_blocking=True)
                    arrived = torch.cuda.Event(); arrived.record(q_in)
                stream.wait_event(arrived)
                if done_o[b] is not None:
                    stream.wait_event(done_o[b])
                e3j.e3j_conv_radial_fwd(plan, s["x"], s["y"], s["h"], s["W"], s["snd"], s["rcv"], rowptr, out=r["out"],
                                        workspace=ws_rf)
                e3j.e3j_conv_radial_bwd(plan, s["x"], s["y"], s["h"], s["W"], s["snd"], s["rcv"], s["g"], rowptr, perm,
                                        colptr, grad_x=r["gx"], grad_sh=r["gy"], grad_h=r["gh"], grad_W=r["gW"],
                                        workspace=ws_rb)
                done_c[b] = torch.cuda.Event(); done_c[b].record(stream)
                with torch.cuda.stream(q_out):
                    q_out.wait_event(done_c[b])
                    for k in host_res:
                        host_res[k].copy_(r[k], non_blocking=True)
                    done_o[b] = torch.cuda.Event(); done_o[b].record(q_out)

            def radial_run(k):
                for i in range(k):
                    radial_step(i)
                for evd in done_o:
                    if evd is not None:
                        stream.wait_event(evd)

            radial_run(max(3, args.warmup)); torch.cuda.synchronize()
            k_re = max(3, min(args.steps, 50))
            a0, a1 = ev(), ev()
            a0.record(stream)
            q_in.wait_event(a0)
            radial_run(k_re)
            a1.record(stream)
            torch.cuda.synchronize()
            re_ms = a0.elapsed_time(a1) / k_re
            radial["e2e"] = {"value": e / (re_ms * 1e-3), "unit": "edges/s", "ms_per_step": re_ms, "steps": k_re,
                             "h2d_bytes_per_step": r_h2d, "d2h_bytes_per_step": r_d2h,
                             "note": "e3j_conv_radial_fwd + e3j_conv_radial_bwd from pinned host buffers, copies inside "
                                     "the timed region on streams of their own, two buffer sets"}
            del sets, results, host_res
        del ws_rf, ws_rb, w_mat, hh, WW, gh, gW

    # ---- the backward over a processing order built once per neighbour list (runs of one sender summed in registers)
    sched_block = None
    if want_radial and not args.pad and not args.collapse and not args.generic and \
            e3j.e3j_bwd_schedule_bytes(plan, n, e) > 0:
        t_b = time.perf_counter()
        sched = e3j.e3j_bwd_schedule_build(plan, n, d["snd"], d["rcv"])
        torch.cuda.synchronize()
        build_ms = (time.perf_counter() - t_b) * 1e3
        hdr = sched[:64].view(torch.int32).cpu()
        k_s = max(3, min(args.steps, 50))
        for _ in range(3):
            e3j.e3j_conv_bwd_scheduled(plan, d["x"], d["y"], d["w"], sched, d["g"], grad_x=gx, grad_sh=gy, grad_w=gw, workspace=ws_b)
        a_, b_ = ev(), ev()
        torch.cuda.synchronize()
        a_.record(stream)
        for _ in range(k_s):
            e3j.e3j_conv_bwd_scheduled(plan, d["x"], d["y"], d["w"], sched, d["g"], grad_x=gx, grad_sh=gy, grad_w=gw, workspace=ws_b)
        b_.record(stream)
        torch.cuda.synchronize()
        sb_ms = a_.elapsed_time(b_) / k_s
        sched_block = {"bwd_ms": sb_ms, "fwd_plus_bwd_ms": statistics.mean(fwd_ms) + sb_ms,
                       "fwd_plus_bwd_edges_per_s": e / ((statistics.mean(fwd_ms) + sb_ms) * 1e-3),
                       "schedule_build_ms": build_ms,
                       "schedule_build": "host (graph arrays copied to the host, order copied back), once per neighbour list",
                       "rows_written": int(hdr[5]), "edges_per_row": e / max(int(hdr[5]), 1), "tiles": int(hdr[4]),
                       "note": "e3j_conv_bwd_scheduled: same gradients, grad_x summed in another fixed order; "
                               "the headline backward is the unscheduled call"}
        del sched

    # ---- the convolution on edge vectors: harmonics formed in the kernel's table warp, beside the two-step form
    vec_block = None
    if want_radial and not args.pad and not args.collapse and not args.generic and plan.d_sh in (1, 4, 9, 16):
        lmax = int(round(plan.d_sh ** 0.5)) - 1
        vv = torch.from_numpy(wl.vectors.astype("float32")).to(dev)
        ws_vf = torch.empty(max(e3j.e3j_conv_vec_fwd_workspace_bytes(plan, n, e), 256), dtype=torch.uint8, device=dev)
        ws_vb = torch.empty(max(e3j.e3j_conv_vec_bwd_workspace_bytes(plan, n, e), 256), dtype=torch.uint8, device=dev)
        y_buf, gv = torch.empty((e, plan.d_sh), device=dev), torch.empty((e, 3), device=dev)

        def timed_v(fn, k):
            for _ in range(3):
                fn()
            a, b = ev(), ev()
            torch.cuda.synchronize()
            a.record(stream)
            for _ in range(k):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / k

        k_v = max(3, min(args.steps, 50))
        vec_block = {
            "fwd_ms": timed_v(lambda: e3j.e3j_conv_vec_fwd(plan, d["x"], vv, d["w"], d["snd"], d["rcv"], rowptr, out=out,
                                                           workspace=ws_vf), k_v),
            "harmonics_fwd_ms": timed_v(lambda: e3j.e3j_harmonics_fwd(lmax, vv, out=y_buf), k_v),
            "harmonics_bwd_ms": timed_v(lambda: e3j.e3j_harmonics_bwd(lmax, vv, d["y"], out=gv), k_v),
            "bwd_ms": timed_v(lambda: e3j.e3j_conv_vec_bwd(plan, d["x"], vv, d["w"], d["snd"], d["rcv"], d["g"], rowptr, perm,
                                                           colptr, grad_x=gx, grad_vec=gv, grad_w=gw, workspace=ws_vb), k_v),
            "note": "fwd: harmonics formed inside the convolution kernel (specialised signatures); bwd: harmonics kernel, "
                    "e3j_conv_bwd, harmonics gradient kernel",
        }
        del vv, ws_vf, ws_vb, y_buf, gv

    # ---- end to end: pinned host buffers in, results out, inside the timed region.  Every step copies its inputs
    # from pinned host memory and its four results back; the copies run on streams of their own with two sets
    # of device buffers, so that the transfers of neighbouring steps overlap each other and the kernels.
    e2e = None
    if not args.no_e2e:
        res_host = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in
                    dict(out=out, gx=gx, gy=gy, gw=gw).items()}
        nbuf = 2
        stage = [{k: torch.empty_like(v) for k, v in d.items()} for _ in range(nbuf)]
        res_dev = [dict(out=torch.empty_like(out), gx=torch.empty_like(gx), gy=torch.empty_like(gy),
                        gw=torch.empty_like(gw)) for _ in range(nbuf)]
        h2d = sum(v.numel() * v.element_size() for v in pinned.values())
        d2h = sum(v.numel() * v.element_size() for v in res_host.values())
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        comp_done, d2h_done = [None] * nbuf, [None] * nbuf

        def e2e_step(i):
            b = i % nbuf
            t, r = stage[b], res_dev[b]
            with torch.cuda.stream(s_in):
                if comp_done[b] is not None:
                    s_in.wait_event(comp_done[b])      # the kernels that read this input set are done
                for k in t:
                    t[k].copy_(pinned[k], non_blocking=True)
                arrived = torch.cuda.Event(); arrived.record(s_in)
            stream.wait_event(arrived)
            if d2h_done[b] is not None:
                stream.wait_event(d2h_done[b])         # this result set has left the device
            conv_fwd(plan, t["x"], t["y"], t["w"], t["snd"], t["rcv"], rowptr, out=r["out"], workspace=ws_f)
            conv_bwd(plan, t["x"], t["y"], t["w"], t["snd"], t["rcv"], t["g"], rowptr, perm, colptr,
                     grad_x=r["gx"], grad_sh=r["gy"], grad_w=r["gw"], workspace=ws_b)
            comp_done[b] = torch.cuda.Event(); comp_done[b].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[b])
                for k in res_host:
                    res_host[k].copy_(r[k], non_blocking=True)
                d2h_done[b] = torch.cuda.Event(); d2h_done[b].record(s_out)

        def e2e_run(k):
            for i in range(k):
                e2e_step(i)
            for evd in d2h_done:                       # the timed region ends when the last result is on the host
                if evd is not None:
                    stream.wait_event(evd)

        e2e_run(max(3, args.warmup)); torch.cuda.synchronize()   # untimed warm-up steps of the same pipeline
        k_e2e = args.steps
        barrier(); torch.cuda.synchronize()
        s0, s1 = ev(), ev()
        s0.record(stream)
        s_in.wait_event(s0)
        e2e_run(k_e2e)
        s1.record(stream)
        torch.cuda.synchronize(); barrier()
        e2e_ms = s0.elapsed_time(s1)
        if world > 1:
            tm = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
            dist.all_reduce(tm, op=dist.ReduceOp.MAX)
            e2e_ms = float(tm.item())
        e2e = {"value": e * world * k_e2e / (e2e_ms * 1e-3), "unit": "edges/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / k_e2e, "steps": k_e2e,
               "overlap": "two buffer sets; host-to-device, kernels and device-to-host of neighbouring steps overlap"}
        del stage, res_dev

    if rank == 0:
        peak, peak_src = measured_peak()
        fb, bb = algorithmic_bytes(n, e, plan.d_in, plan.d_sh, plan.n_paths, plan.d_out, plan.n_channels)
        f_ms, b_ms = statistics.mean(fwd_ms), statistics.mean(bwd_ms)

        def roof(nbytes, ms, kernel, key):
            ach = nbytes / (ms * 1e-3) / 1e9
            plain = plan.specialised and not args.pad and not args.collapse
            traffic = NCU_TRAFFIC.get((wl.name, key)) if plain else None
            r = {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s",
                 "frac": ach / peak, "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS, "peak_source": peak_src,
                 "algorithmic_bytes_per_launch": nbytes, "avg_ms": ms, "traffic": traffic}
            if traffic:   # what the memory system moved in the committed ncu capture, at this run's duration
                r["traffic_GBs"] = traffic / (ms * 1e-3) / 1e9
                r["traffic_frac_of_peak"] = r["traffic_GBs"] / peak
                r["traffic_source"] = ("committed ncu captures (not measured in this run): " +
                                       ", ".join(sorted({"profiles/" + f for f, _, _, _ in NCU_TRAFFIC_SOURCE[(wl.name, key)]})))
            return r

        spec = bool(plan.specialised)
        roofs = {"fwd": roof(fb, f_ms, "e3j_conv_fwd call: fast_fwd_kernel (97 %) + fwd_fixup_kernel" if spec
                             else "e3j_conv_fwd call: generic conv_fwd_kernel", "fwd"),
                 "bwd": roof(bb, b_ms, "e3j_conv_bwd call: fast_bwd1_kernel (89 %) + bwd_dx_reduce_kernel" if spec
                             else "e3j_conv_bwd call: generic edge + node kernels", "bwd")}
        dominant = roofs["bwd"] if b_ms >= f_ms else roofs["fwd"]
        line = {
            "metric": "conv_fwd_bwd_edges_per_s", "value": e * world / (ms_per_step * 1e-3), "unit": "edges/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "n_nodes": n, "n_edges": e, "padding_edges": n_pad, "collapsed_outputs": bool(args.collapse), "irreps_in": c["irreps_in"],
                       "sh_lmax": c["sh_lmax"], "n_paths": plan.n_paths, "d_out": plan.d_out,
                       "channels": plan.n_channels, "specialised_kernels": bool(plan.specialised),
                       "l2": "inputs (>1 GB per step) exceed the 126 MB L2; no explicit flush",
                       "parallelism": "independent systems per rank, no collective"},
            "fwd_edges_per_s": e * world / (f_ms * 1e-3), "fwd_ms": f_ms, "bwd_ms": b_ms,
            "fwd_plus_bwd_frac_of_nominal_8TBs": (fb + bb) / ((f_ms + b_ms) * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
            # per-call statistics over the timed steps: median, the paper's statistic (mean of the fastest
            # 20 % of the runs, as in its efficiency-comparison section), minimum and maximum
            "call_stats_ms": {"fwd": call_stats(fwd_ms), "bwd": call_stats(bwd_ms)},
            "outside_the_step_ms": {"plan_build_host": plan_build_ms, "graph_prepare_device": graph_prepare_ms},
            "double_backward": dbl, "radial": radial, "edge_vectors": vec_block, "scheduled_backward": sched_block, "sustained": sustained,
            "roofline": dominant, "roofline_fwd": roofs["fwd"], "roofline_bwd": roofs["bwd"],
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        }
        if world == 1 and not args.no_cpu_baseline:
            from oracle import conv as oconv
            cp = oconv.Coupling(c["irreps_in"], c["sh_lmax"], c["irreps_out"], c["out_lmax"])
            probe = oracle_sample(wl, cp, x, y, w, g, 64)
            tf, tb = time_oracle(cp, probe)
            per_edge = (tf + tb) / max(probe["edges"], 1)
            rows = int(min(n, max(64, 15.0 / per_edge / (e / n))))  # about 15 s of wall time at most
            smp = oracle_sample(wl, cp, x, y, w, g, rows)
            tf, tb = time_oracle(cp, smp)
            line["cpu_baseline"] = {
                "value": smp["edges"] / (tf + tb), "unit": "edges/s", "cores": oconv.threads(), "kind": "oracle",
                "fwd_edges_per_s": smp["edges"] / tf,
                "sample": f"first {smp['rows']} receivers of {wl.name} ({smp['edges']} of {e} edges), fwd+bwd once, fp64"}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
