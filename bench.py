#!/usr/bin/env python
"""Benchmark of the streaming tensor-product convolution on B200.

One step = one pass of the whole hot path over one synthetic workload: forward, first
backward (all four adjoints) and double backward (all five outputs), each called through
the C ABI.  `value` is edges per second of a whole step with inputs resident in HBM;
`orders` gives edges/s of each differentiation order on its own; `e2e` is the same step
with host buffers (pinned host -> device copies of every floating-point input and
device -> host copies of every output inside the timed region).

Prints one JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import synth  # noqa: E402

METRIC = "edges/s (one step = fwd + bwd + double-bwd)"
FP32_FMA_LANES = 148 * 128            # SMs x FP32 lanes
L2_FLUSH_BYTES = 512 << 20

DTYPE = "f32 storage; products as split bf16 x3 (hi*hi + lo*hi + hi*lo) with f32 accumulation (tcgen05)"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of an edge-kernel class, measured with
# ncu on the named profile at 20,000 nodes and stored per edge of the launch (a launch of these classes processes
# the edges of one node chunk once; its traffic grows in proportion to them).  At this profile the stream's figure is
# the state of the chunk written once (0.92 MB per node as bf16 hi + lo, i.e. 23 KB per edge at 40 edges per node)
# plus the gathered sender rows.
NCU_TRAFFIC_BYTES_PER_EDGE = {
    ("cfg5", "edge_stream_state"): (719.4e6 + 2082.7e6) / 90891.0,     # k_stream_tc, two launches
    ("cfg5", "edge_pass"): (359.0e6 + 15.3e6) / 90891.0,                # k_edge_tc, three launches
}
STATE_BUDGET_MIB = None         # --state-budget-mib: the plan's scratch budget (None = the library's default, 2048)
STREAM_CALLS_PER_STEP = 7      # edge-stream passes over all edges per step: 1 fwd + 2 bwd + 4 dbwd


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "sm_max_mhz": d.get("sm_max_mhz", 1965.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "sm_max_mhz": 1965.0, "source": "fallback"}


def work_model(plan):
    """Algorithmic multiply-adds per edge / per node of each order, from the path table."""
    K = plan.info.K
    KF = KFt = CG = CGt = Gf = Gt = 0
    for k in range(plan.info.n_paths):
        p = plan.path(k)
        di, do = 2 * p.l_in + 1, 2 * p.l_out + 1
        nnz = int((np.abs(plan.cg(k)) > 0).sum())
        if plan.mode == "uvu":
            # channelwise mode: the cheapest form of every pass is the direct one, K multiply-adds for the edge's weight
            # of a channel and path plus d_in d_out for the contraction with the coupling matrix (both directions);
            # passes that still go through the K-expanded state do more than this count credits them for
            KF += K * p.c_in
            KFt += K * p.c_in
            CG += p.c_in * di * do
            CGt += p.c_in * di * do
        else:
            KF += K * p.c_in * do
            KFt += K * p.c_out * di
            CG += p.c_in * nnz
            CGt += p.c_out * nnz
        co = 1 if plan.mode == "uvu" else p.c_out      # tied multiplicities: no sum over a second channel index
        Gf += K * p.c_in * co * do
        Gt += K * p.c_in * co * di
    edge = {"fwd": KF + CG, "bwd": 3 * KF + KFt + 3 * CG + CGt, "dbwd": 8 * KF + 3 * KFt + 5 * CG + 2 * CGt}
    node = {"fwd": Gf, "bwd": 2 * Gf + Gt, "dbwd": 5 * Gf + 2 * Gt}
    # split of the edge work between the two edge-stream kernel classes
    cls = {"edge_stream_state": (KF + CG) + (KF + CG + KFt + CGt) + (3 * KF + 2 * CG + 3 * KFt + 2 * CGt),
           "edge_pass": (2 * KF + 2 * CG) + (5 * KF + 3 * CG),
           "fused_stream_gemm": 0}
    # algorithmic HBM bytes per edge and step of the same classes (edge inputs read once per launch, one gathered
    # feature row per edge; the bounded state and the node-sized outputs are not edge-sized and not counted)
    i = plan.info
    e_in = 4 * i.dim_sh + 4 * K
    b_r, b_s = 4 + e_in + 4 * i.C_x, 8 + e_in + 4 * i.C_y
    cls_bytes = {"edge_stream_state": 3 * b_r + (4 + 2 * e_in + 8 * i.C_x) + 2 * b_s + (8 + 2 * e_in + 4 * i.C_y),
                 # gphi / gY (hphi / hY) written, the dual pass reads both copies of the edge inputs and of x
                 "edge_pass": 2 * (b_r + e_in) + (4 + 3 * e_in + 8 * i.C_x),
                 "fused_stream_gemm": 0}
    return edge, node, cls, cls_bytes


def aggregate_over_ranks(dist, device, step_ms, e2e_ms, order_ms, E):
    """Replicas only: every rank times its own copy of the workload.  The job's step time is the MAX over the ranks
    (the slowest replica), its work the SUM of the ranks' edges.  `dist` is torch.distributed with an initialised
    process group, or None for a single process.  Returns (step_ms, e2e_ms, order_ms[3], E_total)."""
    if dist is None:
        return float(step_ms), float(e2e_ms), np.asarray(order_ms, dtype=np.float64), float(E)
    import torch
    v = torch.tensor([step_ms, e2e_ms] + list(order_ms), device=device, dtype=torch.float64)
    dist.all_reduce(v, op=dist.ReduceOp.MAX)
    es = torch.tensor([E], device=device, dtype=torch.float64)
    dist.all_reduce(es, op=dist.ReduceOp.SUM)
    return float(v[0]), float(v[1]), v[2:].cpu().numpy(), float(es[0])


class ClockSampler:
    def __init__(self, device_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={device_index}", f"--query-gpu={q}",
                                       "--format=csv,noheader,nounits", "-lms", "25"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.strip()]
        os.unlink(self.f.name)
        sm, names = [], ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in rows:
            try:
                sm.append(float(r[0]))
                out["sm_max_mhz"] = float(r[1])
                for nm, v in zip(names, r[3:7]):
                    if v.strip().lower().startswith("active"):
                        reasons.add(nm)
            except (ValueError, IndexError):
                pass
        if sm:
            out["sm_mhz"] = statistics.median(sm)
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


def oracle_sample_rate(w, d, oracle, target_s=15.0):
    """Times the fp64 oracle (fwd + bwd + dbwd) on a contiguous receiver sample and returns
    (edges/s, edges in the sample, seconds, per-order seconds)."""
    def run(act):
        t = {}
        t0 = time.perf_counter()
        oracle.fwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, act=act)
        t["fwd"] = time.perf_counter() - t0
        t0 = time.perf_counter()
        oracle.bwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, d.gy, act=act)
        t["bwd"] = time.perf_counter() - t0
        t0 = time.perf_counter()
        oracle.dbwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, d.gy, d.vx, d.vY, d.vphi, d.vR, act=act)
        t["dbwd"] = time.perf_counter() - t0
        return t

    from oracle import conv as oconv
    cores = oconv.threads()
    n0 = min(d.N, max(2 * cores, 16))
    t = run(np.arange(n0))
    tot = sum(t.values())
    n1 = int(min(d.N, max(n0, n0 * target_s / max(tot, 1e-6))))
    if n1 > 2 * n0:
        t = run(np.arange(n1))
        n0 = n1
        tot = sum(t.values())
    edges = int(d.row_ptr[n0] - d.row_ptr[0])
    return edges / tot, edges, tot, t, n0, cores


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import conv as oconv
    w = synth.config(args.workload)
    oracle = oconv.Oracle(w.irreps_in, w.irreps_out, w.l_max, w.K, mode=w.mode)
    d = synth.make_inputs(w, oracle.col_std())
    cores = oconv.threads()
    # one step = fwd+bwd+dbwd on a bounded contiguous receiver sample
    n = min(d.N, max(8 * cores, 64))
    act = np.arange(n)
    edges = int(d.row_ptr[n] - d.row_ptr[0])

    def step():
        oracle.fwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, act=act)
        oracle.bwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, d.gy, act=act)
        oracle.dbwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, d.gy, d.vx, d.vY, d.vphi, d.vR, act=act)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    val = edges / dt
    sample = f"{n} contiguous receivers ({edges} edges) of {w.name} per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "edges/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "N": d.N, "E": d.E, "sample": sample},
        "cpu_baseline": {"value": val, "unit": "edges/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "edges/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


class Run:
    """One workload resident on the device, with the three calls of a step bound to its buffers."""

    def __init__(self, sb, torch, dev, w, seed):
        self.sb, self.torch, self.dev, self.w = sb, torch, dev, w
        self.plan = plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K, mode=w.mode, state_budget_mib=STATE_BUDGET_MIB)
        w.seed = seed
        self.d = d = synth.make_inputs(w, synth.plan_col_std(plan))
        self.info = i = plan.info
        self.N, self.E = N, E = d.N, d.E
        self.host = {k: torch.from_numpy(np.ascontiguousarray(getattr(d, k))).pin_memory()
                     for k in ("x", "Y", "phi", "R", "gy", "vx", "vY", "vphi", "vR")}
        torch.cuda.reset_peak_memory_stats(dev)
        self.base_alloc = torch.cuda.memory_allocated(dev)
        self.t = {k: v.to(dev) for k, v in self.host.items()}
        rp = torch.from_numpy(d.row_ptr.astype(np.int64)).to(dev)
        col = torch.from_numpy(d.col.astype(np.int32)).to(dev)
        sp, perm = sb.graph_prepare(rp, col)
        recv = sb.graph_receivers(rp, perm)
        self.g = sb.make_graph(rp, col, sp, perm, recv)
        self.in_bytes = torch.cuda.memory_allocated(dev) - self.base_alloc
        new = lambda *s: torch.empty(*s, dtype=torch.float32, device=dev)
        self.out = {"y": new(N, i.C_y), "gx": new(N, i.C_x), "gY": new(E, i.dim_sh), "gphi": new(E, i.K),
                    "gR": new(i.K, i.N_w), "ggy": new(N, i.C_y), "hx": new(N, i.C_x), "hY": new(E, i.dim_sh),
                    "hphi": new(E, i.K), "hR": new(i.K, i.N_w)}
        self.out_bytes = sum(v.numel() * 4 for v in self.out.values())
        self.ws_bytes = sb.workspace_bytes(plan, N, E, 2)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        self.flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def run_orders(self, tt, oo, which=(0, 1, 2)):
        sb, plan, g, ws = self.sb, self.plan, self.g, self.ws
        if 0 in which:
            sb.conv_fwd(plan, g, tt["x"], tt["Y"], tt["phi"], tt["R"], oo["y"], ws)
        if 1 in which:
            sb.conv_bwd(plan, g, tt["x"], tt["Y"], tt["phi"], tt["R"], tt["gy"], oo["gx"], oo["gY"], oo["gphi"],
                        oo["gR"], ws)
        if 2 in which:
            sb.conv_dbwd(plan, g, tt["x"], tt["Y"], tt["phi"], tt["R"], tt["gy"], tt["vx"], tt["vY"], tt["vphi"],
                         tt["vR"], oo["ggy"], oo["hx"], oo["hY"], oo["hphi"], oo["hR"], ws)

    def timed_step(self):
        """One step; returns per-order device milliseconds.  L2 is flushed (a buffer larger than L2 is
        overwritten) before every order, outside the event brackets."""
        torch = self.torch
        evs = []
        for o in (0, 1, 2):
            self.flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            self.run_orders(self.t, self.out, (o,))
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize(self.dev)
        return [a.elapsed_time(b) for a, b in evs]

    def class_times(self, steps):
        """{kernel class: (device ms, launches)} over `steps` steps, CUDA events around every launch."""
        self.sb.timing_enable(True)
        for _ in range(steps):
            for o in (0, 1, 2):
                self.flush.fill_(1)
                self.run_orders(self.t, self.out, (o,))
        self.torch.cuda.synchronize(self.dev)
        self.sb.timing_enable(False)
        return self.sb.timing_collect()


ORDER_NAMES = ("fwd", "bwd", "dbwd")


def side_table(sb, torch, dev, names, steps=5, warmup=3):
    """The other single-GPU configurations, measured in the same process with the same protocol (median of
    `steps` steps after `warmup`): edges/s per order and per step, and the edge-stream class time."""
    rows = {}
    for name in names:
        r = Run(sb, torch, dev, synth.config(name), 0)
        for _ in range(warmup):
            r.timed_step()
        per = np.array([r.timed_step() for _ in range(steps)])
        assert sb.last_device_status(r.ws) == 0
        cls = r.class_times(2)
        _, _, cls_w, _ = work_model(r.plan)
        ms = np.median(per, axis=0)
        st_ms = cls["edge_stream_state"][0] / 2
        rows[r.w.name] = {
            "N": r.N, "E": r.E, "ms_per_step": float(np.median(per.sum(axis=1))),
            "edges_per_s": {nm: r.E / (m * 1e-3) for nm, m in zip(ORDER_NAMES, ms)},
            "step_edges_per_s": r.E / (float(np.median(per.sum(axis=1))) * 1e-3),
            "edge_stream_state_tflops": 2.0 * cls_w["edge_stream_state"] * r.E / (st_ms * 1e-3) / 1e12 if st_ms > 0 else None,
            "workspace_bytes": int(r.ws_bytes), "steps": steps}
        del r
        torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-table", action="store_true", help="skip the table of the other configurations")
    ap.add_argument("--state-budget-mib", type=int, default=0,
                    help="scratch budget of the plan in MiB (0 = the library default, 2048); a throughput knob")
    ap.add_argument("--nodes", type=int, default=0,
                    help="run the workload's profile on a graph scaled to this many nodes (same density and degree): for profiler captures")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    global STATE_BUDGET_MIB
    STATE_BUDGET_MIB = args.state_budget_mib if args.state_budget_mib > 0 else None
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2607_18074_b200 as sb
    sb.lib()   # fails loudly if the CUDA library is missing
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod

    # replicas only: every rank runs the same workload on its own GPU (different seed per rank)
    wl = synth.config(args.workload)
    if args.nodes > 0:
        wl = synth.scaled(wl, args.nodes)
    r = Run(sb, torch, dev, wl, rank)
    w, plan, i, N, E, t, out, ws, g, host, flush = r.w, r.plan, r.info, r.N, r.E, r.t, r.out, r.ws, r.g, r.host, r.flush
    host_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in out.items()}

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        r.timed_step()
    assert sb.last_device_status(ws) == 0
    peak_bytes = torch.cuda.max_memory_allocated(dev) - r.base_alloc

    # ---- timed region: exactly K steps; every step is one sample, the reported time is their median ----
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    l0 = sb.launch_count()
    per = []
    wall0 = time.perf_counter()
    for _ in range(args.steps):
        per.append(r.timed_step())
    barrier()
    wall = time.perf_counter() - wall0
    launches = sb.launch_count() - l0
    per = np.array(per)                                  # [steps, 3] device ms
    step_ms = float(np.median(per.sum(axis=1)))
    step_ms_mean = float(per.sum(axis=1).mean())
    order_ms = np.median(per, axis=0)

    # ---- per-kernel-class device time over a few more steps (events around every launch)
    cls_steps = min(args.steps, 5)
    classes = r.class_times(cls_steps)
    clocks = sampler.stop() if sampler else None

    # ---- the FP32 multiply-add rate of this GPU, measured for about a second, with the SM clock sampled meanwhile
    fp32_peak, fp32_clock = None, None
    if rank == 0:
        cs = ClockSampler(local)
        fp32_peak = sb.measure_fp32_peak(1.0)
        fp32_clock = cs.stop()

    # ---- backward after a retaining forward (extra figure, not part of the step): the forward leaves the receiver
    # state in the workspace when all nodes fit one chunk, and the backward then skips its own edge stream for gR
    bwd_retained_ms = None
    if world == 1:
        ms = []
        for _ in range(4):
            kept = sb.conv_fwd_retain(plan, g, t["x"], t["Y"], t["phi"], t["R"], out["y"], ws)
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            sb.conv_bwd_retained(plan, g, t["x"], t["Y"], t["phi"], t["R"], t["gy"], out["gx"], out["gY"], out["gphi"],
                                 out["gR"], ws, kept)
            b.record()
            torch.cuda.synchronize(dev)
            ms.append(a.elapsed_time(b))
        bwd_retained_ms = (float(np.median(ms[1:])), int(kept))

    # ---- geometry front end (extra figure, not part of the step): the same forward and backward with Y and phi
    # recomputed from the edge vectors inside the edge kernels; outputs gx, the edge-vector adjoint and gR
    geo = None
    if world == 1 and w.mode == "uvw":
        try:
            pos = torch.from_numpy(np.ascontiguousarray(r.d.pos, dtype=np.float32)).to(dev)
            rvec, g_rv = torch.empty(E, 3, device=dev), torch.empty(E, 3, device=dev)
            sb.edge_vectors(g, pos, rvec)
            basis = sb.BASIS_BESSEL if w.basis == "bessel" else sb.BASIS_GAUSSIAN
            calls = (lambda: sb.conv_geo_fwd(plan, g, rvec, basis, w.r_c, 6, t["x"], t["R"], out["y"], ws),
                     lambda: sb.conv_geo_bwd(plan, g, rvec, basis, w.r_c, 6, t["x"], t["R"], t["gy"], out["gx"], g_rv,
                                             out["gR"], ws))
            geo_ms = []
            for f in calls:
                ms = []
                for _ in range(4):
                    flush.fill_(1)
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(); f(); b.record()
                    torch.cuda.synchronize(dev)
                    ms.append(a.elapsed_time(b))
                geo_ms.append(float(np.median(ms[1:])))
            assert sb.last_device_status(ws) == 0
            geo = {"fwd_edges_per_s": E / (geo_ms[0] * 1e-3), "bwd_edges_per_s": E / (geo_ms[1] * 1e-3),
                   "fwd_ms": geo_ms[0], "bwd_ms": geo_ms[1], "edge_input_bytes_per_edge": 12,
                   "stored_edge_input_bytes_per_edge": 4 * (i.dim_sh + i.K)}
            del pos, rvec, g_rv
        except sb.SobekError as e:       # profiles without the tensor-core edge kernels have no geometry mode
            geo = {"unavailable": str(e)}

    # ---- end to end: host buffers in, host buffers out ---------------------------------
    # Every step copies all of its inputs from pinned host memory and all of its outputs back, through the public
    # API.  Where device memory allows a second set of input / output buffers, the copies run on two copy streams
    # and overlap the previous / next step's kernels (double buffering); otherwise everything is serial.
    run_orders = r.run_orders
    h2d = sum(v.numel() * 4 for v in host.values())
    d2h = r.out_bytes
    free_b, _ = torch.cuda.mem_get_info(dev)
    pipelined = free_b > 1.25 * (h2d + d2h) + (1 << 30)
    if pipelined:
        t_sets = [t, {k: torch.empty_like(v) for k, v in t.items()}]
        o_sets = [out, {k: torch.empty_like(v) for k, v in out.items()}]
        s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        main = torch.cuda.current_stream(dev)

        def e2e_run(n):
            in_ready = [torch.cuda.Event(), torch.cuda.Event()]
            done = [torch.cuda.Event(), torch.cuda.Event()]
            with torch.cuda.stream(s_in):                      # inputs of step 0
                s_in.wait_stream(main)
                for k, v in host.items():
                    t_sets[0][k].copy_(v, non_blocking=True)
                in_ready[0].record(s_in)
            for i in range(n):
                cur = i & 1
                flush.fill_(1)
                main.wait_event(in_ready[cur])
                if i >= 2:
                    main.wait_stream(s_out)                    # the outputs of step i-2 have left o_sets[cur]
                run_orders(t_sets[cur], o_sets[cur])
                done[cur].record(main)
                with torch.cuda.stream(s_out):                 # outputs of step i go back while step i+1 runs
                    s_out.wait_event(done[cur])
                    for k, v in o_sets[cur].items():
                        host_out[k].copy_(v, non_blocking=True)
                if i + 1 < n:
                    with torch.cuda.stream(s_in):              # inputs of step i+1 come in while step i runs
                        if i >= 1:
                            s_in.wait_event(done[1 - cur])     # step i-1 no longer reads t_sets[1-cur]
                        for k, v in host.items():
                            t_sets[1 - cur][k].copy_(v, non_blocking=True)
                        in_ready[1 - cur].record(s_in)
            main.wait_stream(s_out)
            main.wait_stream(s_in)
    else:
        def e2e_run(n):
            for _ in range(n):
                flush.fill_(1)
                for k, v in host.items():
                    t[k].copy_(v, non_blocking=True)
                run_orders(t, out)
                for k, v in out.items():
                    host_out[k].copy_(v, non_blocking=True)

    e2e_run(2)
    torch.cuda.synchronize(dev)
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    e2e_run(args.steps)
    b.record()
    barrier()
    e2e_ms = a.elapsed_time(b) / args.steps
    assert sb.last_device_status(ws) == 0

    # ---- max over ranks ------------------------------------------------------------------
    step_ms, e2e_ms, order_ms, E_total = aggregate_over_ranks(dist, dev, step_ms, e2e_ms, order_ms, E)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    edge_w, node_w, cls_w, cls_b = work_model(plan)
    # dominant kernel class and its roofline
    tot_cls = sum(v[0] for v in classes.values()) or 1.0
    dom = max(classes, key=lambda k: classes[k][0])
    dom_ms, dom_launches = classes[dom]
    steps_timed = cls_steps
    alu_derived = FP32_FMA_LANES * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12       # TFLOP/s at max clock
    alu_peak = fp32_peak if fp32_peak else alu_derived
    traffic_pe = NCU_TRAFFIC_BYTES_PER_EDGE.get((w.name.split("_N")[0], dom))
    # edges of one launch = edges of one node chunk = E / chunks, chunks = stream launches per pass over the edges
    n_chunks = max(1.0, classes["edge_stream_state"][1] / steps_timed / STREAM_CALLS_PER_STEP) if "edge_stream_state" in classes else 1.0
    traffic = None if traffic_pe is None else traffic_pe * E / n_chunks
    if dom == "node_gemm":
        # the node contractions stream the bounded state once per pass (4 bytes per state element as bf16
        # hi + lo, read or written): HBM-bound; passes per step: 8 over the receiver state, 3 over the sender state
        info = plan.info
        nbytes = 4.0 * (8 * info.state_floats_fwd + 3 * info.state_floats_bwd) * N * steps_timed
        achieved = nbytes / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else 0.0
        roofline = {"kernel": dom, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "traffic": traffic,
                    "peak_source": f"HBM copy bandwidth, {peaks['source']}"}
    else:
        # the edge kernels: algorithmic multiply-adds of the method per edge against the FP32 multiply-add rate
        # measured on this GPU in this run (the tensor-core kernels move the part of the work that scales with the
        # multiplicity off those pipes, so the fraction may pass 1); beside it the same launches' algorithmic HBM
        # bytes against the measured copy bandwidth
        fmas = cls_w.get(dom, 0) * E * steps_timed
        achieved = 2.0 * fmas / (dom_ms * 1e-3) / 1e12 if dom_ms > 0 else 0.0
        hbm = cls_b.get(dom, 0) * E * steps_timed / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else 0.0
        roofline = {"kernel": dom, "bound": "alu", "achieved": achieved, "peak": alu_peak, "unit": "TFLOP/s",
                    "frac": achieved / alu_peak, "traffic": traffic,
                    "peak_source": ("measured: independent FP32 fused multiply-add chains on all SMs for 1 s, CUDA events"
                                    if fp32_peak else "derived"),
                    "peak_derived": alu_derived,
                    "peak_derived_source": f"148 SMs x 128 FP32 lanes x 2 x {peaks['sm_max_mhz']:.0f} MHz",
                    "frac_of_derived": achieved / alu_derived,
                    "fp32_peak_clocks": fp32_clock,
                    "hbm": {"algorithmic_gbs": hbm, "peak_gbs": peaks["hbm_gbs"], "frac": hbm / peaks["hbm_gbs"],
                            "peak_source": f"copy bandwidth, {peaks['source']}"}}
    roofline.update({
                "avg_launch_ms": dom_ms / max(dom_launches, 1), "launches": int(dom_launches),
                "share_of_kernel_time": dom_ms / tot_cls,
                "classes": {k: {"ms_per_step": v[0] / steps_timed, "launches_per_step": v[1] / steps_timed}
                            for k, v in classes.items()}})

    res = {
        "metric": METRIC, "value": E_total / (step_ms * 1e-3), "unit": "edges/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": w.name, "mode": w.mode, "N": N, "E": E, "K": i.K, "N_w": int(i.N_w), "C_x": i.C_x, "C_y": i.C_y,
                   "state_budget_mib": STATE_BUDGET_MIB or 2048,
                   "l_max": i.l_max, "replicas": world, "l2": f"flushed before every order ({L2_FLUSH_BYTES >> 20} MiB write)",
                   "timing": "every step is one sample (CUDA events per order); ms_per_step and the per-order times are medians"},
        "ms_per_step_mean": step_ms_mean, "timed_ms_total": float(per.sum()),
        "orders": {nm: {"edges_per_s": E_total / (ms * 1e-3), "ms": float(ms),
                        "edge_fma_per_edge": edge_w[nm], "node_fma_per_node": node_w[nm]}
                   for nm, ms in zip(ORDER_NAMES, order_ms)},
        "e2e": {"value": E_total / (e2e_ms * 1e-3), "unit": "edges/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                "copies": "double-buffered on two copy streams" if pipelined else "serial"},
        "bwd_after_retaining_fwd": None if bwd_retained_ms is None else {
            "edges_per_s": E_total / (bwd_retained_ms[0] * 1e-3), "ms": bwd_retained_ms[0], "state_retained": bwd_retained_ms[1]},
        "geometry_front_end": geo,
        "gpu_launches": int(launches),
        "wall_s_timed_region": wall,
        "peak_bytes": {"total": int(peak_bytes), "inputs_and_graph": int(r.in_bytes), "outputs": int(r.out_bytes),
                       "workspace": int(r.ws_bytes), "l2_flush_buffer": L2_FLUSH_BYTES},
        "roofline": roofline,
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        from oracle import conv as oconv
        oracle = oconv.Oracle(w.irreps_in, w.irreps_out, w.l_max, w.K, mode=w.mode)
        rate, edges, secs, tt, nrecv, cores = oracle_sample_rate(w, r.d, oracle)
        res["cpu_baseline"] = {"value": rate, "unit": "edges/s", "cores": cores, "kind": "oracle",
                               "sample": f"first {nrecv} receivers ({edges} edges) of {w.name}, fwd+bwd+dbwd, {secs:.1f} s",
                               "seconds": {k: round(v, 3) for k, v in tt.items()}}
    if world == 1 and not args.no_table and args.workload == "cfg5":
        # the other single-GPU configurations, same process and protocol
        del t, out, ws, g, host, flush, host_out, run_orders
        if pipelined:
            del t_sets, o_sets
        del r
        torch.cuda.empty_cache()
        res["other_configs"] = side_table(sb, torch, dev, ["cfg2", "cfg3", "cfg4_1e6"])
    print(json.dumps(res))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
