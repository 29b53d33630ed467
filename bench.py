#!/usr/bin/env python
"""Benchmark of the DETOX aggregation step (vote -> hierarchical mean -> robust aggregator) on B200.

Default workload: n = 45 workers, r = 3, d = 11,173,962 (ResNet-18-sized), q = 5 ALIE attackers placed
worst-case; one step = detox_aggregate(vote -> mean over 3 sets of 5 -> Multi-Krum(f=1, m_sel=1)).
The metric is aggregation input throughput n*d*4 bytes per second.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload cfg2|cfg1|cfg3|cfg4]

With N > 1 (launched by torch.distributed.run) every rank aggregates its own independent copy of the
workload (replicas; the path has no exchange step) and rank 0 reports the sum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "aggregation_input_throughput"
UNIT = "GB/s"
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def pipeline_for(name, w, dx):
    """The DETOX leg and the direct (non-DETOX) leg of each named configuration."""
    s = w.spec
    G = s.n // s.r
    if name == "cfg1":
        return (dict(a0=dx.AGG_NONE, a1=dx.AGG_COORD_MEDIAN, f=0, m_sel=1), ("coord_median", {}))
    if name == "cfg2":
        return (dict(a0=dx.AGG_MEAN, a1=dx.AGG_MULTIKRUM, f=1, m_sel=1), ("multikrum", dict(f=5, m_sel=s.n - 5)))
    if name == "cfg3":
        return (dict(a0=dx.AGG_NONE, a1=dx.AGG_BULYAN, f=3, m_sel=1), ("bulyan", dict(f=9)))
    if name == "cfg4":
        return (dict(a0=dx.AGG_MEAN, a1=dx.AGG_COORD_MEDIAN, f=0, m_sel=1), ("coord_median", {}))
    raise ValueError(name)


ORACLE_A1 = {1: "mean", 2: "coord_median", 3: "multikrum", 4: "bulyan"}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures summarised in
# profiles/vote_kernels_cfg2.md (same kernel code; reset an entry to None when its kernel changes).
NCU_TRAFFIC_BYTES = {
    ("cfg2", "vote_mean_kernel"): 2_011_333_000 + 117_863_424,
    ("cfg3", "vote_kernel (winners only)"): 2_011_344_896 + 3_232_768,
    # config 4 holds 11.8 GB, too much for a multi-pass capture: config 2's traffic of the same streaming kernel,
    # scaled by the algorithmic bytes (12,544,000,000 / 2,145,400,704)
    ("cfg4", "vote_mean_kernel"): int((2_011_333_000 + 117_863_424) * 12_544_000_000 / 2_145_400_704),
}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={CLOCK_QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def wait_first(self, seconds: float = 5.0):
        """nvidia-smi needs a moment to start; block until it has printed its first sample."""
        t0 = time.time()
        while self.proc is not None and not self.rows and time.time() - t0 < seconds:
            time.sleep(0.02)

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for nm, v in zip(names, r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


def time_calls(torch, fn, steps, warmup):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    st = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st)
    for _ in range(steps):
        fn()
    e1.record(st)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def max_over_ranks(ms: float, device=None) -> float:
    """The step time of a multi-rank run is the slowest rank's (all ranks start and stop at a barrier)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(bytes_per_rank: int, world: int, ms_per_step: float) -> float:
    """Replicas: every rank aggregates its own workload, so the job's throughput is the sum over ranks (GB/s)."""
    return world * bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def oracle_step(w, cfg, X_host):
    import oracle
    s = w.spec
    return oracle.detox_aggregate(X_host, w.members, s.r, "mean" if cfg["a0"] == 1 else "none", w.set_offsets,
                                  w.set_members, ORACLE_A1[cfg["a1"]], cfg["f"], cfg["m_sel"])


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import oracle
    import paper_1907_12205_b200 as dx  # constants only; nothing is launched
    import workloads as wl
    spec = wl.CONFIGS[args.workload]
    w = wl.make_workload(spec)
    cfg, _ = pipeline_for(args.workload, w, dx)
    X = w.data().numpy()
    for _ in range(min(args.warmup, 1)):
        oracle_step(w, cfg, X)
    steps = max(1, min(args.steps, 5))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(w, cfg, X)
    ms = (time.perf_counter() - t0) * 1e3 / steps
    val = spec.n * spec.d * 4 / (ms * 1e-3) / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_label(args.workload, spec, cfg)},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": "full workload, every step"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_label(name, spec, cfg):
    a0 = {0: "none", 1: "mean"}[cfg["a0"]]
    return (f"{name}: n={spec.n} r={spec.r} d={spec.d} q={spec.q} {spec.attack}/{spec.placement}; "
            f"vote -> A0={a0} -> A1={ORACLE_A1[cfg['a1']]}(f={cfg['f']}, m_sel={cfg['m_sel']})")


def median_minmax_ops(m: int) -> int:
    """min/max operations per coordinate that a median over m rows needs on the register path.

    The merge-exchange network on M inputs (M = m up to 32, else m rounded up to the next network size with an
    even gap) is walked backwards from the middle output: a comparator costs one operation per output that
    something later still reads.  Above 128 rows two lanes share a coordinate and no closed count is given."""
    if m <= 32:
        M = m
    elif m <= 128:
        step = 8 if m <= 64 else 16
        M = (m + step - 1) // step * step
        if (M - m) & 1:
            M -= 1
    else:
        return 0
    net = []
    p = 1
    while p < M:
        k = p
        while k >= 1:
            j = k % p
            while j <= M - 1 - k:
                for i in range(min(k - 1, M - j - k - 1) + 1):
                    if (i + j) // (2 * p) == (i + j + k) // (2 * p):
                        net.append((i + j, i + j + k))
                j += 2 * k
            k //= 2
        p *= 2
    live = {M // 2} if M & 1 else {M // 2 - 1, M // 2}
    ops = 0
    for a, b in reversed(net):
        used = (a in live) + (b in live)
        if used:
            ops += used
            live.update((a, b))
    return ops


# Integer min/max issue on the plain-ALU pipe: 64 lanes per clock and SM, 148 SMs, at the sampled SM clock.
ALU_LANES_PER_CLK_SM, N_SMS = 64, 148


def run_sweep(args):
    """Config 5: every aggregator with and without the DETOX front end over n x d x attack.

    One JSON line per point (not the headline line).  Times are CUDA-event means on one stream after
    warm-up; GB/s is n*d*4 / t; "alg" is the algorithmic bytes of the leg over the same time."""
    import torch

    import paper_1907_12205_b200 as dx
    import workloads as wl

    dev = "cuda:0"
    torch.cuda.set_device(0)
    peaks, peak_kind = measured_peaks()
    ns = [int(x) for x in args.sweep_n.split(",")]
    ds = [int(x) for x in args.sweep_d.split(",")]
    for spec in wl.sweep_specs(ns=ns, ds=ds, attacks=tuple(args.sweep_attacks.split(","))):
        w = wl.make_workload(spec, device=dev)
        n, r, d, G, S, q = spec.n, spec.r, spec.d, w.G, w.S, spec.q
        X = w.X[:, :d]
        out = torch.empty(d, dtype=torch.float32, device=dev)
        in_bytes = n * d * 4
        reps = max(3, min(args.steps, 10))
        legs = {}

        def timed(name, fn, alg_bytes):
            ms = time_calls(torch, fn, reps, 3)
            legs[name] = {"ms": round(ms, 4), "GBps": round(in_bytes / ms / 1e6, 1),
                          "alg_GBps": round(alg_bytes / ms / 1e6, 1),
                          "alg_frac_of_hbm": round(alg_bytes / ms / 1e6 / peaks["hbm_gbs"], 3)}

        def pipe_leg(name, a0, a1, f, m_sel, alg_bytes):
            p = dx.Pipeline(n, r, d, w.members, a0, w.set_offsets if a0 == dx.AGG_MEAN else None,
                            w.set_members if a0 == dx.AGG_MEAN else None, a1, f, m_sel)
            ws = torch.empty(p.workspace_bytes(), dtype=torch.uint8, device=dev)
            win = torch.empty(G, dtype=torch.int32, device=dev)
            sel = torch.empty(max(p.n_selected, 1), dtype=torch.int32, device=dev)
            timed(name, lambda: dx.detox_aggregate(p, X, out=out, winner=win, sel=sel, ws=ws), alg_bytes)
            del ws

        # DETOX legs.  Median: vote -> mean over sets of 5 -> median over the S means (S >= 3), else over the votes.
        if S >= 3:
            pipe_leg("detox_median", dx.AGG_MEAN, dx.AGG_COORD_MEDIAN, 0, 1, (n + 2 * S + 1) * d * 4)
        else:
            pipe_leg("detox_median", dx.AGG_NONE, dx.AGG_COORD_MEDIAN, 0, 1, (n + 2 * G + 1) * d * 4)
        # Krum family: vote -> aggregator over the G votes, tolerance for the few Byzantine votes that survive
        fv = min(2, max((G - 3) // 4, 0))
        pipe_leg("detox_multikrum", dx.AGG_NONE, dx.AGG_MULTIKRUM, fv, G - fv, (n + 2 * G + (G - fv) + 1) * d * 4)
        pipe_leg("detox_bulyan", dx.AGG_NONE, dx.AGG_BULYAN, fv, 1, (n + 2 * G + (G - 2 * fv) + 1) * d * 4)
        # direct legs on all n rows
        timed("direct_median", lambda: dx.agg_coord_median(X, out=out), (n + 1) * d * 4)
        ops = median_minmax_ops(n)
        if n > 16 and ops:
            # beyond ~16 rows the register networks are bound by the plain ALUs, not by HBM: report that roof too
            clk = float(peaks.get("sm_max_mhz", 1965.0))
            peak = ALU_LANES_PER_CLK_SM * N_SMS * clk * 1e6 / 1e12
            ach = ops * d / (legs["direct_median"]["ms"] * 1e-3) / 1e12
            legs["direct_median"]["alu"] = {"bound": "alu", "minmax_per_coordinate": ops, "achieved": round(ach, 2),
                                            "peak": round(peak, 2), "unit": "T min/max per s",
                                            "frac": round(ach / peak, 3), "peak_kind": "64 lanes/clk/SM x 148 SMs x max SM clock"}
        ws = torch.empty(dx.agg_multikrum_workspace_bytes(n, d), dtype=torch.uint8, device=dev)
        sel = torch.empty(n, dtype=torch.int32, device=dev)
        sc = torch.empty(n, dtype=torch.float64, device=dev)
        timed("direct_multikrum", lambda: dx.agg_multikrum(X, q, n - q, out=out, sel=sel[: n - q], scores=sc, ws=ws),
              (n + (n - q) + 1) * d * 4)
        if n >= 4 * q + 3:
            timed("direct_bulyan", lambda: dx.agg_bulyan(X, q, out=out, sel=sel[: n - 2 * q], ws=ws),
                  (n + (n - 2 * q) + 1) * d * 4)
        del ws
        line = {"sweep_point": spec.name, "n": n, "r": r, "d": d, "q": q, "q_hat": w.q_hat, "attack": spec.attack,
                "sets": S, "f_votes": fv, "unit": "GB/s = n*d*4/t", "hbm_peak": peaks["hbm_gbs"],
                "peak_kind": peak_kind, "legs": legs,
                "speedup": {k: round(legs["direct_" + k]["ms"] / legs["detox_" + k]["ms"], 2)
                            for k in ("median", "multikrum", "bulyan") if "direct_" + k in legs}}
        print(json.dumps(line), flush=True)
        del w, X, out
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="detox", choices=["detox", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="config 5: one JSON line per (n, d, attack) point")
    ap.add_argument("--sweep-n", default="15,45,105,225")
    ap.add_argument("--sweep-d", default="1000000,11173962,25557032")
    ap.add_argument("--sweep-attacks", default="reverse,alie")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "detox" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.sweep:
        if rank == 0:
            run_sweep(args)
        return

    import torch
    import torch.distributed as dist

    import paper_1907_12205_b200 as dx
    import workloads as wl

    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    dx.load()

    spec = wl.CONFIGS[args.workload]
    if world > 1:  # every replica draws its own inputs
        import dataclasses
        spec = dataclasses.replace(spec, seed=spec.seed + rank)
    w = wl.make_workload(spec, device=dev)
    cfg, (direct_name, direct_args) = pipeline_for(args.workload, w, dx)
    X = w.X[:, : spec.d]
    pipe = dx.Pipeline(spec.n, spec.r, spec.d, w.members, cfg["a0"], w.set_offsets, w.set_members, cfg["a1"],
                       cfg["f"], cfg["m_sel"])
    ws = torch.empty(pipe.workspace_bytes(), dtype=torch.uint8, device=dev)
    out = torch.empty(spec.d, dtype=torch.float32, device=dev)
    winner = torch.empty(pipe.G, dtype=torch.int32, device=dev)
    sel = torch.empty(max(pipe.n_selected, 1), dtype=torch.int32, device=dev)

    def step():
        dx.detox_aggregate(pipe, X, out=out, winner=winner, sel=sel, ws=ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K steps, barrier + synchronize on both sides, max over ranks ----
    for _ in range(args.warmup):
        step()
    barrier()
    st = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        clocks.wait_first()
        for _ in range(3):
            step()
        torch.cuda.synchronize()
        e0.record(st)
        for _ in range(args.steps):
            step()
        e1.record(st)
        barrier()
        # the dominant kernel alone, same inputs, same stream: the vote (reads n*d*4, writes G*d*4), or the vote
        # fused with the set means when A_0 is the mean (reads n*d*4, writes S*d*4)
        vws = torch.empty(dx.detox_vote_workspace_bytes(spec.n, spec.r), dtype=torch.uint8, device=dev)
        if cfg["a0"] == dx.AGG_MEAN:
            Mbuf = torch.empty((w.S, w.ld), dtype=torch.float32, device=dev)[:, : spec.d]
            dom_name, dom_rows_out = "vote_mean_kernel", w.S
            dom = lambda: dx.detox_vote_hier_mean(X, spec.r, w.members, w.set_offsets, w.set_members, M=Mbuf,
                                                  winner=winner, ws=vws)
        elif cfg["a1"] not in (dx.AGG_MULTIKRUM, dx.AGG_BULYAN) or pipe.G <= 16:
            # the library reads the votes through winner[] here: the vote kernel writes no vote matrix
            dom_name, dom_rows_out = "vote_kernel (winners only)", 0
            dom = lambda: dx.detox_vote(X, spec.r, w.members, want_Z=False, winner=winner, ws=vws)
        else:
            Zbuf = torch.empty((pipe.G, w.ld), dtype=torch.float32, device=dev)[:, : spec.d]
            dom_name, dom_rows_out = "vote_kernel", pipe.G
            dom = lambda: dx.detox_vote(X, spec.r, w.members, Z=Zbuf, winner=winner, ws=vws)
        vote_ms = time_calls(torch, dom, max(args.steps, 10), 3)
    ms_per_step = max_over_ranks(e0.elapsed_time(e1), dev) / args.steps
    in_bytes = spec.n * spec.d * 4
    value = whole_job_value(in_bytes, world, ms_per_step)

    # ---- end to end: pinned host input -> device, aggregate, result -> pinned host ----
    Xh = torch.empty((spec.n, w.ld), dtype=torch.float32, pin_memory=True)
    Xh.copy_(w.X)
    Xd = torch.empty_like(w.X)
    outh = torch.empty(spec.d, dtype=torch.float32, pin_memory=True)

    def e2e_step():
        Xd.copy_(Xh, non_blocking=True)
        dx.detox_aggregate(pipe, Xd[:, : spec.d], out=out, winner=winner, sel=sel, ws=ws)
        outh.copy_(out, non_blocking=True)

    e2e_steps = max(2, min(args.steps, 5))
    barrier()
    e2e_ms = max_over_ranks(time_calls(torch, e2e_step, e2e_steps, 1), dev)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- other legs on the same inputs (rank 0, N = 1 reporting only) ----
    legs = {"detox_pipeline": {"ms": ms_per_step, "GBps": in_bytes / ms_per_step / 1e6}}
    if direct_name == "multikrum":
        dws = torch.empty(dx.agg_multikrum_workspace_bytes(spec.n, spec.d), dtype=torch.uint8, device=dev)
        dsel = torch.empty(direct_args["m_sel"], dtype=torch.int32, device=dev)
        dsc = torch.empty(spec.n, dtype=torch.float64, device=dev)
        fn = lambda: dx.agg_multikrum(X, direct_args["f"], direct_args["m_sel"], out=out, sel=dsel, scores=dsc, ws=dws)
    elif direct_name == "bulyan":
        dws = torch.empty(dx.agg_bulyan_workspace_bytes(spec.n, spec.d), dtype=torch.uint8, device=dev)
        dsel = torch.empty(spec.n - 2 * direct_args["f"], dtype=torch.int32, device=dev)
        fn = lambda: dx.agg_bulyan(X, direct_args["f"], out=out, sel=dsel, ws=dws)
    else:
        fn = lambda: dx.agg_coord_median(X, out=out)
    dms = time_calls(torch, fn, max(3, min(args.steps, 10)), 3)
    legs[f"direct_{direct_name}"] = {"ms": dms, "GBps": in_bytes / dms / 1e6, "args": direct_args}
    legs["detox_speedup_vs_direct"] = dms / ms_per_step

    peaks, peak_kind = measured_peaks()
    vote_bytes = (spec.n + dom_rows_out) * spec.d * 4
    achieved = vote_bytes / (vote_ms * 1e-3) / 1e9
    roofline = {"kernel": dom_name, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                "frac_of_8TBps": achieved / 8000.0, "ms_per_launch": vote_ms, "algorithmic_bytes": vote_bytes,
                "traffic": NCU_TRAFFIC_BYTES.get((args.workload, dom_name))}

    cpu_baseline = None
    parity = None
    if not args.no_cpu_baseline:
        import oracle
        Xn = w.X.cpu().numpy()[:, : spec.d]
        t0 = time.perf_counter()
        ref = oracle_step(w, cfg, Xn)
        cpu_s = time.perf_counter() - t0
        cpu_baseline = {"value": in_bytes / cpu_s / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": "full workload, 1 repetition", "ms": cpu_s * 1e3}
        step()
        torch.cuda.synchronize()
        o = out.cpu().numpy().astype(np.float64)
        den = np.linalg.norm(ref["out"].astype(np.float64))
        parity = {"winner_exact": winner.cpu().numpy().tolist() == ref["winner"].tolist(),
                  "out_rel_l2": float(np.linalg.norm(o - ref["out"]) / (den if den else 1.0))}
        if ref["sel"] is not None:
            parity["sel_exact"] = sel.cpu().numpy()[: len(ref["sel"])].tolist() == ref["sel"].tolist()

    kernels_per_step = {"cfg1": 3, "cfg2": 6, "cfg3": 6, "cfg4": 4}[args.workload]
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_label(args.workload, spec, cfg), "l2": "inputs larger than L2"
                       if in_bytes > 2 * 126e6 else "inputs fit in L2 (warm)", "replicas": world},
            "clocks": clocks.summary(),
            "e2e": {"value": whole_job_value(in_bytes, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": int(Xh.numel() * 4), "d2h_bytes_per_step": int(outh.numel() * 4)},
            "gpu_launches": kernels_per_step * args.steps, "kernels_per_step": kernels_per_step,
            "roofline": roofline, "cpu_baseline": cpu_baseline, "legs": legs, "parity": parity}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
