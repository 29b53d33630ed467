#!/usr/bin/env python
"""Benchmark of the DETOX aggregation step (vote -> hierarchical mean -> robust aggregator) on B200.

Default workload: the largest named single-GPU configuration, n = 105 workers, r = 3, d = 28,000,000 (VGG-class),
q = 15 ALIE attackers; one step = detox_aggregate(vote -> mean over 7 sets of 5 -> coordinate median over the 7).
The metric is aggregation input throughput n*d*4 bytes per second.  Prints ONE JSON line, which also carries the
direct (non-DETOX) aggregators on the same buffer, each with the roofline that bounds its dominant kernel.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload cfg4|cfg1|cfg2|cfg3]
  python bench.py --sweep            (one JSON line per point of the n x d x attack sweep)
  python bench.py --mean-estimation  (the synthetic experiment with 220,000 nodes: one JSON line per dimension)

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
# Dense TF32 tensor throughput is nominally 1.1 / 2.25 of the bf16 one; the tensor roof is the measured bf16 peak
# times that ratio.
TF32_OVER_BF16 = 1.1 / 2.25


def pipeline_for(name, w, dx):
    """The DETOX leg and the direct (non-DETOX) legs of each named configuration."""
    s = w.spec
    if name == "cfg1":
        return (dict(a0=dx.AGG_NONE, a1=dx.AGG_COORD_MEDIAN, f=0, m_sel=1), [("coord_median", {})])
    if name == "cfg2":
        return (dict(a0=dx.AGG_MEAN, a1=dx.AGG_MULTIKRUM, f=1, m_sel=1), [("multikrum", dict(f=5, m_sel=s.n - 5))])
    if name == "cfg3":
        return (dict(a0=dx.AGG_NONE, a1=dx.AGG_BULYAN, f=3, m_sel=1), [("bulyan", dict(f=9))])
    if name == "cfg4":
        return (dict(a0=dx.AGG_MEAN, a1=dx.AGG_COORD_MEDIAN, f=0, m_sel=1),
                [("coord_median", {}), ("multikrum", dict(f=15, m_sel=s.n - 15))])
    raise ValueError(name)


def paper_pairings(name, w, dx):
    """The pairings the paper found most resilient (Section 5.2, setups 2 and 3; vote-set shapes of Appendix B.1):
    the Krum-type aggregator inside every vote set, then the mean of the set results."""
    G = w.G
    if name in ("cfg2", "cfg3"):   # 15 votes: Multi-Krum in sets of 7 and 8 (f = 2); Bulyan on one set of 15 (f = 3)
        return [("vote_multikrum_in_sets_7_8_mean", dx.AGG_MULTIKRUM, [0, 7, G], 2, 0),
                ("vote_bulyan_in_one_set_mean", dx.AGG_BULYAN, [0, G], 3, 0)]
    if name == "cfg4":             # 35 votes: Multi-Krum (f = 1, all but one kept) inside the 7 sets of 5
        return [("vote_multikrum_in_sets_of_5_mean", dx.AGG_MULTIKRUM, [int(x) for x in w.set_offsets], 1, 0)]
    return []


ORACLE_A1 = {1: "mean", 2: "coord_median", 3: "multikrum", 4: "bulyan"}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel of the DETOX step, from ncu captures of
# the same kernel code (reset an entry to None when its kernel changes).
NCU_TRAFFIC_BYTES = {
    ("cfg2", "vote_mean_kernel"): 2_011_332_000 + 118_065_152,
    ("cfg3", "vote_kernel (winners only)"): 2_011_382_000 + 5_457_920,
    # config 4 holds 11.8 GB, too much for a multi-pass capture: the traffic of the same streaming kernel on 105 rows of
    # 2,500,000 columns, scaled by the algorithmic bytes (11,872,000,000 / 1,060,000,000)
    ("cfg4", "vote_mean_select_kernel"): int((1_050_018_000 + 7_588_096) * 11_872_000_000 / 1_060_000_000),
}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={CLOCK_QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
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
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0}, "fallback"


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


def workload_label(name, spec, cfg):
    a0 = {0: "none", 1: "mean"}[cfg["a0"]]
    return (f"{name}: n={spec.n} r={spec.r} d={spec.d} q={spec.q} {spec.attack}/{spec.placement}; "
            f"vote -> A0={a0} -> A1={ORACLE_A1[cfg['a1']]}(f={cfg['f']}, m_sel={cfg['m_sel']})")


def config_entry(name, spec, cfg, world):
    """The `config` object of the JSON line; both arms print the same one."""
    in_bytes = spec.n * spec.d * 4
    return {"workload": workload_label(name, spec, cfg),
            "l2": "inputs larger than L2" if in_bytes > 2 * 126e6 else "inputs fit in L2 (warm)", "replicas": world}


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only).  A step is the whole
    workload when K such steps end within a few minutes, else its first d' columns (all rows)."""
    if rank != 0:
        return
    import oracle
    import paper_1907_12205_b200 as dx  # constants only; nothing is launched
    import workloads as wl
    spec = wl.CONFIGS[args.workload]
    w = wl.make_workload(spec)
    cfg, _ = pipeline_for(args.workload, w, dx)
    X = w.data().numpy()
    t0 = time.perf_counter()
    oracle_step(w, cfg, X)                       # first touch + a full-size estimate
    full_s = time.perf_counter() - t0
    budget_s = 150.0
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    d_s, sample = spec.d, "full workload, every step"
    if full_s * (steps + warmup) > budget_s:
        d_s = max(1024, int(spec.d * budget_s / (full_s * (steps + warmup))))
        sample = f"first {d_s} of {spec.d} columns of all {spec.n} rows, every step"
    Xs = np.ascontiguousarray(X[:, :d_s]) if d_s < spec.d else X
    for _ in range(warmup):
        oracle_step(w, cfg, Xs)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(w, cfg, Xs)
    ms = (time.perf_counter() - t0) * 1e3 / steps
    val = spec.n * d_s * 4 / (ms * 1e-3) / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_entry(args.workload, spec, cfg, world),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------- rooflines

def merge_exchange_net(M: int):
    """Comparators of Batcher's merge-exchange network on M inputs, in network order."""
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
    return net


def median_minmax_ops(m: int) -> int:
    """min/max operations per coordinate that a median over m rows costs in the library's kernels.

    Up to 128 rows (one thread per coordinate): the merge-exchange network on M inputs (M = m up to 32, else m
    rounded up to the next network size with an even gap) is walked backwards from the middle output; a comparator
    costs one operation per output that something later still reads.  129 to 256 rows (two lanes per coordinate, H
    keys each, H = half of m rounded up to 8): each lane sorts its H keys completely (two operations per
    comparator), takes H operations in the split against its partner's keys and H - 1 to reduce its half to the
    extreme value.  Beyond 256 rows (shared-memory path) no count is given."""
    if m > 256:
        return 0
    if m > 128:
        H = ((m + 1) // 2 + 7) // 8 * 8
        return 2 * (2 * len(merge_exchange_net(H)) + H + H - 1)
    if m <= 32:
        M = m
    else:
        step = 8 if m <= 64 else 16
        M = (m + step - 1) // step * step
        if (M - m) & 1:
            M -= 1
    live = {M // 2} if M & 1 else {M // 2 - 1, M // 2}
    ops = 0
    for a, b in reversed(merge_exchange_net(M)):
        used = (a in live) + (b in live)
        if used:
            ops += used
            live.update((a, b))
    return ops


# Integer min/max issue on the plain-ALU pipe: 64 lanes per clock and SM, 148 SMs, at the maximum SM clock.
ALU_LANES_PER_CLK_SM, N_SMS = 64, 148


def median_alu_roofline(m, d, ms, peaks):
    """The plain-ALU roof of a coordinate median over m rows (bound by integer min/max issue beyond ~16 rows)."""
    ops = median_minmax_ops(m)
    if m <= 16 or not ops:
        return None
    clk = float(peaks.get("sm_max_mhz", 1965.0))
    peak = ALU_LANES_PER_CLK_SM * N_SMS * clk * 1e6 / 1e12
    ach = ops * d / (ms * 1e-3) / 1e12
    return {"kernel": "colselect_reg_kernel" if m <= 128 else "colselect_pair_kernel", "bound": "alu",
            "minmax_per_coordinate": ops, "achieved": round(ach, 3), "peak": round(peak, 2), "unit": "T min/max per s",
            "frac": round(ach / peak, 3), "peak_kind": "64 lanes/clk/SM x 148 SMs x max SM clock",
            "hbm_frac": round((m + 1) * d * 4 / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 3), "ms_per_launch": ms,
            "traffic": None}


# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the tensor-core distance kernel over the algorithmic
# bytes m d 4, from ncu captures at d = 2.5 M (the kernel reads every row once, so its traffic grows with m d); reset an
# entry to None when the kernel changes.
NCU_GRAM_TRAFFIC_RATIO = {45: 1.034, 105: 1.043, 225: 1.095}


def gram_roofline(m, d, ms, peaks, peak_kind, ms_tf32=None):
    """Roofline of the distance pass of Multi-Krum / Bulyan over m rows, timed through agg_pairwise_sqdist (the
    streaming kernel plus the small kernels around it: sample, check, reduction).

    17 to 256 aligned rows run on the tensor cores with every entry split into an fp16 pair.  The pass reads every
    row once, so `hbm` is m d 4 / t.  `tensor.issued` is what the tensor pipe was given -- two fp16 products (hi.hi
    and hi.lo), padded to the MMA shape (rows to 64 / 128 / 256, columns to m rounded up to 16) -- against the fp16
    dense peak (= the measured bf16 one); `tensor.useful` = 2 m^2 d / t, the flops of the Gram matrix the split
    products stand for, also as a multiple of what three-product TF32 could reach at most (TF32 peak / 3).  The bound
    named is the one with the larger fraction.  ms_tf32: the same call with the split-TF32 kernels, for comparison."""
    hbm = m * d * 4 / (ms * 1e-3) / 1e9
    if m <= 16:
        return {"kernel": "sqdist_staged_kernel / sqdist_direct_kernel", "bound": "hbm", "achieved": round(hbm, 1),
                "peak": peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": round(hbm / peaks["hbm_gbs"], 3), "ms_per_launch": ms, "algorithmic_bytes": m * d * 4,
                "traffic": None}
    ncol = (m + 15) // 16 * 16
    mrows = 64 if m <= 64 else (128 if m <= 128 else 256)
    useful = 2.0 * m * m * d / (ms * 1e-3) / 1e12
    issued = 2.0 * mrows * (2 * ncol) * d / (ms * 1e-3) / 1e12
    peak_f16 = peaks["bf16_tflops"]
    peak_3xtf32 = peaks["bf16_tflops"] * TF32_OVER_BF16 / 3.0
    hbm_frac, tensor_frac = hbm / peaks["hbm_gbs"], issued / peak_f16
    ratio = NCU_GRAM_TRAFFIC_RATIO.get(m)
    out = {"kernel": "gram_f16_kernel", "bound": "hbm" if hbm_frac >= tensor_frac else "tensor",
           "achieved": round(hbm, 1) if hbm_frac >= tensor_frac else round(issued, 1),
           "peak": peaks["hbm_gbs"] if hbm_frac >= tensor_frac else round(peak_f16, 1),
           "unit": "GB/s" if hbm_frac >= tensor_frac else "TFLOP/s", "peak_kind": f"of {peak_kind}",
           "frac": round(max(hbm_frac, tensor_frac), 3),
           "hbm": {"GBps": round(hbm, 1), "frac": round(hbm_frac, 3)},
           "tensor": {"issued": round(issued, 1), "peak": round(peak_f16, 1), "frac": round(tensor_frac, 3),
                      "peak_kind": f"{peak_kind} bf16 burst peak (fp16 runs at the same rate)",
                      "useful": round(useful, 1), "peak_3xTF32": round(peak_3xtf32, 1),
                      "useful_over_peak_3xTF32": round(useful / peak_3xtf32, 3), "unit": "TFLOP/s"},
           "ms_per_launch": ms, "algorithmic_bytes": m * d * 4, "algorithmic_flops": 2.0 * m * m * d,
           "traffic": None if ratio is None else int(ratio * m * d * 4)}
    if ms_tf32 is not None:
        issued32 = 2.0 * mrows * (2 * ncol) * d / (ms_tf32 * 1e-3) / 1e12
        peak32 = peaks["bf16_tflops"] * TF32_OVER_BF16
        out["split_tf32"] = {"kernel": "gram_staged_kernel" if m <= 128 else "gram_wide_kernel", "ms_per_launch": ms_tf32,
                             "hbm_frac": round(m * d * 4 / (ms_tf32 * 1e-3) / 1e9 / peaks["hbm_gbs"], 3),
                             "issued": round(issued32, 1), "peak": round(peak32, 1),
                             "peak_kind": f"{peak_kind} bf16 burst peak x nominal TF32/bf16 ratio {TF32_OVER_BF16:.3f}",
                             "frac": round(issued32 / peak32, 3)}
    return out


def time_distance_pass(torch, dx, X, D, ws, reps):
    """agg_pairwise_sqdist with the default operand split and, for the tensor-core sizes, with the split-TF32 kernels."""
    ms = time_calls(torch, lambda: dx.agg_pairwise_sqdist(X, D=D, ws=ws), reps, 3)
    ms32 = None
    if 16 < X.shape[0] <= 256:
        prev = dx.tc_split_mode(dx.SPLIT_TF32)
        try:
            ms32 = time_calls(torch, lambda: dx.agg_pairwise_sqdist(X, D=D, ws=ws), reps, 3)
        finally:
            dx.tc_split_mode(prev)
    return ms, ms32


def run_sweep(args):
    """The sweep: every aggregator with and without the DETOX front end over n x d x attack.

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
    code = {"none": dx.AGG_NONE, "mean": dx.AGG_MEAN, "coord_median": dx.AGG_COORD_MEDIAN,
            "multikrum": dx.AGG_MULTIKRUM, "bulyan": dx.AGG_BULYAN}
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
            return ms

        ws = torch.empty(dx.agg_multikrum_workspace_bytes(n, d), dtype=torch.uint8, device=dev)
        sel = torch.empty(n, dtype=torch.int32, device=dev)
        sc = torch.empty(n, dtype=torch.float64, device=dev)
        plan = wl.sweep_legs(spec, G, S)
        for name, leg in plan.items():
            if name.startswith("detox_"):
                mean0 = leg["a0"] == "mean"
                rows1 = S if mean0 else G
                p = dx.Pipeline(n, r, d, w.members, code[leg["a0"]], w.set_offsets if mean0 else None,
                                w.set_members if mean0 else None, code[leg["a1"]], leg["f"], leg["m_sel"])
                pws = torch.empty(p.workspace_bytes(), dtype=torch.uint8, device=dev)
                win = torch.empty(G, dtype=torch.int32, device=dev)
                psel = torch.empty(max(p.n_selected, 1), dtype=torch.int32, device=dev)
                second = {"coord_median": 0, "multikrum": leg["m_sel"], "bulyan": rows1 - 2 * leg["f"]}[leg["a1"]]
                # compulsory traffic: every worker's row once, the rows the second sweep averages or sorts, the result
                # (votes and set means need not travel: the vote runs inside the pass that consumes it)
                timed(name, lambda: dx.detox_aggregate(p, X, out=out, winner=win, sel=psel, ws=pws),
                      (n + second + 1) * d * 4)
                del pws
            elif leg["a1"] == "coord_median":
                ms = timed(name, lambda: dx.agg_coord_median(X, out=out), (n + 1) * d * 4)
                roof = median_alu_roofline(n, d, ms, peaks)
                if roof:
                    legs[name]["alu"] = roof
            elif leg["a1"] == "multikrum":
                timed(name, lambda: dx.agg_multikrum(X, leg["f"], leg["m_sel"], out=out, sel=sel[: leg["m_sel"]],
                                                     scores=sc, ws=ws), (n + leg["m_sel"] + 1) * d * 4)
                D = torch.empty((n, n), dtype=torch.float64, device=dev)
                gms, gms32 = time_distance_pass(torch, dx, X, D, ws, reps)
                legs[name]["distance_pass"] = gram_roofline(n, d, gms, peaks, peak_kind, gms32)
            else:
                timed(name, lambda: dx.agg_bulyan(X, leg["f"], out=out, sel=sel[: n - 2 * leg["f"]], ws=ws),
                      (n + (n - 2 * leg["f"]) + 1) * d * 4)
        del ws
        line = {"sweep_point": spec.name, "n": n, "r": r, "d": d, "q": q, "q_hat": w.q_hat, "attack": spec.attack,
                "sets": S, "f_votes": plan["detox_multikrum"]["f"], "unit": "GB/s = n*d*4/t",
                "hbm_peak": peaks["hbm_gbs"], "peak_kind": peak_kind, "legs": legs,
                "speedup": {k: round(legs["direct_" + k]["ms"] / legs["detox_" + k]["ms"], 2)
                            for k in ("median", "multikrum", "bulyan") if "direct_" + k in legs}}
        print(json.dumps(line), flush=True)
        del w, X, out
        torch.cuda.empty_cache()


def run_mean_estimation(args):
    """The paper's synthetic experiment (Section 5.3, "Mean estimation on synthetic data"): p = 220,000 nodes, r = 11,
    q = floor(e^r / 3) Byzantine nodes sending a constant vector of norm 100, d = 20 .. 100.  DETOX = vote -> mean
    inside 25 vote sets -> geometric median (or coordinate median) of the 25 means; the error is the l2 norm of the
    estimate (the true mean is zero).  One JSON line per d; times are CUDA-event means after warm-up."""
    import torch

    import oracle
    import paper_1907_12205_b200 as dx
    import workloads as wl

    dev = "cuda:0"
    torch.cuda.set_device(0)
    reps = max(3, min(args.steps, 20))
    for d in range(20, 101, 10):
        w = wl.make_mean_estimation(d=d, seed=d, device=dev)
        X = w.X
        members = torch.as_tensor(w.members, device=dev)
        G, S = w.p // w.r, len(w.set_offsets) - 1
        M = torch.empty((S, (d + 31) // 32 * 32), dtype=torch.float32, device=dev)[:, :d]
        win = torch.empty(G, dtype=torch.int32, device=dev)
        out = torch.empty(d, dtype=torch.float32, device=dev)
        gws = torch.empty(max(int(dx.load().agg_geometric_median_workspace_bytes(S, d)), 256), dtype=torch.uint8, device=dev)

        def step_gm():
            dx.detox_vote_hier_mean_many(X, w.r, members, w.set_offsets, M=M, winner=win)
            dx.agg_geometric_median(M, iters=32, out=out, ws=gws)

        def step_med():
            dx.detox_vote_hier_mean_many(X, w.r, members, w.set_offsets, M=M, winner=win)
            dx.agg_coord_median(M, out=out)

        ms_gm = time_calls(torch, step_gm, reps, 3)
        step_gm(); torch.cuda.synchronize()
        err_gm = float(torch.linalg.vector_norm(out))
        ms_med = time_calls(torch, step_med, reps, 3)
        step_med(); torch.cuda.synchronize()
        err_med = float(torch.linalg.vector_norm(out))
        ms_front = time_calls(torch, lambda: dx.detox_vote_hier_mean_many(X, w.r, members, w.set_offsets, M=M, winner=win),
                              reps, 3)
        Xh = X.cpu().numpy()
        t0 = time.perf_counter()
        Zo, wo = oracle.vote(Xh, w.members, w.r)
        Mo = oracle.hier_mean(Zo, w.set_offsets, np.arange(G, dtype=np.int32))
        go = oracle.geometric_median(Mo, iters=32)
        cpu_ms = (time.perf_counter() - t0) * 1e3
        in_bytes = w.p * d * 4
        print(json.dumps({"mean_estimation": True, "p": w.p, "r": w.r, "q": w.q, "q_hat": w.q_hat, "d": d, "sets": S,
                          "detox_geometric_median": {"ms": round(ms_gm, 4), "l2_error": err_gm,
                                                     "GBps": round(in_bytes / ms_gm / 1e6, 1)},
                          "detox_coord_median": {"ms": round(ms_med, 4), "l2_error": err_med,
                                                 "GBps": round(in_bytes / ms_med / 1e6, 1)},
                          "vote_and_set_means": {"ms": round(ms_front, 4), "GBps": round(in_bytes / ms_front / 1e6, 1)},
                          "oracle": {"ms": round(cpu_ms, 1), "cores": oracle.num_threads(),
                                     "l2_error_geometric_median": float(np.linalg.norm(go)),
                                     "winners_equal": win.cpu().numpy().tolist() == wo.tolist()}}), flush=True)
        del w, X


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="detox", choices=["detox", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="one JSON line per (n, d, attack) point of the sweep")
    ap.add_argument("--sweep-n", default="15,45,105,225")
    ap.add_argument("--sweep-d", default="1000000,11173962,25557032")
    ap.add_argument("--sweep-attacks", default="reverse,alie")
    ap.add_argument("--mean-estimation", action="store_true",
                    help="the synthetic mean-estimation experiment: one JSON line per dimension")
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
    if args.mean_estimation:
        if rank == 0:
            run_mean_estimation(args)
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
    cfg, direct_legs = pipeline_for(args.workload, w, dx)
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
        launches_before = dx.kernel_launch_count()
        e0.record(st)
        for _ in range(args.steps):
            step()
        e1.record(st)
        barrier()
        gpu_launches = dx.kernel_launch_count() - launches_before   # counted by the library at every launch
        # the dominant kernel alone, same inputs, same stream: the vote (reads n*d*4, writes G*d*4), or the vote
        # fused with the set means when A_0 is the mean (reads n*d*4, writes S*d*4)
        vws = torch.empty(dx.detox_vote_workspace_bytes(spec.n, spec.r), dtype=torch.uint8, device=dev)
        fused_a1 = cfg["a1"] in (dx.AGG_COORD_MEDIAN, dx.AGG_TRIMMED_MEAN, dx.AGG_MEAN)
        if cfg["a0"] == dx.AGG_MEAN and fused_a1 and w.S <= 16 and spec.r in (1, 3, 5):
            # vote, set means and the coordinate-wise A_1 are one kernel (reads n*d*4, writes d*4): the step itself,
            # which only adds two ~3 us helper kernels
            dom_name, dom_rows_out = "vote_mean_select_kernel", 1
            dom = step
        elif cfg["a0"] == dx.AGG_MEAN:
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
    del Xd

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- other legs on the same inputs (rank 0 reporting only) ----
    peaks, peak_kind = measured_peaks()
    reps = max(3, min(args.steps, 10))
    legs = {"detox_pipeline": {"ms": ms_per_step, "GBps": in_bytes / ms_per_step / 1e6}}
    for direct_name, direct_args in direct_legs:
        leg = {"args": direct_args}
        if direct_name in ("multikrum", "bulyan"):
            dws = torch.empty(dx.agg_multikrum_workspace_bytes(spec.n, spec.d), dtype=torch.uint8, device=dev)
            if direct_name == "multikrum":
                dsel = torch.empty(direct_args["m_sel"], dtype=torch.int32, device=dev)
                dsc = torch.empty(spec.n, dtype=torch.float64, device=dev)
                fn = lambda: dx.agg_multikrum(X, direct_args["f"], direct_args["m_sel"], out=out, sel=dsel, scores=dsc,
                                              ws=dws)
            else:
                dsel = torch.empty(spec.n - 2 * direct_args["f"], dtype=torch.int32, device=dev)
                fn = lambda: dx.agg_bulyan(X, direct_args["f"], out=out, sel=dsel, ws=dws)
            dms = time_calls(torch, fn, reps, 3)
            D = torch.empty((spec.n, spec.n), dtype=torch.float64, device=dev)
            gms, gms32 = time_distance_pass(torch, dx, X, D, dws, reps)
            leg["roofline"] = gram_roofline(spec.n, spec.d, gms, peaks, peak_kind, gms32)
            del dws
        else:
            dms = time_calls(torch, lambda: dx.agg_coord_median(X, out=out), reps, 3)
            hbm = (spec.n + 1) * spec.d * 4 / (dms * 1e-3) / 1e9
            leg["roofline"] = median_alu_roofline(spec.n, spec.d, dms, peaks) or {
                "kernel": "colselect_reg_kernel", "bound": "hbm", "achieved": hbm, "peak": peaks["hbm_gbs"],
                "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": hbm / peaks["hbm_gbs"], "ms_per_launch": dms,
                "traffic": None}
        leg.update(ms=dms, GBps=in_bytes / dms / 1e6, detox_speedup=dms / ms_per_step)
        legs[f"direct_{direct_name}"] = leg
    legs["detox_speedup_vs_direct"] = legs[f"direct_{direct_legs[0][0]}"]["ms"] / ms_per_step
    for name, a0, offsets, f, m_sel in paper_pairings(args.workload, w, dx):
        p2 = dx.Pipeline(spec.n, spec.r, spec.d, w.members, a0, offsets, w.set_members, dx.AGG_MEAN, f, m_sel)
        ws2 = torch.empty(p2.workspace_bytes(), dtype=torch.uint8, device=dev)
        sel2 = torch.empty(max(p2.n_selected, 1), dtype=torch.int32, device=dev)
        ms2 = time_calls(torch, lambda: dx.detox_aggregate(p2, X, out=out, winner=winner, sel=sel2, ws=ws2), reps, 3)
        legs[name] = {"ms": ms2, "GBps": in_bytes / ms2 / 1e6, "f": f, "sets": offsets}
        del ws2

    G_votes = spec.n // spec.r
    if spec.r == 3 and 16 < G_votes <= 85:
        # A Krum-type A_1 over all votes: the vote runs inside the tensor-core distance pass (one pass over X for both),
        # then the kept winners' rows are averaged (Multi-Krum) or go through Bulyan's second stage.  Reported against
        # the step's compulsory traffic: every row once, the rows of the second sweep, the result.
        fv = min(2, (G_votes - 3) // 4)
        for name, a1, second in (("vote_in_distance_pass_multikrum", dx.AGG_MULTIKRUM, G_votes - fv),
                                 ("vote_in_distance_pass_bulyan", dx.AGG_BULYAN, G_votes - 2 * fv)):
            p3 = dx.Pipeline(spec.n, spec.r, spec.d, w.members, dx.AGG_NONE, None, None, a1, fv, G_votes - fv)
            ws3 = torch.empty(p3.workspace_bytes(), dtype=torch.uint8, device=dev)
            sel3 = torch.empty(max(p3.n_selected, 1), dtype=torch.int32, device=dev)
            ms3 = time_calls(torch, lambda: dx.detox_aggregate(p3, X, out=out, winner=winner, sel=sel3, ws=ws3), reps, 3)
            comp = (spec.n + second + 1) * spec.d * 4
            legs[name] = {"ms": ms3, "GBps": in_bytes / ms3 / 1e6, "f": fv, "votes": G_votes,
                          "compulsory_bytes": comp, "compulsory_GBps": comp / ms3 / 1e6,
                          "compulsory_frac_of_hbm": comp / ms3 / 1e6 / peaks["hbm_gbs"], "status_word": dx.read_status(ws3)}
            del ws3

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
                  "out_rel_l2": float(np.linalg.norm(o - ref["out"]) / (den if den else 1.0)),
                  "status_word": dx.read_status(ws)}
        if ref["sel"] is not None:
            parity["sel_exact"] = sel.cpu().numpy()[: len(ref["sel"])].tolist() == ref["sel"].tolist()

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_entry(args.workload, spec, cfg, world),
            "clocks": clocks.summary(),
            "e2e": {"value": whole_job_value(in_bytes, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": int(Xh.numel() * 4), "d2h_bytes_per_step": int(outh.numel() * 4)},
            "gpu_launches": gpu_launches, "kernels_per_step": gpu_launches / args.steps,
            "roofline": roofline, "cpu_baseline": cpu_baseline, "legs": legs, "parity": parity}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
