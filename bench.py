#!/usr/bin/env python
"""Benchmark of the whole RandomTMA hot path on one B200 (or N independent replicas).

One step = one pass of the whole path over the workload: broadcast of the initial weights,
partition, induced CSR (count + fill), row gather, then R x (K local steps on all M parts +
aggregation).  The default workload is Large, the largest of the named shapes that one GPU
holds (Chung-Lu power-law graph, 25M nodes, ~1.3B directed entries with 64-bit row offsets,
128-d features, 2 classes with 1% positives, M=32 trainers, 128-256-2 GraphSAGE-mean, 5 local
steps, one aggregation; about 35 GB of host memory and a minute of 16 host threads to
generate).  --workload selects the other shapes: medium (200k nodes, ~5M entries, M=8,
128-256-256-47, 20 steps x 5 rounds), supertma (planted communities, super-node assignment,
M=16), sweep (the same graph at width 512 with bf16 GEMM operands; --M and --assign pick the
point of the sweep); --scale shrinks any of them; averaging times the aggregation kernel
alone on a shape large enough to be bound by HBM.

Metric: aggregated edges/s = (sum over parts of kept entries) x (aggregations a local step is
made of: L forward + L-1 backward) x (local steps) / time.  Local trainer-steps/s is reported
beside it.  The library computes the aggregate of the (constant) input features once per
rtma_local_steps call instead of once per step; the unit still counts it per step, as the
method defines it, and `edges_gathered_per_s` gives the rate of the gathers actually executed.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload large|medium|supertma|sweep|averaging] [--scale S] [--M M] [--assign node|super]

Prints one JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "aggregated_edges_per_s"
UNIT = "edges/s"
NOMINAL_HBM_GBS = 8000.0   # the figure the bandwidth targets are quoted on; fractions are given against both
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS, bf16_tflops_sustained=1400.0,
                sm_max_mhz=1965.0, source="fallback")


# ---------------------------------------------------------------------------------------
# workload arithmetic (algorithmic work per kernel class for one bench step)
# ---------------------------------------------------------------------------------------
def algorithmic_work(dims, n_parts, e_parts, K, R, entries=0, rowptr_bytes=8, grouped=False):
    """Per kernel class: (bound, algorithmic bytes, algorithmic flops) summed over one bench
    step.  Bytes are compulsory traffic (every operand read once, every result written once)."""
    L = len(dims) - 1
    n, e = float(sum(n_parts)), float(sum(e_parts))
    steps = K * R
    work = {}
    # preprocessing, once per bench step.  Partition: part_id, perm, local_id written (12 B per node; the
    # super-node id read by each of its two passes); with super-nodes kept together, four radix passes
    # of (order read, super-node id gathered) x 2 + order written
    E = float(entries)
    part_count = (4.0 * n if grouped else 0.0) + (4 * (8.0 * n) if grouped else 0.0)
    part_scatter = 12.0 * n + (4.0 * n if grouped else 0.0) + (4 * (12.0 * n) if grouped else 0.0)
    work["partition_count"] = ("hbm", part_count, 0.0)
    work["partition_scatter"] = ("hbm", part_scatter, 0.0)
    # induced subgraphs: per entry the column id, the part of its end point and one bit (kept or not) written
    # (count pass); that bit, and per kept entry its column id, the end point's local id and the entry written
    # (fill pass); per row its offsets, its node id and its part
    work["induced_count"] = ("hbm", E * 8 + E / 8 + 4 * n + n * (2 * rowptr_bytes + 8 + 8), 0.0)
    work["induced_fill"] = ("hbm", E / 8 + 4 * n + e * 12 + n * (2 * rowptr_bytes + 8 + 8), 0.0)
    work["gather_rows"] = ("hbm", 12.0 * n, 0.0)                         # labels only: perm, label in, label out
    work["to_planes"] = ("hbm", R * (8.0 * n * dims[0] + 4.0 * n), 0.0)   # features gathered through perm into planes
    # The last layer's aggregate is taken after its product when that is narrower (the library's rule:
    # at most 64 classes and [H Ws | H Wn], 2 Cp wide, at most half as wide as the layer's input):
    # scores = H Ws + Abar (H Wn) + b, dWn = H^T (Abar^T dZ).  Bytes below are those of the products and
    # aggregations actually defined by that form.
    Mtr = len(n_parts)
    C = dims[L]
    Cp = (C + 7) // 8 * 8
    head = C <= 64 and 4 * Cp <= dims[L - 1]
    full = range(L - 1) if head else range(L)          # layers whose products take [H | Abar H]
    # aggregations per local step: Abar H^l for l >= 1 (l = 0 once per call), Abar^T dZ^l for l >= 1
    agg_f = [dims[l] for l in full if l >= 1] + ([Cp] if head else [])
    agg_b = [dims[l + 1] for l in range(1, L) if not (head and l == L - 1)] + ([Cp] if head else [])
    first = (n * 8 * dims[0] + 4 * e + 8 * n) / K if (L > 1 or not head) else 0.0
    spmm_f = sum(n * 8 * d + 4 * e + 8 * n for d in agg_f) + first
    spmm_b = sum(n * 8 * d + 4 * e + 12 * n for d in agg_b)
    work["spmm_forward"] = ("hbm", steps * spmm_f, steps * (sum(e * d for d in agg_f) + (e * dims[0] / K if first else 0.0)))
    work["spmm_backward"] = ("hbm", steps * spmm_b, steps * sum(2 * e * d for d in agg_b))
    gf_b = sum(4 * n * (2 * dims[l] + dims[l + 1]) + 4 * Mtr * (2 * dims[l] + 1) * dims[l + 1] for l in full)
    gf_f = sum(2 * n * (2 * dims[l] + 1) * dims[l + 1] for l in full)
    gw_b, gw_f = gf_b, gf_f
    if head:   # T = H [Ws | Wn] (2 Cp wide out);  [dWs | dWn] = H^T [dZ | Q]
        gf_b += 4 * n * (dims[L - 1] + 2 * Cp) + 4 * Mtr * 2 * dims[L - 1] * C
        gf_f += 2 * n * dims[L - 1] * 2 * C
        gw_b += 4 * n * (dims[L - 1] + 2 * Cp) + 4 * Mtr * (2 * dims[L - 1] + 1) * C
        gw_f += 2 * n * (dims[L - 1] + 1) * 2 * C
    work["gemm_forward"] = ("gemm", steps * gf_b, steps * gf_f)
    work["gemm_wgrad"] = ("gemm", steps * gw_b, steps * gw_f)
    # dgrad reads dZ and Abar^T dZ (planes), the gate (hi plane of H) and writes dZ of the layer below
    gd_b = sum(n * (8 * (Cp if head and l == L - 1 else dims[l + 1]) + 2 * dims[l] + 4 * dims[l]) +
               4 * Mtr * 2 * dims[l] * dims[l + 1] for l in range(1, L))
    gd_f = sum(2 * n * 2 * dims[l] * dims[l + 1] for l in range(1, L))
    work["gemm_dgrad"] = ("gemm", steps * gd_b, steps * gd_f)
    P = sum((2 * dims[l] + 1) * dims[l + 1] for l in range(L))
    # scores in (head form: the row's own product and the aggregated one), gradient out, label
    work["softmax_xent"] = ("hbm", steps * ((12 * n * Cp if head else 8 * n * C) + 4 * n), 0.0)
    work["reduce_sgd"] = ("hbm", steps * 12.0 * Mtr * P, 0.0)
    work["aggregate"] = ("hbm", R * 8.0 * Mtr * P, 0.0)
    return work


# ---------------------------------------------------------------------------------------
# clock sampling during the timed region
# ---------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []      # (arrival time, line)
        self.thread = None
        self.t_begin = None  # the timed region, on the host's monotonic clock
        self.t_end = None

    def begin(self):
        """The timed region starts now (the sampler itself is started earlier: nvidia-smi takes a
        few hundred milliseconds to deliver its first sample)."""
        self.t_begin = time.monotonic()

    def end(self):
        self.t_end = time.monotonic()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        lo = self.t_begin if self.t_begin is not None else float("-inf")
        hi = (self.t_end if self.t_end is not None else float("inf")) + 0.1   # a sample arrives up to one period late
        for at, ln in self.lines:
            if not (lo <= at <= hi):
                continue
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------
# CPU baseline: the checker program as it stands, on a bounded sample
# ---------------------------------------------------------------------------------------
def host_info():
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as f:
            for ln in f:
                if ln.lower().startswith("model name"):
                    model = ln.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"nproc": os.cpu_count(), "cpu_model": model}


def cpu_sample(w, local_steps=1, flop_budget=1.2e10):
    """Times the CPU checker, as it stands and on one core, on a bounded sample of the workload:
    the assignment and relabelling of ALL nodes; the induced subgraph and the gathered feature /
    label rows of trainer 0's part only; `local_steps` local steps on the first `slice_rows` rows
    of that part (entries between those rows).  The whole-workload figure is extrapolated:
    preprocessing as t_assign + M * t_part0, training by rows (the checker spends > 99 % of a step
    in the per-row dense products)."""
    import oracle
    g = w.graph
    L = len(w.dims) - 1
    t0 = time.perf_counter()
    part_id, part_offsets, perm, local_id = oracle.partition(g.n, g.group_id if w.use_groups else None,
                                                             w.partition_seed, w.M, grouped=w.use_groups and w.grouped_order)
    t_assign = time.perf_counter() - t0
    n0 = int(part_offsets[1])
    t0 = time.perf_counter()
    # trainer 0's part alone: the checker's routine with a single part whose members are perm[0:n0]
    rowptr0, col0, _, kept0, _ = oracle.induced_csr(g.rowptr, g.col, 1, part_id, np.array([0, n0], dtype=np.int64),
                                                    perm, local_id)
    X0 = oracle.gather_rows(w.X, perm[:n0])
    y0 = oracle.gather_rows(w.y, perm[:n0])
    t_part0 = time.perf_counter() - t0
    # rows whose step costs the checker about three seconds (6 flops per weight and row)
    flops_per_row = 6.0 * sum((2 * w.dims[l] + 1) * w.dims[l + 1] for l in range(L))
    S = min(n0, max(1024, int(flop_budget / flops_per_row)))
    rp = rowptr0[:S + 1]
    cols = col0[:int(rp[-1])]
    inside = cols < S                                          # entries between the slice's rows
    rows = np.repeat(np.arange(S), np.diff(rp))
    srp = np.concatenate([[0], np.cumsum(np.bincount(rows[inside], minlength=S))]).astype(np.int64)
    scol = np.ascontiguousarray(cols[inside])
    t1 = time.perf_counter()
    oracle.local_steps_variant(w.variant, w.dims, w.lr, srp, scol, X0[:S], y0[:S], w.params0, local_steps)
    t_slice = (time.perf_counter() - t1) / local_steps
    # kept entries of the whole workload: expected value for the assignment in use, from part 0
    kept_est = float(kept0) * g.n / max(n0, 1)
    passes = 2 * L - 1
    units_full = kept_est * passes * w.K * w.R
    t_step_all_parts = t_slice * g.n / max(S, 1)               # one local step of every trainer
    est_full_s = t_assign + w.M * t_part0 + w.K * w.R * t_step_all_parts
    return dict(value=units_full / est_full_s, sample_s=t_assign + t_part0 + t_slice * local_steps,
                trainer_steps_per_s=w.M / t_step_all_parts,
                sample=(f"assignment+relabel of all {g.n} nodes ({t_assign:.2f} s); induced subgraph + row gather of "
                        f"trainer 0's part ({n0} nodes, {kept0} kept entries; {t_part0:.2f} s); {local_steps} local "
                        f"step(s) on its first {S} rows ({scol.size} entries; {t_slice:.2f} s/step); whole workload "
                        f"extrapolated as t_assign + M*t_part0 + K*R*(n/{S})*t_slice"))


def run_reference(args, w):
    """`--impl reference`: the CPU checker, single-threaded, timed on the host cores."""
    steps, warmup = args.steps, args.warmup
    for _ in range(min(warmup, 1)):     # the checker has no caches to warm beyond the first touch of its inputs
        cpu_sample(w)
    t0 = time.perf_counter()
    samples = [cpu_sample(w) for _ in range(steps)]
    wall = time.perf_counter() - t0
    value = statistics.mean(s["value"] for s in samples)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": 1e3 * wall / max(steps, 1), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "nodes": w.graph.n, "entries": w.graph.num_entries, "M": w.M,
                   "dims": list(w.dims), "K": w.K, "R": w.R, "timing": "host wall clock, bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": samples[-1]["sample"],
                         "host": host_info()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "trainer_steps_per_s": statistics.mean(s["trainer_steps_per_s"] for s in samples),
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------
def make_workload(args):
    from paper_2305_09887_b200 import inputs
    s = args.scale
    if args.workload == "medium":
        w = inputs.medium(1.0 if s is None else s)
    elif args.workload == "supertma":
        w = inputs.supertma(1.0 if s is None else s, M=args.M or 16)
    elif args.workload == "sweep":
        w = inputs.supertma(1.0 if s is None else s, width=512, M=args.M or 16,
                            use_groups=args.assign == "super", gemm_dtype=1)
    else:
        w = inputs.large(1.0 if s is None else s)
    w.grouped_order = args.order == "group"   # only matters with super-node assignment
    variant = (1 if args.encoder == "gcn" else 0, 1 if args.act == "prelu" else 0, 1 if args.norm == "layernorm" else 0)
    if variant != (0, 0, 0):   # the paper's own encoders (Sec. 4.1) on the same graph, features and widths
        w.variant = variant
        w.params0 = inputs.variant_params(variant, w.dims, inputs.SEED_WEIGHT + 7)
        w.name += "_" + "-".join([args.encoder, args.act, args.norm])
    return w


def run_averaging_stress(args, local_rank):
    """`--workload averaging`: the aggregation kernel alone on a shape large enough to be bound by
    HBM (M = 32 replicas of 16 Mi parameters, 2 GiB read and 2 GiB written per launch; the named
    workloads average at most 4.4 MB).  One step = one rtma_aggregate."""
    import torch
    from paper_2305_09887_b200 import binding
    torch.cuda.set_device(local_rank)
    ctx = binding.Context(local_rank)
    M, P = args.M or 32, 16 << 20
    params = torch.randn(M, P, dtype=torch.float32, device="cuda")
    glob = torch.empty(P, dtype=torch.float32, device="cuda")
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        ctx.aggregate(params, glob)
    torch.cuda.synchronize()
    # one launch takes 0.7 ms: time at least 400 of them, so that the clock sampler (100 ms period) sees the region
    args.steps = max(args.steps, 400)
    time.sleep(0.5)                      # the sampler's first sample takes a few hundred milliseconds
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.begin()
    e0.record()
    for _ in range(args.steps):
        ctx.aggregate(params, glob)
    e1.record()
    torch.cuda.synchronize()
    sampler.end()
    ctx.check()
    clocks = sampler.stop()
    seconds = e0.elapsed_time(e1) / 1e3
    peaks = load_peaks()
    abytes = 4.0 * P * (2 * M + 1)          # every replica read once and overwritten, the global copy written
    achieved = abytes * args.steps / seconds / 1e9
    print(json.dumps({
        "metric": "averaging_bytes_per_s", "value": abytes * args.steps / seconds, "unit": "B/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": 1e3 * seconds / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "averaging_stress", "M": M, "P": P, "l2": "4 GiB touched per launch > L2"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS,
                     "traffic": load_dram_traffic().get(("averaging_stress", "aggregate")), "kernel": "aggregate",
                     "peak_source": peaks["source"]},
        "gpu_launches": args.steps, "clocks": clocks}))


def run_link(args, rank, local_rank, world):
    """`--task link`: the paper's own task on the workload's graph and features.  One step = the
    whole path (partition, induced CSR, row gather, R x (K link-prediction steps on all M parts +
    aggregation)).  Encoder: the workload's widths with the last layer as wide as the hidden ones
    (--encoder / --act / --norm pick the variant); decoder: two layers of that width; pairs: up to
    65,536 edges of each part as positives plus one random-tail negative each, drawn once."""
    import torch
    import torch.distributed as dist
    from paper_2305_09887_b200 import binding, inputs

    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    args.warmup = max(args.warmup, 3)
    w = make_workload(args)
    g = w.graph
    hid = w.dims[1]
    dims, ddims = tuple(w.dims[:-1]) + (hid,), (hid, hid, 1)
    L = len(dims) - 1
    params0 = inputs.link_params(w.variant, dims, ddims, inputs.SEED_WEIGHT + 9)
    P = params0.size
    ctx = binding.Context(local_rank)
    assert P == binding.link_param_count(dims, ddims, w.variant)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    host = dict(rowptr=pin(g.rowptr), col=pin(g.col), X=pin(w.X), p0=pin(params0),
                gid=pin(g.group_id) if w.use_groups else None)
    res = {k: (v.to(device) if v is not None else None) for k, v in host.items()}

    def preprocess():
        part_id, part_offsets, perm, local_id = ctx.partition(g.n, res["gid"], w.partition_seed, w.M, grouped=w.grouped_order)
        rowptr_out, col_out, edge_offsets, kept_cut, edge_host = ctx.build_induced_csr(
            res["rowptr"], res["col"], w.M, part_id, part_offsets, perm, local_id)
        Xp = ctx.gather_rows(res["X"], perm)
        return part_offsets, rowptr_out, col_out, edge_offsets, edge_host, Xp

    # the training pairs are inputs: drawn once from the parts' subgraphs, outside the timed region
    part_offsets, rowptr_out, col_out, edge_offsets, edge_host, _ = preprocess()
    pu, pv, lab, pair_off = inputs.link_pairs(rowptr_out.cpu().numpy(), col_out.cpu().numpy(), part_offsets.cpu().numpy(),
                                              np.asarray(edge_host), w.M, 77, 65536)
    host.update(pu=pin(pu), pv=pin(pv), lab=pin(lab))
    res.update(pu=host["pu"].to(device), pv=host["pv"].to(device), lab=host["lab"].to(device))
    params = torch.empty(w.M, P, dtype=torch.float32, device=device)
    loss = torch.zeros(w.R, w.M, w.K, dtype=torch.float32, device=device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    state = {}

    def step():
        params.copy_(res["p0"].expand(w.M, P))
        part_offsets, rowptr_out, col_out, edge_offsets, edge_host, Xp = preprocess()
        part_host = part_offsets.cpu().tolist()
        for r in range(w.R):
            ctx.link_steps(dims, ddims, w.lr, w.M, part_host, edge_host, rowptr_out, col_out, Xp, pair_off,
                           res["pu"], res["pv"], res["lab"], params, w.K, loss_out=loss[r], gemm_dtype=w.gemm_dtype,
                           variant=w.variant)
            ctx.aggregate(params)
        state.update(edge_host=edge_host)

    def timed(fn, n):
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        for i in range(n):
            flush.fill_(i & 0xFF)
            starts[i].record()
            fn()
            stops[i].record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return max_over_ranks(sum(a.elapsed_time(b) for a, b in zip(starts, stops)) / 1e3, dist if world > 1 else None, device)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    ctx.profile_read()
    sampler = ClockSampler(local_rank)
    sampler.start()
    ctx.profile(True)
    elapsed_s = timed(step, args.steps)
    ctx.profile(False)
    prof = ctx.profile_read()
    clocks = sampler.stop()

    def host_step():   # inputs from pinned host memory every step, result read back
        for k in ("rowptr", "col", "X", "p0", "gid", "pu", "pv", "lab"):
            if host[k] is not None:
                res[k].copy_(host[k], non_blocking=True)
        step()
        state["out"] = (params[0].cpu(), loss.cpu())

    e2e_steps = max(1, min(args.steps, 3))
    host_step()
    e2e_s = timed(host_step, e2e_steps)
    h2d = sum(v.numel() * v.element_size() for v in host.values() if v is not None)
    d2h = P * 4 + loss.numel() * 4 + 2 * 8 * (w.M + 1)

    kept = float(state["edge_host"][-1])
    passes = 2 * L - 1
    units = kept * passes * w.K * w.R
    total_ms = sum(ms for ms, _ in prof.values())
    top = max(prof, key=lambda k: prof[k][0])
    peaks = load_peaks()
    if rank == 0:
        line = {
            "metric": METRIC, "value": world * args.steps * units / elapsed_s, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * elapsed_s / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16x3-split products, f32 accumulate and elementwise", "data": "synthetic",
            "config": {"workload": w.name + "_link", "task": "link prediction", "nodes": g.n, "entries": g.num_entries,
                       "kept_entries": int(kept), "M": w.M, "dims": list(dims), "decoder": list(ddims), "K": w.K, "R": w.R,
                       "pairs": int(pair_off[-1]), "variant": {"encoder": args.encoder, "act": args.act, "norm": args.norm},
                       "parallelism": "replicas only" if world > 1 else f"single GPU, {w.M} trainers batched on one stream",
                       "l2": "256 MB written between timed steps"},
            "trainer_steps_per_s": world * args.steps * w.M * w.K * w.R / elapsed_s,
            "pairs_per_s": world * args.steps * pair_off[-1] * w.K * w.R / elapsed_s,
            "loss_first_last": [loss[0, :, 0].mean().item(), loss[-1, :, -1].mean().item()],
            "roofline": {"bound": "hbm", "achieved": None, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": None,
                         "traffic": None, "kernel": top, "share_of_kernel_time": prof[top][0] / total_ms,
                         "peak_source": peaks["source"]},
            "kernels": {k: {"ms_per_step": ms / args.steps, "launches_per_step": cnt / args.steps, "share": ms / total_ms}
                        for k, (ms, cnt) in prof.items() if cnt},
            "gpu_launches": int(sum(cnt for _, cnt in prof.values())), "clocks": clocks,
            "e2e": {"value": world * e2e_steps * units / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(d2h), "ms_per_step": 1e3 * e2e_s / e2e_steps, "steps": e2e_steps},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def kernel_sources_digest(files) -> str:
    """Digest of the named CUDA sources: ncu counters taken on other sources are not reported."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2305_09887_b200", "csrc")
    for name in sorted(files):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()[:16]


def load_dram_traffic():
    """{(workload, kernel class): DRAM bytes per launch} from the ncu capture recorded in
    profiles/dram_traffic.txt (lines: workload, class, bytes per launch, digest, the comma-separated
    sources of the class's kernels the digest was taken over).  Entries whose sources have changed
    since the capture are dropped."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    out = {}
    if not os.path.exists(path):
        return out
    with open(path) as f:
        for ln in f:
            parts = ln.split()
            if len(parts) == 5 and not ln.startswith("#"):
                try:
                    if kernel_sources_digest(parts[4].split(",")) == parts[3]:
                        out[(parts[0], parts[1])] = float(parts[2])
                except OSError:
                    pass
    return out


def max_over_ranks(seconds: float, dist_mod=None, device=None) -> float:
    """Largest value over all ranks (the slowest rank sets the job's time)."""
    if dist_mod is None or not dist_mod.is_initialized() or dist_mod.get_world_size() == 1:
        return seconds
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device if device is not None else "cpu")
    dist_mod.all_reduce(t, op=dist_mod.ReduceOp.MAX)
    return float(t.item())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="large", choices=["large", "medium", "supertma", "sweep", "averaging"])
    ap.add_argument("--profile-steps", type=int, default=1,
                    help="steps of the separate pass that times every kernel class (CUDA events round each launch)")
    ap.add_argument("--scale", type=float, default=None, help="shrink (or grow) the workload's graph")
    ap.add_argument("--M", type=int, default=None, help="trainers (supertma / sweep)")
    ap.add_argument("--assign", default="super", choices=["node", "super"], help="sweep: assignment scheme")
    ap.add_argument("--order", default="group", choices=["id", "group"],
                    help="rows inside a part: by node id, or super-nodes kept together (super-node assignment only)")
    ap.add_argument("--task", default="node", choices=["node", "link"],
                    help="node classification (the named workloads) or link prediction (the paper's task)")
    ap.add_argument("--encoder", default="sage", choices=["sage", "gcn"])
    ap.add_argument("--act", default="relu", choices=["relu", "prelu"])
    ap.add_argument("--norm", default="none", choices=["none", "layernorm"])
    ap.add_argument("--aggregation", default="auto", choices=["auto", "gather", "tiles"],
                    help="mean aggregation: per part by itself (default), always by gathering, or tensor-core tiles for every part")
    ap.add_argument("--streams", type=int, default=1,
                    help="CUDA streams the trainers are spread over (trainers sharing a stream are batched)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, make_workload(args))
        return

    if args.workload == "averaging":
        if rank == 0:
            run_averaging_stress(args, local_rank)
        return
    if args.task == "link":
        run_link(args, rank, local_rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2305_09887_b200 import binding

    if args.warmup < 3:
        args.warmup = 3
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    w = make_workload(args)
    g = w.graph
    L = len(w.dims) - 1
    ctx = binding.Context(local_rank)
    ctx.set_dense_aggregation({"auto": 1, "gather": 0, "tiles": 2}[args.aggregation])
    resident = dict(rowptr=torch.from_numpy(g.rowptr).to(device), col=torch.from_numpy(g.col).to(device),
                    X=torch.from_numpy(w.X).to(device), y=torch.from_numpy(w.y).to(device),
                    gid=torch.from_numpy(g.group_id).to(device) if w.use_groups else None)
    d_params0 = torch.from_numpy(w.params0).to(device)
    P = w.params0.size
    params = torch.empty(w.M, P, dtype=torch.float32, device=device)
    loss = torch.zeros(w.R, w.M, w.K, dtype=torch.float32, device=device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)  # > 126 MB of L2
    n_streams = max(1, min(args.streams, w.M))
    pool = [torch.cuda.Stream(device=device) for _ in range(n_streams)] if n_streams > 1 else None
    trainer_streams = [pool[i * n_streams // w.M] for i in range(w.M)] if pool else None
    state = {}

    def step():
        params.copy_(d_params0.expand(w.M, P))                      # W_global[0] broadcast to the trainers
        part_id, part_offsets, perm, local_id = ctx.partition(g.n, resident["gid"], w.partition_seed, w.M, grouped=w.grouped_order)
        rowptr_out, col_out, edge_offsets, kept_cut, edge_host = ctx.build_induced_csr(
            resident["rowptr"], resident["col"], w.M, part_id, part_offsets, perm, local_id)
        yp = ctx.gather_rows(resident["y"], perm)
        part_host = part_offsets.cpu().tolist()
        for r in range(w.R):
            if pool:  # the trainers' streams start after the preprocessing / the previous aggregation
                for st in pool:
                    st.wait_stream(torch.cuda.current_stream())
            # the features stay in node order: the training call gathers them through perm
            ctx.local_steps(w.dims, w.lr, w.M, part_host, edge_host, rowptr_out, col_out, resident["X"], yp, params, w.K,
                            loss_out=loss[r], gemm_dtype=w.gemm_dtype, streams=trainer_streams, variant=w.variant, perm=perm)
            if pool:
                for st in pool:
                    torch.cuda.current_stream().wait_stream(st)
            ctx.aggregate(params)
        state.update(part_host=part_host, edge_host=edge_host)

    sampler = ClockSampler(local_rank)
    sampler.start()                      # started before the warm-up, windowed to the timed region below
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    ctx.check()
    ctx.profile_read()

    # ---- the timed region: K steps, no per-launch instrumentation ------------------------
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.begin()
    for i in range(args.steps):
        flush.fill_(i & 0xFF)                                       # evict L2 between timed steps
        starts[i].record()
        step()
        stops[i].record()
    torch.cuda.synchronize()
    sampler.end()
    if world > 1:
        dist.barrier()
    ctx.check()                          # a kernel that gave up on a bounded wait voids the run
    _, launch_counts = zip(*ctx.profile_read().values())
    gpu_launches = int(sum(launch_counts))
    clocks = sampler.stop()
    elapsed_s = sum(a.elapsed_time(b) for a, b in zip(starts, stops)) / 1e3
    elapsed_s = max_over_ranks(elapsed_s, dist if world > 1 else None, device)

    # ---- a separate pass with CUDA events round every launch: time per kernel class ---------
    prof_steps = max(1, args.profile_steps)
    ctx.profile(True)
    for i in range(prof_steps):
        flush.fill_(i & 0xFF)
        step()
    torch.cuda.synchronize()
    ctx.profile(False)
    ctx.check()
    prof = ctx.profile_read()

    n_parts = np.diff(state["part_host"]).tolist()
    e_parts = np.diff(state["edge_host"]).tolist()
    kept = float(sum(e_parts))
    passes = 2 * L - 1
    units_per_step = kept * passes * w.K * w.R
    trainer_steps = w.M * w.K * w.R
    value = world * args.steps * units_per_step / elapsed_s
    final_loss = loss[-1, :, -1].mean().item()
    first_loss = loss[0, :, 0].mean().item()

    # ---- roofline of the dominant kernel class, and of the aggregation (SpMM) classes ------
    peaks = load_peaks()
    work = (algorithmic_work(w.dims, n_parts, e_parts, w.K, w.R, entries=g.num_entries, rowptr_bytes=g.rowptr.itemsize,
                             grouped=w.use_groups and w.grouped_order) if w.variant == (0, 0, 0) else {})
    total_kernel_ms = sum(ms for ms, _ in prof.values())
    shares = {k: ms / total_kernel_ms for k, (ms, _) in prof.items() if ms > 0}
    top = max(shares, key=shares.get)
    # A layer product is three bf16 MMAs (hi*hi + lo*hi + hi*lo): the tensor pipe executes 3x the
    # algorithmic flops.  Its roofline is whichever is slower for the algorithmic work: the operand
    # bytes at the HBM peak or 3x the flops at the bf16 peak (sustained figure: timed inside a long step).
    MMAS_PER_PRODUCT = 1 if w.gemm_dtype == 1 else 3
    traffic_table = load_dram_traffic()

    def roofline_of(cls):
        ms, launches = prof[cls]
        roof = {"bound": "hbm", "achieved": None, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
        if cls in work and ms > 0:
            bound, abytes, aflops = work[cls]
            seconds = ms / 1e3
            if bound == "gemm":
                t_hbm = abytes / (peaks["hbm_gbs"] * 1e9)
                t_tensor = MMAS_PER_PRODUCT * aflops / (peaks["bf16_tflops_sustained"] * 1e12)
                bound = "hbm" if t_hbm >= t_tensor else "tensor"
            if bound == "hbm":
                roof = {"bound": "hbm", "achieved": abytes * prof_steps / seconds / 1e9, "peak": peaks["hbm_gbs"],
                        "unit": "GB/s"}
                roof["frac_of_nominal_8TBps"] = roof["achieved"] / NOMINAL_HBM_GBS
            else:
                roof = {"bound": "tensor", "achieved": aflops * prof_steps / seconds / 1e12,
                        "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                        "note": f"algorithmic flops; the tensor pipe executes {MMAS_PER_PRODUCT} bf16 MMA(s) per product"}
        roof.update({"frac": (roof["achieved"] / roof["peak"]) if roof["achieved"] else None,
                     "traffic": traffic_table.get((w.name, cls)), "kernel": cls,
                     "launches_per_step": launches / prof_steps, "avg_launch_us": 1e3 * ms / max(launches, 1),
                     "share_of_kernel_time": shares.get(cls), "peak_source": peaks["source"],
                     "timing": f"CUDA events round every launch of the class, {prof_steps} step(s) after the timed region"})
        return roof

    roof = roofline_of(top)
    spmm_ms = prof["spmm_forward"][0] + prof["spmm_backward"][0]
    spmm_bytes = sum(work[k][1] for k in ("spmm_forward", "spmm_backward") if k in work)
    roof_spmm = {"bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"], "peak_source": peaks["source"],
                 "kernels": {k: roofline_of(k) for k in ("spmm_forward", "spmm_backward") if prof[k][1]}}
    if spmm_ms > 0 and spmm_bytes > 0:
        roof_spmm["achieved"] = spmm_bytes * prof_steps / (spmm_ms / 1e3) / 1e9
        roof_spmm["frac"] = roof_spmm["achieved"] / peaks["hbm_gbs"]
        roof_spmm["frac_of_nominal_8TBps"] = roof_spmm["achieved"] / NOMINAL_HBM_GBS
        roof_spmm["share_of_kernel_time"] = spmm_ms / total_kernel_ms
    per_class = {}
    for k, (ms, cnt) in prof.items():
        if cnt == 0:
            continue
        entry = {"ms_per_step": ms / prof_steps, "launches_per_step": cnt / prof_steps,
                 "share": ms / total_kernel_ms if total_kernel_ms else None}
        if k in work and ms > 0 and work[k][1] > 0:
            bound, abytes, aflops = work[k]
            entry["GBps"] = abytes * prof_steps / (ms / 1e3) / 1e9
            entry["frac_of_measured_hbm"] = entry["GBps"] / peaks["hbm_gbs"]
            entry["frac_of_nominal_8TBps"] = entry["GBps"] / NOMINAL_HBM_GBS
            if aflops:
                entry["TFLOPps"] = aflops * prof_steps / (ms / 1e3) / 1e12
        per_class[k] = entry
    # the partition as a whole: its count, scan and scatter launches (the scan class also holds the short
    # scan of the induced-subgraph offsets) against the 12 B per node it must write
    part_ms = sum(prof[k][0] for k in ("partition_count", "scan", "partition_scatter"))
    if part_ms > 0 and work:
        gbps = (work["partition_count"][1] + work["partition_scatter"][1]) * prof_steps / (part_ms / 1e3) / 1e9
        per_class["partition_total"] = {"ms_per_step": part_ms / prof_steps, "GBps": gbps,
                                        "frac_of_measured_hbm": gbps / peaks["hbm_gbs"],
                                        "frac_of_nominal_8TBps": gbps / NOMINAL_HBM_GBS}

    # ---- end to end through the host-buffer entry point ------------------------------
    resident.clear()              # the host-buffer call brings its own copies
    torch.cuda.empty_cache()
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory().numpy()
    h_rowptr, h_col, h_X, h_y, h_p0 = pin(g.rowptr), pin(g.col), pin(w.X), pin(w.y), pin(w.params0)
    e2e_steps = max(1, min(args.steps, 3))
    h_gid = pin(g.group_id) if w.use_groups else None
    host_kw = dict(group_id=h_gid, gemm_dtype=w.gemm_dtype, variant=w.variant)
    ctx.train_host(h_rowptr, h_col, h_X, h_y, w.dims, w.M, w.K, w.R, w.lr, w.partition_seed, h_p0, **host_kw)  # warm-up
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    e0.record()
    for _ in range(e2e_steps):
        out_params, out_losses, _, _ = ctx.train_host(h_rowptr, h_col, h_X, h_y, w.dims, w.M, w.K, w.R, w.lr,
                                                      w.partition_seed, h_p0, **host_kw)
    e1.record()
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(e0.elapsed_time(e1) / 1e3, dist if world > 1 else None, device)
    h2d = h_rowptr.nbytes + h_col.nbytes + h_X.nbytes + h_y.nbytes + w.M * h_p0.nbytes + (h_gid.nbytes if w.use_groups else 0)
    d2h = out_params.nbytes + out_losses.nbytes + 16 + 2 * 8 * (w.M + 1)
    e2e_value = world * e2e_steps * units_per_step / e2e_s

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * elapsed_s / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("bf16 products, f32 accumulate and elementwise" if w.gemm_dtype == 1 else
                  "bf16x3-split products, f32 accumulate and elementwise"), "data": "synthetic",
        "config": {"workload": w.name, "nodes": g.n, "entries": g.num_entries, "kept_entries": int(kept), "M": w.M,
                   "dims": list(w.dims), "K": w.K, "R": w.R, "spmm_passes_per_local_step": passes,
                   "input_layer_aggregate": "computed once per local_steps call (constant over its K steps), "
                                            "counted once per step in the unit",
                   "variant": {"encoder": args.encoder, "act": args.act, "norm": args.norm},
                   "assignment": "super-node" if w.use_groups else "node",
                   "row_order": "super-node id, then node id" if (w.use_groups and w.grouped_order) else "node id",
                   "kept_fraction": kept / g.num_entries,
                   "parallelism": ("replicas only" if world > 1 else
                                   f"single GPU, {w.M} trainers batched on {n_streams} stream(s)"),
                   "aggregation": args.aggregation,
                   "l2": "256 MB written between timed steps"},
        "trainer_steps_per_s": world * args.steps * trainer_steps / elapsed_s,
        "edges_gathered_per_s": world * args.steps * kept * ((passes - 1) * w.K + 1) * w.R / elapsed_s,
        "loss_first_last": [first_loss, final_loss],
        "roofline": roof,
        "roofline_spmm": roof_spmm,
        "kernels": per_class,
        "gpu_launches": gpu_launches,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": 1e3 * e2e_s / e2e_steps, "steps": e2e_steps},
    }
    if world == 1 and not args.no_cpu_baseline:
        cb = cpu_sample(w, local_steps=2)
        line["cpu_baseline"] = {"value": cb["value"], "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": cb["sample"], "sample_seconds": cb["sample_s"],
                                "trainer_steps_per_s": cb["trainer_steps_per_s"], "host": host_info()}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
