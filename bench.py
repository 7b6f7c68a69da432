#!/usr/bin/env python
"""Benchmark of the HAG aggregation hot path on B200.

A step is one pass of the whole path over one synthetic workload: for every
layer the forward aggregation over the HAG (level pair-sum kernels, then the
gather over the residual rows) and then for every layer the backward aggregation
(gathers over the transposed HAG, last level first).  Inputs are resident in
HBM when the timed region starts; the L2 is flushed between timed steps (a
256 MiB write) so every step starts cold.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5]
    python bench.py --impl reference       # the fp64 CPU oracle on the host cores

Prints ONE JSON line.  With N > 1 (under torchrun) every rank runs the same
workload on its own GPU (independent problems, no data-path collective): weak
scaling, value = units of all ranks / max-over-ranks time.
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

METRIC = "HAG fwd+bwd aggregation GB/s"
# dram__bytes_read.sum + dram__bytes_write.sum of ONE forward-gather launch, from ncu captures of this
# program at the workload's full size (None: not captured)
NCU_DRAM_BYTES_FWD_GATHER = {"cfg2": 23.40e6 + 0.02e6, "cfg4": 228.2e6 + 105.5e6}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 256 << 20


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- #
# clocks
# --------------------------------------------------------------------------- #
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = sorted(sm)[len(sm) // 2:]          # upper half: samples taken under load
        return {"sm_mhz": float(np.median(busy)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- #
# bytes
# --------------------------------------------------------------------------- #
def algorithmic_bytes(n, d, dtype, arr, info):
    """Rows read + rows written per pass, at their stored width.  Rows of the
    aggregation nodes (a-hat / their gradients) are fp32 whatever the dtype."""
    s = 4 if dtype == "f32" else 2
    k = info["num_agg"]
    res_sec = int((arr["res_idx"] >= n).sum())
    agg_sec = int((arr["agg_in"] >= n).sum())
    e_res = int(arr["res_idx"].shape[0])
    reads_prim = (e_res - res_sec) + (2 * k - agg_sec)
    reads_sec = res_sec + agg_sec
    per_pass = d * (s * reads_prim + 4 * reads_sec + s * n + 4 * k)      # forward; backward moves the same rows
    plain = d * s * (info["e"] + n)
    fwd_gather = d * (s * (e_res - res_sec) + 4 * res_sec + s * n)       # the dominant launch
    return dict(hag_pass=per_pass, plain_pass=plain, fwd_gather=fwd_gather)


# --------------------------------------------------------------------------- #
# CPU oracle legs
# --------------------------------------------------------------------------- #
def oracle_step_factory(w, budget_edges=3.0e7):
    """One oracle 'step': direct fp64 forward + backward on a bounded sample of the
    workload's rows.  Returns (fn, fraction_of_workload, description)."""
    from oracle import oracle as O
    from paper_1906_03707_b200 import synth
    g = w.graph
    x = synth.features(w.seed, g.n, w.d, w.feat_dist, w.dtype).astype(np.float64)
    gr = synth.upstream_grad(w.seed, g.n, w.d, w.feat_dist, w.dtype).astype(np.float64)
    work = g.e * w.d / 64.0
    if work <= budget_edges:
        rows, frac, what = None, 1.0, "all rows"
    else:
        frac = budget_edges / work
        m = max(1, int(g.n * frac))
        rows = np.sort(np.random.default_rng(0).choice(g.n, m, replace=False))
        frac = m / g.n
        what = f"{m} of {g.n} rows drawn uniformly (forward and backward each)"

    def step():
        for _ in range(w.layers):
            O.direct_forward(g.row_ptr, g.col_idx, x, w.reduce, rows=rows)
        for _ in range(w.layers):
            O.direct_backward(g.row_ptr, g.col_idx, gr, w.reduce, rows=rows)

    return step, frac, what


def run_reference(args, w, bytes_per_step_fn):
    """--impl reference: the oracle as it stands, timed on the host cores."""
    step, frac, what = oracle_step_factory(w)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    sec = (time.perf_counter() - t0) / max(args.steps, 1)
    bytes_step = bytes_per_step_fn() * frac
    value = bytes_step / sec / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: {w.graph.name}, N={w.graph.n}, E={w.graph.e}, D={w.d}, {w.dtype} storage, {w.reduce}, "
                               f"{w.layers} layer(s), fwd+bwd; the oracle evaluates the GNN-graph directly in fp64",
                   "sample": what},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- #
# main
# --------------------------------------------------------------------------- #
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2, help="1-5: the named shapes (2 = the 50 000-node clustered power-law graph); 6: clique-union graph")
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--capacity-frac", type=float, default=0.25)
    ap.add_argument("--min-redundancy", type=int, default=2,
                    help="stop the search below this redundancy (2 = the paper's rule; 4 = no merge that loses bytes)")
    ap.add_argument("--capacity-sweep", action="store_true",
                    help="also time capacities 0, N/8, N/4, N/2 from ONE search (hag_truncate); reported under capacity_sweep")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--permute-ids", action="store_true",
                    help="relabel the nodes by a seeded random permutation first (locality stress: communities no longer contiguous)")
    ap.add_argument("--max-leg", action="store_true",
                    help="also time the element-wise max aggregation (hag_max_fwd/bwd against csr_max_fwd/bwd); reported under max_aggregation")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_1906_03707_b200 import synth

    if args.impl == "reference":
        if rank != 0:
            return
        w = synth.workload(args.workload, scale=args.scale, capacity_frac=args.capacity_frac)
        s = 4 if w.dtype == "f32" else 2

        def plain_bytes():      # the oracle evaluates the GNN-graph directly
            return 2 * w.layers * w.d * s * (w.graph.e + w.graph.n)

        run_reference(args, w, plain_bytes)
        return

    import torch
    import torch.distributed as dist

    import paper_1906_03707_b200 as hb
    from paper_1906_03707_b200 import sharding
    from paper_1906_03707_b200.build import build as build_library

    build_library()
    hb.load_library()                       # raises if the CUDA library is missing: no fallback
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (use --impl reference for the CPU oracle)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = synth.workload(args.workload, scale=args.scale, capacity_frac=args.capacity_frac)
    if args.permute_ids:
        w.graph = synth.permute_ids(w.graph, seed=w.seed + 77)
    g = w.graph
    t0 = time.perf_counter()
    h = hb.Hag.build(g.row_ptr, g.col_idx, w.capacity, min_redundancy=args.min_redundancy).to_device(local_rank)
    build_s = time.perf_counter() - t0
    info = h.info()
    arr = h.arrays()
    nbytes = algorithmic_bytes(g.n, w.d, w.dtype, arr, info)
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    x = torch.from_numpy(synth.features(w.seed, g.n, w.d, w.feat_dist, w.dtype)).to(dev).to(tdt)
    gr = torch.from_numpy(synth.upstream_grad(w.seed, g.n, w.d, w.feat_dist, w.dtype)).to(dev).to(tdt)
    bufs = [torch.empty_like(x) for _ in range(2 * w.layers)]
    ws_bytes = max(h.workspace_bytes(w.d), h.csr_workspace_bytes(w.d))
    ws = torch.empty(max(ws_bytes // 4, 4), dtype=torch.float32, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)

    def step(hag: bool):
        launches = 0
        cur = x
        for l in range(w.layers):
            if hag:
                h.aggregate_fwd(cur, w.reduce, out=bufs[l], workspace=ws)
            else:
                h.csr_fwd(cur, w.reduce, out=bufs[l], workspace=ws)
            launches += h.last_launch_count
            cur = bufs[l]
        cur = gr
        for l in range(w.layers):
            o = bufs[w.layers + l]
            if hag:
                h.aggregate_bwd(cur, w.reduce, out=o, workspace=ws)
            else:
                h.csr_bwd(cur, w.reduce, out=o, workspace=ws)
            launches += h.last_launch_count
            cur = o
        return launches

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()

    def timed(hag: bool, steps: int, cold: bool):
        """Sum of the per-step device times (events on the launching stream); the L2 flush sits between steps."""
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        launches = 0
        barrier()
        for i in range(steps):
            if cold:
                flush.zero_()
            starts[i].record(stream)
            launches += step(hag)
            stops[i].record(stream)
        barrier()
        ms = sharding.max_over_ranks(sum(a.elapsed_time(b) for a, b in zip(starts, stops)), dev)
        return ms / max(steps, 1), launches

    for _ in range(args.warmup):
        step(True)
        step(False)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    hag_ms, launches = timed(True, args.steps, cold=True)
    csr_ms, _ = timed(False, args.steps, cold=True)
    hag_warm_ms, _ = timed(True, args.steps, cold=False)
    csr_warm_ms, _ = timed(False, args.steps, cold=False)

    # the dominant kernel, timed live with event pairs around every launch
    h.profile(True)
    kinds = {0: [], 1: [], 2: []}
    fwd_gather, bwd_gather = [], []
    for _ in range(args.steps):
        flush.zero_()
        h.aggregate_fwd(x, w.reduce, out=bufs[0], workspace=ws)
        rec = h.profile_read()
        for ms, kind, _, _ in rec:
            kinds[kind].append(ms)
        fwd_gather.append(rec[-1][0])
        h.aggregate_bwd(gr, w.reduce, out=bufs[w.layers], workspace=ws)
        rec = h.profile_read()
        for ms, kind, _, _ in rec:
            kinds[kind].append(ms)
        bwd_gather.append(rec[-1][0])
    h.profile(False)
    # a timed arm lasts milliseconds, below nvidia-smi's sampling period: the sampler ran across all GPU arms
    clocks = sampler.stop() if rank == 0 else {}
    peak, peak_kind = measured_peak()
    fg_ms = float(np.mean(fwd_gather))
    achieved = nbytes["fwd_gather"] / (fg_ms * 1e-3) / 1e9

    # end to end through the host-buffer entry point: pinned host inputs and outputs
    e2e = None
    if not args.no_e2e:
        xh = x.cpu().pin_memory()
        gh = gr.cpu().pin_memory()
        oh = [torch.empty_like(xh).pin_memory() for _ in range(2 * w.layers)]

        def host_step():
            cur = xh
            for l in range(w.layers):
                h.aggregate_host(cur, oh[l], w.reduce, backward=False, use_hag=True)
                cur = oh[l]
                if w.layers > 1:
                    torch.cuda.synchronize(dev)      # the next layer reads this host buffer
            cur = gh
            for l in range(w.layers):
                h.aggregate_host(cur, oh[w.layers + l], w.reduce, backward=True, use_hag=True)
                cur = oh[w.layers + l]
                if w.layers > 1:
                    torch.cuda.synchronize(dev)

        for _ in range(3):
            host_step()
        barrier()
        t0 = time.perf_counter()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            host_step()
        e1.record(stream)
        barrier()
        e2e_ms = sharding.max_over_ranks(e0.elapsed_time(e1) / max(args.steps, 1), dev)
        io = 2 * w.layers * x.numel() * x.element_size()
        e2e = {"value": world * 2 * w.layers * nbytes["hag_pass"] / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s",
               "h2d_bytes_per_step": io, "d2h_bytes_per_step": io, "ms_per_step": e2e_ms,
               "api": "hag_aggregate_host (pinned host buffers in and out, copies inside the timed region)"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        ostep, frac, what = oracle_step_factory(w)
        ostep()
        reps, t0 = 0, time.perf_counter()
        while reps < 3 or time.perf_counter() - t0 < 10.0:
            ostep()
            reps += 1
            if time.perf_counter() - t0 > 30.0:
                break
        sec = (time.perf_counter() - t0) / reps
        s = 4 if w.dtype == "f32" else 2
        plain_step = 2 * w.layers * w.d * s * (g.e + g.n)
        cpu = {"value": plain_step * frac / sec / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
               "sample": f"{what}; {reps} repetitions; bytes counted as (|E|+N)*D*{s} per pass like the GPU's plain path",
               "ms_per_step_full_workload": sec / frac * 1e3}

    sweep = None
    if args.capacity_sweep and rank == 0:
        # Section 5.4's capacity study: one search at N/2, every smaller capacity is a prefix of its merges
        t0 = time.perf_counter()
        big = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 2)
        search_s = time.perf_counter() - t0
        sweep = {"search_seconds_at_half_n": search_s, "points": []}
        keep_h, keep_ws = h, ws
        for frac_name, cap in (("0", 0), ("N/8", g.n // 8), ("N/4", g.n // 4), ("N/2", g.n // 2)):
            hc = big.truncate(cap).to_device(local_rank)
            ic, ac = hc.info(), hc.arrays()
            nb = algorithmic_bytes(g.n, w.d, w.dtype, ac, ic)
            h = hc
            ws = torch.empty(max(hc.workspace_bytes(w.d), hc.csr_workspace_bytes(w.d), 16) // 4, dtype=torch.float32, device=dev)
            for _ in range(3):
                step(True)
            ms, _ = timed(True, max(args.steps // 4, 5), cold=True)
            sweep["points"].append({"capacity": frac_name, "num_agg": ic["num_agg"], "levels": ic["num_levels"],
                                    "e_hat": ic["e_hat"], "ms_per_step": ms,
                                    "gbps": 2 * w.layers * nb["hag_pass"] / (ms * 1e-3) / 1e9,
                                    "speedup_vs_capacity_0": None})
            hc.close()
        h, ws = keep_h, keep_ws
        base_ms = sweep["points"][0]["ms_per_step"]
        for pt in sweep["points"]:
            pt["speedup_vs_capacity_0"] = base_ms / pt["ms_per_step"]

    readout = None
    meta = getattr(g, "meta", None) or {}
    if rank == 0 and "graph_size" in meta and g.n % int(meta["graph_size"]) == 0:
        # graph classification (Section 5.1): the mean-pooling layer after the GNN layers, one row per graph
        size = int(meta["graph_size"])
        seg = torch.arange(0, g.n + 1, size, dtype=torch.int32, device=dev)
        pooled = torch.empty((g.n // size, w.d), dtype=x.dtype, device=dev)
        gpool = torch.empty_like(x)
        for _ in range(3):
            hb.graph_pool_fwd(seg, x, "mean", out=pooled)
            hb.graph_pool_bwd(seg, pooled, g.n, "mean", out=gpool)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
        torch.cuda.synchronize(dev)
        for e3 in ev:
            flush.zero_()
            e3[0].record(stream)
            hb.graph_pool_fwd(seg, x, "mean", out=pooled)
            e3[1].record(stream)
            hb.graph_pool_bwd(seg, pooled, g.n, "mean", out=gpool)
            e3[2].record(stream)
        torch.cuda.synchronize(dev)
        f_ms = float(np.mean([e3[0].elapsed_time(e3[1]) for e3 in ev]))
        b_ms = float(np.mean([e3[1].elapsed_time(e3[2]) for e3 in ev]))
        rb = (x.numel() + pooled.numel()) * x.element_size()        # each pass reads one matrix and writes the other
        readout = {"what": f"mean-pooling read-out, {g.n // size} graphs of {size} nodes, cold L2", "fwd_ms": f_ms, "bwd_ms": b_ms,
                   "fwd_gbps": rb / (f_ms * 1e-3) / 1e9, "bwd_gbps": rb / (b_ms * 1e-3) / 1e9,
                   "fwd_frac_of_measured_hbm": rb / (f_ms * 1e-3) / 1e9 / measured_peak()[0],
                   "bwd_frac_of_measured_hbm": rb / (b_ms * 1e-3) / 1e9 / measured_peak()[0]}

    maxagg = None
    if rank == 0 and args.max_leg:
        # the max Aggregate of Table 1 (GraphSAGE-P) over the same HAG, against the same kernels on the plain graph
        mo = torch.empty_like(x)
        mg = torch.empty_like(x)
        mws = [h.max_workspace(w.d, dev), h.max_workspace(w.d, dev)]

        def max_step(use_hag):
            h.max_fwd(x, out=mo, workspace=mws[0], use_hag=use_hag)
            n_l = h.last_launch_count
            h.max_bwd(x, mo, mws[0], gr, out=mg, workspace=mws[1], use_hag=use_hag)
            return n_l + h.last_launch_count

        res = {}
        for use_hag in (True, False):
            for _ in range(3):
                max_step(use_hag)
            ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(max(args.steps // 4, 5))]
            torch.cuda.synchronize(dev)
            for e3 in ev:
                flush.zero_()
                e3[0].record(stream)
                h.max_fwd(x, out=mo, workspace=mws[0], use_hag=use_hag)
                e3[1].record(stream)
                h.max_bwd(x, mo, mws[0], gr, out=mg, workspace=mws[1], use_hag=use_hag)
                e3[2].record(stream)
            torch.cuda.synchronize(dev)
            res[use_hag] = (float(np.mean([e3[0].elapsed_time(e3[1]) for e3 in ev])),
                            float(np.mean([e3[1].elapsed_time(e3[2]) for e3 in ev])))
        maxagg = {"what": "element-wise max aggregation, fwd and bwd timed apart, cold L2; forward bytes counted like the sum's",
                  "hag_fwd_ms": res[True][0], "hag_bwd_ms": res[True][1], "plain_fwd_ms": res[False][0], "plain_bwd_ms": res[False][1],
                  "hag_fwd_gbps": nbytes["hag_pass"] / (res[True][0] * 1e-3) / 1e9,
                  "plain_fwd_gbps": nbytes["plain_pass"] / (res[False][0] * 1e-3) / 1e9,
                  "speedup_hag_vs_plain_fwd": res[False][0] / res[True][0],
                  "speedup_hag_vs_plain_fwd_bwd": sum(res[False]) / sum(res[True])}

    if rank == 0:
        bytes_step = 2 * w.layers * nbytes["hag_pass"]
        value = world * bytes_step / (hag_ms * 1e-3) / 1e9
        plain_step = 2 * w.layers * nbytes["plain_pass"]
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": hag_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {
                "workload": f"{w.name}: {g.name}, N={g.n}, E={info['e']}, D={w.d}, {w.dtype} storage, {w.reduce}, "
                            f"|V_A|={info['num_agg']} (capacity {w.capacity}, stop below redundancy "
                            f"{args.min_redundancy}), {w.layers} layer(s), fwd+bwd",
                "l2": "flushed between timed steps (256 MiB write outside the per-step events)",
                "timing": "sum of per-step CUDA-event intervals on the launching stream, max over ranks",
                "clocks": "nvidia-smi sampled every 100 ms across the GPU arms (HAG/plain x cold/warm, per-kernel pass)",
            },
            "clocks": clocks,
            "e2e": e2e,
            "gpu_launches": launches,
            "pct_of_hbm_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
            "pct_of_hbm_measured": 100.0 * value / world / peak,
            "plain_csr": {"ms_per_step": csr_ms, "gbps": world * plain_step / (csr_ms * 1e-3) / 1e9,
                          "speedup_hag_vs_plain": csr_ms / hag_ms},
            "warm_l2": {"hag_ms_per_step": hag_warm_ms, "plain_ms_per_step": csr_warm_ms,
                        "hag_gbps": world * bytes_step / (hag_warm_ms * 1e-3) / 1e9},
            "hag": {"num_agg": info["num_agg"], "levels": info["num_levels"], "e_hat": info["e_hat"],
                    "aggregation_reduction": info["aggregations_gnn"] / max(info["aggregations_hag"], 1),
                    "read_reduction": info["e"] / max(info["e_hat"], 1),
                    "byte_reduction": nbytes["plain_pass"] / nbytes["hag_pass"],
                    "build_seconds": build_s, "bytes_per_step": bytes_step},
            "kernels_ms": {"level_pair_sum_total": float(np.sum(kinds[0])) / args.steps,
                           "bwd_level_gather_total": float(np.sum(kinds[1])) / args.steps,
                           "fwd_final_gather": fg_ms, "bwd_final_gather": float(np.mean(bwd_gather))},
            "roofline": {"bound": "hbm", "kernel": "gather_sum_kernel (forward gather over the residual rows)",
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": f"{peak_kind} copy bandwidth",
                         "traffic": NCU_DRAM_BYTES_FWD_GATHER.get(w.name) if (args.scale == 1.0 and not args.permute_ids) else None,
                         "algorithmic_bytes_per_launch": nbytes["fwd_gather"], "ms_per_launch": fg_ms},
            "cpu_baseline": cpu,
        }
        if sweep is not None:
            line["capacity_sweep"] = sweep
        if readout is not None:
            line["graph_readout"] = readout
        if maxagg is not None:
            line["max_aggregation"] = maxagg
        if w.dtype == "bf16":
            line["dtype"] = "f32 accumulate, bf16 storage"
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
