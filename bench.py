#!/usr/bin/env python
"""Benchmark of the HAG aggregation hot path on B200.

A step is one pass of the whole path over one synthetic workload: for every
layer the forward aggregation over the HAG (aggregation nodes, then the graph
nodes) and then for every layer the backward aggregation over the transposed
HAG.  Inputs are resident in HBM when the timed region starts; the L2 is
flushed between timed steps (a 256 MiB write) so every step starts cold.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..6]
    python bench.py --impl reference       # the fp64 CPU oracle on the host cores

Prints ONE JSON line.  The headline workload is cfg3 (the largest fp32 shape, two
stacked layers); the other shapes are measured in the same run and reported under
``per_config``.  With N > 1 (under torchrun) the default is one whole workload per
rank (independent problems, no data-path collective: weak scaling, value = units of
all ranks / max-over-ranks time); ``--shard graphs`` splits the graph-classification
batch by graph and ``--shard columns`` splits the feature columns of one graph
(strong scaling, still no exchange inside the aggregation).
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
DEFAULT_WORKLOAD = 3
SECONDARY_WORKLOADS = (2, 4, 5, 6)
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 256 << 20
# From the ncu captures summarised under profiles/ (the dominant launch: the gather over the graph nodes of one forward
# pass over the HAG, at the workload's full size): dram__bytes_read.sum + dram__bytes_write.sum per launch, and
# lts__throughput (percent of the L2's peak) of that launch.
NCU_FWD_GATHER = {
    "cfg3": {"dram_bytes": 599.9e6 + 114.4e6, "lts_throughput_pct": 79.2,
             "note": "profiles/gather_sum_persistent_cfg3.md: ncu --set full on this workload at full size"},
    "cfg4": {"dram_bytes": 244.1e6 + 105.1e6, "lts_throughput_pct": 63.5,
             "note": "profiles/gather_sum_sub_cfg4.md: ncu --set full on this workload at full size"},
    "cfg5": {"dram_bytes": 2109.6e6 + 514.7e6, "lts_throughput_pct": 64.5,
             "note": "profiles/gather_sum_bf16_cfg5.md: ncu --set full on this workload at full size"},
    "cfg2": {"dram_bytes": 23.6e6 + 0.2e6, "lts_throughput_pct": 45.8,
             "note": "profiles/gather_sum_sub_cfg2.md: ncu --set full on this workload at full size"},
    "clique-union": {"dram_bytes": 34.6e6 + 2.4e6, "lts_throughput_pct": 45.2,
                     "note": "profiles/gather_sum_sub_clique_union.md: ncu --set full on this workload at full size"},
}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def workload_string(w) -> str:
    """Names the workload the same way in both arms (nothing here depends on the built HAG)."""
    g = w.graph
    return (f"{w.name}: {g.name}, N={g.n}, E={g.e}, D={w.d}, {w.dtype} storage, {w.reduce}, capacity {w.capacity}, "
            f"{w.layers} layer(s), fwd+bwd")


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
    fwd_gather = d * (s * (e_res - res_sec) + 4 * res_sec + s * n)       # the dominant launch: gather over the graph nodes
    return dict(hag_pass=per_pass, plain_pass=plain, fwd_gather=fwd_gather)


# --------------------------------------------------------------------------- #
# CPU oracle legs
# --------------------------------------------------------------------------- #
def oracle_step_factory(w, budget=5.0e6, threads=1):
    """One oracle 'step': direct fp64 forward + backward of every layer on a bounded sample of the workload's
    rows.  With threads > 1 the sampled rows are cut into that many blocks, one oracle call per block and thread
    (the C loops release the interpreter lock); the oracle itself is untouched.
    Returns (fn, fraction_of_workload, description, threads used)."""
    from concurrent.futures import ThreadPoolExecutor

    from oracle import oracle as O
    from paper_1906_03707_b200 import synth
    g = w.graph
    x = synth.features(w.seed, g.n, w.d, w.feat_dist, w.dtype).astype(np.float64)
    gr = synth.upstream_grad(w.seed, g.n, w.d, w.feat_dist, w.dtype).astype(np.float64)
    work = g.e * w.d / 64.0 * w.layers
    if work <= budget:
        rows, frac, what = np.arange(g.n, dtype=np.int64), 1.0, "all rows"
    else:
        m = max(1, int(g.n * budget / work))
        rows = np.sort(np.random.default_rng(0).choice(g.n, m, replace=False))
        frac = m / g.n
        what = f"{m} of {g.n} rows drawn uniformly (forward and backward each)"
    blocks = [b for b in np.array_split(rows, max(1, threads)) if b.size]
    pool = ThreadPoolExecutor(max_workers=len(blocks)) if len(blocks) > 1 else None

    def one(block):
        for _ in range(w.layers):
            O.direct_forward(g.row_ptr, g.col_idx, x, w.reduce, rows=block)
        for _ in range(w.layers):
            O.direct_backward(g.row_ptr, g.col_idx, gr, w.reduce, rows=block)

    def step():
        if pool is None:
            one(blocks[0])
        else:
            list(pool.map(one, blocks))

    return step, frac, what, len(blocks)


def plain_bytes_per_step(w):
    s = 4 if w.dtype == "f32" else 2
    return 2 * w.layers * w.d * s * (w.graph.e + w.graph.n)      # the oracle evaluates the GNN-graph directly


def time_oracle(w, threads, min_seconds=6.0, max_seconds=20.0):
    step, frac, what, used = oracle_step_factory(w, threads=threads)
    step()
    reps, t0 = 0, time.perf_counter()
    while reps < 2 or time.perf_counter() - t0 < min_seconds:
        step()
        reps += 1
        if time.perf_counter() - t0 > max_seconds:
            break
    sec = (time.perf_counter() - t0) / reps
    s = 4 if w.dtype == "f32" else 2
    return {"value": plain_bytes_per_step(w) * frac / sec / 1e9, "unit": "GB/s", "cores": used, "kind": "oracle",
            "sample": f"{what}; {reps} repetitions; bytes counted as (|E|+N)*D*{s} per pass like the GPU's plain path",
            "ms_per_step_full_workload": sec / frac * 1e3}


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except Exception:
        pass
    return "unknown"


def run_reference(args, w):
    """--impl reference: the oracle as it stands, timed on the host cores."""
    step, frac, what, used = oracle_step_factory(w)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    sec = (time.perf_counter() - t0) / max(args.steps, 1)
    value = plain_bytes_per_step(w) * frac / sec / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_string(w)},
        "what": "the fp64 CPU oracle evaluates the GNN-graph directly (Algorithm 1 line 4 and its gradient)",
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": used, "kind": "oracle", "sample": what,
                         "cpu_model": cpu_model()},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- #
# one workload on the GPU
# --------------------------------------------------------------------------- #
class Runner:
    """One workload resident on one GPU: the handle, its tensors and the timed step."""

    def __init__(self, w, args, dev, local_rank, column_slice=None):
        import torch

        import paper_1906_03707_b200 as hb
        from paper_1906_03707_b200 import synth
        self.torch, self.w, self.dev = torch, w, dev
        g = w.graph
        t0 = time.perf_counter()
        h = hb.Hag.build(g.row_ptr, g.col_idx, w.capacity, min_redundancy=args.min_redundancy)
        if args.cuts:
            h.set_cuts(*(int(v) for v in args.cuts.split(",")))
        h.to_device(local_rank)
        h.set_schedule(args.schedule)
        self.build_s = time.perf_counter() - t0
        self.h = h
        self.info = h.info()
        self.d = w.d
        tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
        x = synth.features(w.seed, g.n, w.d, w.feat_dist, w.dtype)
        gr = synth.upstream_grad(w.seed, g.n, w.d, w.feat_dist, w.dtype)
        if column_slice is not None:                    # this rank's columns, as a contiguous matrix of its own
            c0, cn = column_slice
            x, gr = np.ascontiguousarray(x[:, c0:c0 + cn]), np.ascontiguousarray(gr[:, c0:c0 + cn])
            self.d = cn
        arr = h.arrays()
        self.cuts = (int(arr["fwd_cut"]), int(arr["bwd_cut"]))
        self.nbytes = algorithmic_bytes(g.n, self.d, w.dtype, arr, self.info)
        del arr
        self.x = torch.from_numpy(x).to(dev).to(tdt)
        self.gr = torch.from_numpy(gr).to(dev).to(tdt)
        self.bufs = [torch.empty_like(self.x) for _ in range(2 * w.layers)]
        ws_bytes = max(h.workspace_bytes(self.d), h.csr_workspace_bytes(self.d))
        self.ws = torch.empty(max(ws_bytes // 4, 4), dtype=torch.float32, device=dev)
        self.stream = torch.cuda.current_stream(dev)

    def step(self, hag: bool) -> int:
        h, w, ws = self.h, self.w, self.ws
        launches = 0
        cur = self.x
        for l in range(w.layers):
            (h.aggregate_fwd if hag else h.csr_fwd)(cur, w.reduce, out=self.bufs[l], workspace=ws)
            launches += h.last_launch_count
            cur = self.bufs[l]
        cur = self.gr
        for l in range(w.layers):
            o = self.bufs[w.layers + l]
            (h.aggregate_bwd if hag else h.csr_bwd)(cur, w.reduce, out=o, workspace=ws)
            launches += h.last_launch_count
            cur = o
        return launches

    @property
    def bytes_step(self):
        return 2 * self.w.layers * self.nbytes["hag_pass"]

    @property
    def plain_step(self):
        return 2 * self.w.layers * self.nbytes["plain_pass"]

    def hag_block(self):
        info, nb = self.info, self.nbytes
        return {"num_agg": info["num_agg"], "levels": info["num_levels"], "e_hat": info["e_hat"],
                "fwd_cut": self.cuts[0], "bwd_cut": self.cuts[1],
                "aggregation_reduction": info["aggregations_gnn"] / max(info["aggregations_hag"], 1),
                "read_reduction": info["e"] / max(info["e_hat"], 1),
                "byte_reduction": nb["plain_pass"] / nb["hag_pass"],
                "build_seconds": self.build_s, "bytes_per_step": self.bytes_step}

    def close(self):
        self.h.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=DEFAULT_WORKLOAD,
                    help="1-5: the named shapes (3 = 233 000 nodes, degree ~100, two layers: the headline); 6: clique-union graph")
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--capacity-frac", type=float, default=0.25)
    ap.add_argument("--min-redundancy", type=int, default=2,
                    help="stop the search below this redundancy (2 = the paper's rule; 4 = no merge that loses bytes)")
    ap.add_argument("--capacity-sweep", action="store_true",
                    help="also time capacities 0, N/8, N/4, N/2 from ONE search (hag_truncate); reported under capacity_sweep")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="measure the headline workload only")
    ap.add_argument("--schedule", type=int, default=0, choices=[0, 1, 2],
                    help="hag_set_schedule: 0 a launch per level, 1 one launch per pass, 2 the aggregation nodes in one launch "
                         "and the graph nodes in a second")
    ap.add_argument("--single-launch", action="store_const", const=1, dest="schedule", help="same as --schedule 1")
    ap.add_argument("--cuts", type=str, default="", help="forced cuts 'fwd,bwd' (hag_set_cuts); default: the library's choice")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "graphs", "columns"],
                    help="N > 1: one whole workload per rank (weak), the graphs of workload 4 split over ranks, or the "
                         "feature columns of the workload split over ranks (both strong)")
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
        run_reference(args, synth.workload(args.workload, scale=args.scale, capacity_frac=args.capacity_frac))
        return

    secondary = []
    if (not args.no_per_config and world == 1 and args.workload == DEFAULT_WORKLOAD and args.scale == 1.0
            and not args.permute_ids and not args.capacity_sweep and not args.cuts):
        secondary = [i for i in SECONDARY_WORKLOADS if i != args.workload]
    # the graphs of all workloads are drawn side by side, before CUDA is touched (the generators are single-threaded numpy)
    wanted = [args.workload] + secondary
    if len(wanted) > 1:
        from concurrent.futures import ProcessPoolExecutor
        with ProcessPoolExecutor(max_workers=len(wanted)) as pool:
            futs = {i: pool.submit(synth.workload, i, args.scale if i == args.workload else 1.0, args.capacity_frac) for i in wanted}
            workloads = {i: f.result() for i, f in futs.items()}
    else:
        workloads = {args.workload: synth.workload(args.workload, scale=args.scale, capacity_frac=args.capacity_frac)}

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

    w = workloads[args.workload]
    if args.permute_ids:
        w.graph = synth.permute_ids(w.graph, seed=w.seed + 77)
    scaling, column_slice, shard_note = "weak", None, "one whole workload per rank (independent problems, no exchange)"
    if world > 1 and args.shard == "graphs":
        size = int((w.graph.meta or {}).get("graph_size", 0))
        if not size:
            raise SystemExit("--shard graphs needs a batch of disjoint graphs (--workload 4)")
        w.graph = sharding.shard_block_diagonal(w.graph, size, rank, world)
        w.capacity = int(w.graph.n * args.capacity_frac)
        scaling, shard_note = "strong", "the graphs of the batch split over ranks, one HAG per rank, no exchange"
    elif world > 1 and args.shard == "columns":
        column_slice = sharding.shard_columns(w.d, rank, world, 4 if w.dtype == "f32" else 2)
        if column_slice[1] == 0:
            raise SystemExit("--shard columns: more ranks than 16-byte column groups")
        scaling, shard_note = "strong", "feature columns split over ranks, whole structure on every rank, no exchange"
    flush = torch.empty(L2_FLUSH_BYTES // 4, dtype=torch.float32, device=dev)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()

    def timed(r: Runner, hag: bool, steps: int, cold: bool):
        """Sum of the per-step device times (events on the launching stream); the L2 flush sits between steps."""
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        launches = 0
        barrier()
        for i in range(steps):
            if cold:
                flush.zero_()
            starts[i].record(r.stream)
            launches += r.step(hag)
            stops[i].record(r.stream)
        barrier()
        ms = sharding.max_over_ranks(sum(a.elapsed_time(b) for a, b in zip(starts, stops)), dev)
        return ms / max(steps, 1), launches

    def ratio_of(r: Runner, steps: int, reps: int = 7):
        """HAG against plain CSR as the median of interleaved repetitions (cold L2), with the spread."""
        block = max(steps // 4, 3)
        ratios = []
        for _ in range(reps):
            a, _ = timed(r, True, block, cold=True)
            b, _ = timed(r, False, block, cold=True)
            ratios.append(b / a)
        return {"median": float(np.median(ratios)), "min": float(min(ratios)), "max": float(max(ratios)),
                "repetitions": reps, "steps_per_repetition": block}

    def measure(r: Runner, steps: int, warm: bool):
        for _ in range(args.warmup):
            r.step(True)
            r.step(False)
        hag_ms, launches = timed(r, True, steps, cold=True)
        csr_ms, _ = timed(r, False, steps, cold=True)
        out = {"hag_ms": hag_ms, "csr_ms": csr_ms, "launches": launches, "ratio": ratio_of(r, steps)}
        if warm:
            out["hag_warm_ms"], _ = timed(r, True, steps, cold=False)
            out["csr_warm_ms"], _ = timed(r, False, steps, cold=False)
        if r.h.device_status() != 0:
            raise SystemExit("a bounded device-side wait gave up (HAG_ERR_TIMEOUT): the numbers of this run are void")
        return out

    peak, peak_kind = measured_peak()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()

    # ---- the headline workload --------------------------------------------------------------------------
    r = Runner(w, args, dev, local_rank, column_slice)
    g = w.graph
    m = measure(r, args.steps, warm=True)
    hag_ms, csr_ms, launches = m["hag_ms"], m["csr_ms"], m["launches"]
    total_bytes = sharding.sum_over_ranks(r.bytes_step, dev)
    total_plain = sharding.sum_over_ranks(r.plain_step, dev)

    # the dominant kernel, timed live with an event pair around every launch: the forward pass over the HAG
    r.h.profile(True)
    kinds = {0: [], 1: [], 2: [], 3: []}
    fwd_pass, bwd_pass, fwd_gather = [], [], []
    fwd_kernels = 0
    prof_steps = min(args.steps, 30)
    for _ in range(prof_steps):
        flush.zero_()
        r.h.aggregate_fwd(r.x, w.reduce, out=r.bufs[0], workspace=r.ws)
        rec = r.h.profile_read()
        for ms, kind, _, _ in rec:
            kinds[kind].append(ms)
        fwd_pass.append(sum(v[0] for v in rec))
        fwd_gather.append(rec[-1][0])           # the last launch of the pass: the gather over the graph nodes
        fwd_kernels = len(rec)
        r.h.aggregate_bwd(r.gr, w.reduce, out=r.bufs[w.layers], workspace=r.ws)
        rec = r.h.profile_read()
        for ms, kind, _, _ in rec:
            kinds[kind].append(ms)
        bwd_pass.append(sum(v[0] for v in rec))
    r.h.profile(False)
    fp_ms = float(np.mean(fwd_pass))
    fg_ms = float(np.mean(fwd_gather))
    # the dominant kernel: the whole pass when it is one launch, else its last launch
    dom_ms, dom_bytes = (fp_ms, r.nbytes["hag_pass"]) if fwd_kernels == 1 else (fg_ms, r.nbytes["fwd_gather"])
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9

    # end to end through the host-buffer entry point: pinned host inputs and outputs
    e2e = None
    if not args.no_e2e:
        xh = r.x.cpu().pin_memory()
        gh = r.gr.cpu().pin_memory()
        oh = [torch.empty_like(xh).pin_memory() for _ in range(2 * w.layers)]

        def host_step():
            cur = xh
            for l in range(w.layers):
                r.h.aggregate_host(cur, oh[l], w.reduce, backward=False, use_hag=True)
                cur = oh[l]
                if w.layers > 1:
                    torch.cuda.synchronize(dev)      # the next layer reads this host buffer
            cur = gh
            for l in range(w.layers):
                r.h.aggregate_host(cur, oh[w.layers + l], w.reduce, backward=True, use_hag=True)
                cur = oh[w.layers + l]
                if w.layers > 1:
                    torch.cuda.synchronize(dev)

        e2e_steps = max(min(args.steps, 10), 3)
        for _ in range(2):
            host_step()
        barrier()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(r.stream)
        for _ in range(e2e_steps):
            host_step()
        e1.record(r.stream)
        barrier()
        e2e_ms = sharding.max_over_ranks(e0.elapsed_time(e1) / e2e_steps, dev)
        io = 2 * w.layers * r.x.numel() * r.x.element_size()
        e2e = {"value": total_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s",
               "h2d_bytes_per_step": io, "d2h_bytes_per_step": io, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "api": "hag_aggregate_host (pinned host buffers in and out, copies inside the timed region)"}
        del xh, gh, oh

    sweep = None
    if args.capacity_sweep and rank == 0:
        # Section 5.4's capacity study: one search at N/2, every smaller capacity is a prefix of its merges
        t0 = time.perf_counter()
        big = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 2)
        search_s = time.perf_counter() - t0
        sweep = {"search_seconds_at_half_n": search_s, "points": []}
        keep_h, keep_ws, keep_nb = r.h, r.ws, r.nbytes
        for frac_name, cap in (("0", 0), ("N/8", g.n // 8), ("N/4", g.n // 4), ("N/2", g.n // 2)):
            hc = big.truncate(cap).to_device(local_rank)
            hc.set_schedule(args.schedule)
            ic, ac = hc.info(), hc.arrays()
            r.h, r.nbytes = hc, algorithmic_bytes(g.n, r.d, w.dtype, ac, ic)
            r.ws = torch.empty(max(hc.workspace_bytes(r.d), hc.csr_workspace_bytes(r.d), 16) // 4, dtype=torch.float32, device=dev)
            for _ in range(3):
                r.step(True)
            ms, _ = timed(r, True, max(args.steps // 4, 5), cold=True)
            sweep["points"].append({"capacity": frac_name, "num_agg": ic["num_agg"], "levels": ic["num_levels"],
                                    "e_hat": ic["e_hat"], "ms_per_step": ms, "gbps": r.bytes_step / (ms * 1e-3) / 1e9,
                                    "speedup_vs_capacity_0": None})
            hc.close()
        r.h, r.ws, r.nbytes = keep_h, keep_ws, keep_nb
        base_ms = sweep["points"][0]["ms_per_step"]
        for pt in sweep["points"]:
            pt["speedup_vs_capacity_0"] = base_ms / pt["ms_per_step"]

    readout = None
    meta = getattr(g, "meta", None) or {}
    if rank == 0 and "graph_size" in meta and g.n % int(meta["graph_size"]) == 0 and column_slice is None:
        readout = readout_leg(torch, hb, r, int(meta["graph_size"]), flush, min(args.steps, 30), peak)

    maxagg = max_leg(torch, r, flush, args.steps) if (rank == 0 and args.max_leg) else None

    hag_info = r.hag_block()
    x_bytes = r.x.numel() * r.x.element_size()
    r.close()
    del r
    torch.cuda.empty_cache()

    # ---- the other shapes, same protocol, fewer steps ---------------------------------------------------
    per_config = []
    for i in secondary:
        wi = workloads[i]
        ri = Runner(wi, args, dev, local_rank)
        steps_i = max(args.steps // 2, 10)
        mi = measure(ri, steps_i, warm=False)
        gb = ri.bytes_step / (mi["hag_ms"] * 1e-3) / 1e9
        per_config.append({
            "workload": workload_string(wi), "ms_per_step": mi["hag_ms"], "gbps": gb,
            "pct_of_hbm_nominal_8TBs": 100.0 * gb / NOMINAL_HBM_GBS, "pct_of_hbm_measured": 100.0 * gb / peak,
            "plain_csr_ms_per_step": mi["csr_ms"], "speedup_hag_vs_plain": mi["ratio"], "steps": steps_i,
            "launches_per_step": mi["launches"] / steps_i, "hag": ri.hag_block(),
            "dtype": "f32" if wi.dtype == "f32" else "f32 accumulate, bf16 storage"})
        if wi.name in NCU_FWD_GATHER:       # the ncu capture of this shape's largest launch: which roof it sits under
            ni = NCU_FWD_GATHER[wi.name]
            per_config[-1]["largest_launch_ncu"] = {"l2_frac": ni["lts_throughput_pct"] / 100.0, "dram_bytes": ni["dram_bytes"],
                                                    "bound": "l2", "note": ni["note"]}
        ri.close()
        del ri
        torch.cuda.empty_cache()

    # a timed arm lasts milliseconds, below nvidia-smi's sampling period: the sampler ran across all GPU arms
    clocks = sampler.stop() if rank == 0 else {}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle(w, threads=1)
        cpu["cpu_model"] = cpu_model()
        cores = os.cpu_count() or 1
        if cores > 1:
            cpu["all_cores"] = time_oracle(w, threads=cores)

    if rank == 0:
        value = total_bytes / (hag_ms * 1e-3) / 1e9
        ncu = NCU_FWD_GATHER.get(w.name) if (args.scale == 1.0 and not args.permute_ids and column_slice is None
                                            and not args.schedule and not args.cuts and world == 1) else None
        traffic = ncu["dram_bytes"] if ncu else None
        dram_frac = (traffic / (dom_ms * 1e-3) / 1e9 / peak) if traffic else None
        l2_frac = (ncu["lts_throughput_pct"] / 100.0) if ncu else None
        # the rows come from HBM only when the matrices do not fit in L2; otherwise the L2 / load path binds
        if dram_frac is not None:
            bound = "hbm" if dram_frac >= l2_frac else "l2"      # whichever of the two measured fractions is nearer its peak
        else:
            bound = "hbm" if x_bytes > (126 << 20) else "l2"
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": hag_ms, "higher_is_better": True, "scaling": scaling,
            "vs_baseline": None, "dtype": "f32" if w.dtype == "f32" else "f32 accumulate, bf16 storage", "data": "synthetic",
            "config": {
                "workload": workload_string(w),
                "l2": "flushed between timed steps (256 MiB write outside the per-step events)",
                "timing": "sum of per-step CUDA-event intervals on the launching stream, max over ranks",
                "clocks": "nvidia-smi sampled every 100 ms across all GPU arms",
                "schedule": ("a launch per level", "one launch per pass", "aggregation nodes in one launch, graph nodes in a second")[args.schedule],
                "ranks": shard_note,
            },
            "clocks": clocks,
            "e2e": e2e,
            "gpu_launches": launches,
            "pct_of_hbm_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
            "pct_of_hbm_measured": 100.0 * value / world / peak,
            "plain_csr": {"ms_per_step": csr_ms, "gbps": total_plain / (csr_ms * 1e-3) / 1e9,
                          "speedup_hag_vs_plain": csr_ms / hag_ms, "speedup_interleaved": m["ratio"]},
            "warm_l2": {"hag_ms_per_step": m["hag_warm_ms"], "plain_ms_per_step": m["csr_warm_ms"],
                        "hag_gbps": total_bytes / (m["hag_warm_ms"] * 1e-3) / 1e9},
            "hag": hag_info,
            "kernels_ms": {"level_pair_sum_total": float(np.sum(kinds[0])) / prof_steps,
                           "level_gather_total": float(np.sum(kinds[1])) / prof_steps,
                           "graph_node_gather_total": float(np.sum(kinds[2])) / prof_steps,
                           "single_launch_pass_total": float(np.sum(kinds[3])) / prof_steps,
                           "forward_pass": fp_ms, "backward_pass": float(np.mean(bwd_pass)),
                           "kernels_per_forward_pass": fwd_kernels},
            "roofline": {"bound": bound,
                         "kernel": ("fused_pass_kernel: the forward pass over the HAG in one launch" if fwd_kernels == 1
                                    else "gather_sum_persistent_kernel / gather_sum_kernel: the gather over the graph nodes of the forward "
                                         "pass over the HAG (the last and largest of its launches)"),
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_kind": f"{peak_kind} copy bandwidth",
                         "traffic": traffic, "traffic_note": (ncu or {}).get("note"),
                         "dram_frac": dram_frac, "l2_frac": l2_frac,
                         "algorithmic_bytes_per_launch": dom_bytes, "ms_per_launch": dom_ms,
                         "note": "frac counts every row read as traffic (the metric's formula); repeated reads are served by "
                                 "the L2, so dram_frac (ncu DRAM bytes / time / peak) and l2_frac (ncu lts__throughput) say "
                                 "which roof binds"},
            "cpu_baseline": cpu,
        }
        if per_config:
            line["per_config"] = per_config
        if sweep is not None:
            line["capacity_sweep"] = sweep
        if readout is not None:
            line["graph_readout"] = readout
        if maxagg is not None:
            line["max_aggregation"] = maxagg
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def readout_leg(torch, hb, r, size, flush, steps, peak):
    """Graph classification (Section 5.1): the mean-pooling layer after the GNN layers, one row per graph."""
    g, x = r.w.graph, r.x
    seg = torch.arange(0, g.n + 1, size, dtype=torch.int32, device=r.dev)
    pooled = torch.empty((g.n // size, r.d), dtype=x.dtype, device=r.dev)
    gpool = torch.empty_like(x)
    for _ in range(3):
        hb.graph_pool_fwd(seg, x, "mean", out=pooled)
        hb.graph_pool_bwd(seg, pooled, g.n, "mean", out=gpool)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    torch.cuda.synchronize(r.dev)
    for e3 in ev:
        flush.zero_()
        e3[0].record(r.stream)
        hb.graph_pool_fwd(seg, x, "mean", out=pooled)
        e3[1].record(r.stream)
        hb.graph_pool_bwd(seg, pooled, g.n, "mean", out=gpool)
        e3[2].record(r.stream)
    torch.cuda.synchronize(r.dev)
    f_ms = float(np.mean([e3[0].elapsed_time(e3[1]) for e3 in ev]))
    b_ms = float(np.mean([e3[1].elapsed_time(e3[2]) for e3 in ev]))
    rb = (x.numel() + pooled.numel()) * x.element_size()        # each pass reads one matrix and writes the other
    return {"what": f"mean-pooling read-out, {g.n // size} graphs of {size} nodes, cold L2", "fwd_ms": f_ms, "bwd_ms": b_ms,
            "fwd_gbps": rb / (f_ms * 1e-3) / 1e9, "bwd_gbps": rb / (b_ms * 1e-3) / 1e9,
            "fwd_frac_of_measured_hbm": rb / (f_ms * 1e-3) / 1e9 / peak,
            "bwd_frac_of_measured_hbm": rb / (b_ms * 1e-3) / 1e9 / peak}


def max_leg(torch, r, flush, steps):
    """The max Aggregate of Table 1 (GraphSAGE-P) over the same HAG, against the same kernels on the plain graph."""
    h, x, gr = r.h, r.x, r.gr
    mo = torch.empty_like(x)
    mg = torch.empty_like(x)
    mws = [h.max_workspace(r.d, r.dev), h.max_workspace(r.d, r.dev)]
    res = {}
    for use_hag in (True, False):
        for _ in range(3):
            h.max_fwd(x, out=mo, workspace=mws[0], use_hag=use_hag)
            h.max_bwd(x, mo, mws[0], gr, out=mg, workspace=mws[1], use_hag=use_hag)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(max(steps // 4, 5))]
        torch.cuda.synchronize(r.dev)
        for e3 in ev:
            flush.zero_()
            e3[0].record(r.stream)
            h.max_fwd(x, out=mo, workspace=mws[0], use_hag=use_hag)
            e3[1].record(r.stream)
            h.max_bwd(x, mo, mws[0], gr, out=mg, workspace=mws[1], use_hag=use_hag)
            e3[2].record(r.stream)
        torch.cuda.synchronize(r.dev)
        res[use_hag] = (float(np.mean([e3[0].elapsed_time(e3[1]) for e3 in ev])),
                        float(np.mean([e3[1].elapsed_time(e3[2]) for e3 in ev])))
    nb = r.nbytes
    return {"what": "element-wise max aggregation, fwd and bwd timed apart, cold L2; forward bytes counted like the sum's",
            "hag_fwd_ms": res[True][0], "hag_bwd_ms": res[True][1], "plain_fwd_ms": res[False][0], "plain_bwd_ms": res[False][1],
            "hag_fwd_gbps": nb["hag_pass"] / (res[True][0] * 1e-3) / 1e9,
            "plain_fwd_gbps": nb["plain_pass"] / (res[False][0] * 1e-3) / 1e9,
            "speedup_hag_vs_plain_fwd": res[False][0] / res[True][0],
            "speedup_hag_vs_plain_fwd_bwd": sum(res[False]) / sum(res[True])}


if __name__ == "__main__":
    main()
