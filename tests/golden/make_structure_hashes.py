#!/usr/bin/env python
"""Writes tests/golden/structure_hashes.json from the ORACLE alone.

For each listed workload the oracle's Algorithm 3 (pair-count heap, or with
--search lazy its memory-light variant) and its canonical layout are run, and a SHA-256 over the structure arrays is stored.
tests/test_build_host.py then requires the library's hag_build to reproduce the
digest bit for bit.  Nothing here touches the CUDA package except the input
generator.  Run from the repository root:

    python tests/golden/make_structure_hashes.py [--add 4:1.0]
"""
import argparse
import hashlib
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import oracle as O  # noqa: E402
from paper_1906_03707_b200 import synth  # noqa: E402

ARRAY_ORDER = ["trace", "level_ptr", "agg_in", "res_ptr", "res_idx", "t_ptr", "t_idx", "in_degree"]
DEFAULT_CASES = [(1, 1.0), (2, 0.2), (2, 1.0), (4, 0.05), (5, 0.01)]
OUT = os.path.join(ROOT, "tests", "golden", "structure_hashes.json")


def digest(workload: int, scale: float, search: str = "pairmap") -> dict:
    w = synth.workload(workload, scale=scale)
    g = w.graph
    t0 = time.time()
    fn = {"pairmap": O.greedy_pairmap, "lazy": O.greedy_lazy}[search]
    res = fn(g.row_ptr, g.col_idx, w.capacity)
    h = O.canonical_hag(g.row_ptr, res)
    arrays = dict(trace=res.trace.astype(np.int32), level_ptr=h.level_ptr, agg_in=h.agg_in, res_ptr=h.res_ptr,
                  res_idx=h.res_idx, t_ptr=h.t_ptr, t_idx=h.t_idx, in_degree=h.in_degree)
    dig = hashlib.sha256()
    for k in ARRAY_ORDER:
        dig.update(np.ascontiguousarray(arrays[k]).tobytes())
    c = O.counters(g.row_ptr, h)
    return dict(workload=workload, scale=scale, capacity=w.capacity, n=g.n, e=g.e, num_agg=h.num_agg,
                num_levels=h.num_levels, e_hat=c["e_hat"], sha256=dig.hexdigest(), oracle_search=search,
                oracle_seconds=round(time.time() - t0, 1),
                host_seconds_hint=round(g.e / 5.0e5, 1))   # rough library build time; the CPU suite skips slow cases


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--add", action="append", default=[], help="workload:scale to add to the stored file")
    ap.add_argument("--search", default="pairmap", choices=["pairmap", "lazy"],
                    help="oracle search: the pair-count heap, or the memory-light one for shapes whose pair map does not fit")
    args = ap.parse_args()
    stored = {"array_order": ARRAY_ORDER, "cases": {}}
    if os.path.exists(OUT):
        stored = json.load(open(OUT))
    cases = [tuple(float(v) if i else int(v) for i, v in enumerate(a.split(":"))) for a in args.add] or DEFAULT_CASES
    for workload, scale in cases:
        key = f"cfg{workload}@{scale:g}"
        stored["cases"][key] = digest(workload, scale, args.search)
        print(key, stored["cases"][key], flush=True)
        stored["array_order"] = ARRAY_ORDER
        with open(OUT, "w") as f:
            json.dump(stored, f, indent=1, sort_keys=True)


if __name__ == "__main__":
    main()
