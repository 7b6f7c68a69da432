#!/usr/bin/env python
"""Full-size pin of the oracle's search on the shapes where only its memory-light variant runs.

Writes a ``replay_ok`` record beside the stored digest of each listed case in
tests/golden/structure_hashes.json, from the ORACLE alone (nothing here touches the CUDA
package except the input generator).  For each case:

  1. the oracle's search produces the merge trace (as for the stored digest);
  2. the trace is replayed from the Redundancy definition of Algorithm 3 (oracle.c:
     o_replay_trace -- no bounds, no heap, no pair map): before every merge the recorded
     redundancy must equal the number of rows that hold both nodes; at about twenty seeded
     steps, and once more after the last merge, the redundancy of EVERY pair is recounted
     and the recorded pair must be the largest with the lowest-pair-id tie-break;
  3. on the replayed rows: Theorem 2's cover condition as a multiset (every row expands to
     exactly N(u)), both forms of the cost function of Section 4.1 agree when no row is
     empty, each merge changes |E-hat| by 2 - r_i so that f = |E| - |E-hat| + |V_A| =
     sum(r_i - 1) (proof of Theorem 4), the r_i never rise and stay >= 2, and what is left
     after the last merge is <= the last r_i (and <= 1 if the capacity was not reached);
  4. the layout built from the REPLAYED rows must give the stored SHA-256.

Run from the repository root (cfg3 and cfg5 take some minutes each):

    python tests/golden/make_replay_pins.py [--case 3:1.0 --case 5:1.0]
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

OUT = os.path.join(ROOT, "tests", "golden", "structure_hashes.json")
N_ARGMAX_CHECKS = 20


def replay_record(workload: int, scale: float, stored: dict) -> dict:
    w = synth.workload(workload, scale=scale)
    g = w.graph
    t0 = time.time()
    search = {"pairmap": O.greedy_pairmap, "lazy": O.greedy_lazy}[stored.get("oracle_search", "pairmap")]
    res = search(g.row_ptr, g.col_idx, w.capacity)
    search_s = time.time() - t0
    k = res.num_agg
    rng = np.random.default_rng(1000 * workload + 7)
    steps = sorted(set([0, k - 1] + [int(s) for s in rng.integers(0, max(k, 1), N_ARGMAX_CHECKS - 2)])) if k else []
    t0 = time.time()
    rep = O.replay_trace_full(g.row_ptr, g.col_idx, res.trace, check_argmax_at=steps + [k])
    replay_s = time.time() - t0
    rec = dict(ok=False, merges_replayed=k, argmax_checked_at=steps, search=stored.get("oracle_search", "pairmap"),
               search_seconds=round(search_s, 1), replay_seconds=round(replay_s, 1))
    if not rep["ok"]:
        rec.update(failed_step=rep["failed_step"], failure=rep["failure"], detail=rep["detail"])
        return rec
    r = res.trace[:, 2].astype(np.int64)
    same_rows = all(np.array_equal(a, b) for a, b in zip(res.rows, rep["rows"]))
    cover_bad_row = O.cover_check_rows(g.row_ptr, g.col_idx, res.trace, rep["row_len"], rep["row_store"])
    h = O.canonical_hag(g.row_ptr, O.SearchResult(g.n, res.trace, rep["rows"], rep["final_max_redundancy"]))
    c = O.counters(g.row_ptr, h)
    arrays = dict(trace=res.trace.astype(np.int32), level_ptr=h.level_ptr, agg_in=h.agg_in, res_ptr=h.res_ptr,
                  res_idx=h.res_idx, t_ptr=h.t_ptr, t_idx=h.t_idx, in_degree=h.in_degree)
    dig = hashlib.sha256()
    for name in ("trace", "level_ptr", "agg_in", "res_ptr", "res_idx", "t_ptr", "t_idx", "in_degree"):
        dig.update(np.ascontiguousarray(arrays[name]).tobytes())
    left = rep["final_max_redundancy"]
    checks = dict(
        rows_equal_the_search_rows=bool(same_rows),
        cover_multiset_equals_neighbourhood=bool(cover_bad_row == -1),
        cost_forms_agree=bool((not c["closed_form_applies"]) or c["aggregations_hag"] == c["aggregations_hag_closed_form"]),
        e_hat_follows_2_minus_r=bool(c["e_hat"] == c["e"] + int((2 - r).sum())),
        saved_equals_sum_r_minus_1=bool(c["saved_f"] == int((r - 1).sum())),
        redundancies_never_rise=bool(k == 0 or (np.diff(r) <= 0).all()),
        redundancies_at_least_2=bool(k == 0 or r.min() >= 2),
        left_over_not_above_last=bool(k == 0 or left <= int(r[-1])),
        left_over_at_most_1_if_capacity_not_reached=bool(k == w.capacity or left <= 1),
        digest_of_replayed_layout_equals_stored=bool(dig.hexdigest() == stored["sha256"]),
    )
    rec.update(ok=all(checks.values()), checks=checks, full_recounts=rep["full_recounts"],
               pair_count_updates=rep["pair_count_updates"], first_redundancy=int(r[0]) if k else 0,
               last_redundancy=int(r[-1]) if k else 0, redundancy_left_after_last_merge=left)
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", action="append", default=[], help="workload:scale of a stored case (default 3:1 and 5:1)")
    args = ap.parse_args()
    stored = json.load(open(OUT))
    cases = [tuple(float(v) if i else int(v) for i, v in enumerate(a.split(":"))) for a in args.case] or [(3, 1.0), (5, 1.0)]
    for workload, scale in cases:
        key = f"cfg{workload}@{scale:g}"
        rec = replay_record(workload, scale, stored["cases"][key])
        print(key, json.dumps(rec), flush=True)
        stored = json.load(open(OUT))          # another run may have written meanwhile
        stored["cases"][key]["replay_ok"] = rec
        with open(OUT, "w") as f:
            json.dump(stored, f, indent=1, sort_keys=True)


if __name__ == "__main__":
    main()
