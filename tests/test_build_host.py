"""Host side of the library (no GPU): hag_build against the oracle, bit for bit;
the C ABI's symbols; argument and graph validation."""
import ctypes
import json
import os
import re

import numpy as np
import pytest

import paper_1906_03707_b200 as hb
from oracle import oracle as O
from paper_1906_03707_b200 import synth
from paper_1906_03707_b200.build import build as build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="session", autouse=True)
def _library():
    build_library()
    hb.load_library()


def _same_structure(g, capacity, search=O.greedy_pairmap):
    h = hb.Hag.build(g.row_ptr, g.col_idx, capacity)
    arr = h.arrays()
    res = search(g.row_ptr, g.col_idx, capacity)
    ref = O.canonical_hag(g.row_ptr, res)
    assert arr["trace"].tolist() == res.trace.tolist()
    assert arr["num_agg"] == ref.num_agg and arr["num_levels"] == ref.num_levels
    for key in ("level_ptr", "agg_in", "res_ptr", "res_idx", "t_ptr", "t_idx", "in_degree"):
        got, want = arr[key], getattr(ref, key)
        assert got.dtype == want.dtype and np.array_equal(got, want), key
    t_ptr, t_idx = O.transposed_csr(g.row_ptr, g.col_idx)
    assert np.array_equal(arr["csr_t_ptr"], t_ptr) and np.array_equal(arr["csr_t_idx"], t_idx)
    # the cuts are the library's own choice (a launch heuristic, nothing the paper fixes): any value in
    # 0..L is valid; the lists must be the oracle's for THAT choice
    assert 0 <= arr["fwd_cut"] <= ref.num_levels and 0 <= arr["bwd_cut"] <= ref.num_levels
    tails = O.expanded_tails(ref, int(arr["fwd_cut"]), int(arr["bwd_cut"]))
    for key, want in tails.items():
        assert np.array_equal(arr[key], want), key
    info = h.info()
    c = O.counters(g.row_ptr, ref)
    assert info["n"] == g.n and info["e"] == c["e"] and info["e_hat"] == c["e_hat"]
    assert info["num_agg"] == c["num_agg"] and info["num_levels"] == c["num_levels"]
    assert info["aggregations_gnn"] == c["aggregations_gnn"]
    assert info["aggregations_hag"] == c["aggregations_hag"]
    assert info["aggregations_hag_closed"] == c["aggregations_hag_closed_form"]
    assert info["saved"] == c["saved_f"]
    assert info["device"] == -1
    h.close()
    return info


def test_header_symbols_are_exported():
    text = open(os.path.join(ROOT, "include", "hag.h")).read()
    declared = set(re.findall(r"\b((?:hag|csr)_[a-z_]+)\s*\(", text))
    assert declared == set(hb.EXPORTED_SYMBOLS)
    lib = ctypes.CDLL(hb.LIB_PATH)
    for name in declared:
        assert getattr(lib, name) is not None


@pytest.mark.parametrize("name", ["k4_no_self_loops.json", "k4_self_loops.json", "renumbering_13.json"])
def test_worked_examples(golden_dir, name):
    gold = json.load(open(os.path.join(golden_dir, name)))
    g = synth.csr_from_rows(gold["rows"])
    h = hb.Hag.build(g.row_ptr, g.col_idx, gold["capacity"])
    arr = h.arrays()
    assert arr["trace"].tolist() == gold["trace"]
    for key in ("level_ptr", "agg_in", "res_ptr", "res_idx", "t_ptr", "t_idx"):
        if key in gold:
            assert arr[key].tolist() == gold[key], key


@pytest.mark.parametrize("seed", range(60))
def test_every_merge_matches_brute_force(seed):
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.integers(6, 36))
    g = synth.random_digraph(500 + seed, n, float(rng.uniform(0.15, 0.6)), bool(seed % 2), bool((seed // 2) % 2))
    for cap in (n // 4, 3 * n):
        _same_structure(g, cap, search=O.greedy_bruteforce)


@pytest.mark.parametrize("maker,cap_frac", [
    (lambda: synth.workload(1).graph, 0.25),
    (lambda: synth.config2_graph(seed=11, n=3000, n_comm=30), 0.25),
    (lambda: synth.config2_graph(seed=11, n=3000, n_comm=30), 2.0),
    (lambda: synth.config3_graph(seed=12, n=1800, n_comm=3, d_lo=10, d_hi=300), 0.25),
    (lambda: synth.config4_graph(seed=13, n_graphs=20, graph_size=60), 0.25),
    (lambda: synth.config5_graph(seed=14, n=4000, n_comm=12, s_lo=60, s_hi=900, d_lo=8, d_hi=150), 0.5),
    (lambda: synth.clique_union_graph(seed=15, n=1500, n_groups=400, g_lo=3, g_hi=40), 0.25),
    (lambda: synth.workload(1).graph, 0.0),
])
def test_structure_is_bit_exact_on_workload_shapes(maker, cap_frac):
    g = maker()
    info = _same_structure(g, int(g.n * cap_frac))
    if cap_frac == 0.0:
        assert info["num_agg"] == 0 and info["e_hat"] == info["e"]


@pytest.mark.parametrize("maker", [
    lambda: synth.clique_union_graph(seed=15, n=1500, n_groups=400, g_lo=3, g_hi=40),
    lambda: synth.config2_graph(seed=11, n=3000, n_comm=30),
])
def test_every_forced_cut_gives_the_oracles_lists_and_algorithm_2s_values(maker):
    """hag_set_cuts: for every cut 0..L the library's expansion lists equal the oracle's for that
    cut, and evaluating the deep levels from them gives Algorithm 2's level-by-level values."""
    g = maker()
    res = O.greedy_pairmap(g.row_ptr, g.col_idx, g.n // 4)
    ref = O.canonical_hag(g.row_ptr, res)
    L = ref.num_levels
    assert L >= 3
    x = synth.features(5, g.n, 4, "int").astype(np.float64)
    ahat = np.zeros((g.n + ref.num_agg, 4))
    ahat[:g.n] = x
    for j in range(ref.num_agg):                                   # Algorithm 2 lines 5-6, node by node
        ahat[g.n + j] = ahat[ref.agg_in[2 * j]] + ahat[ref.agg_in[2 * j + 1]]
    h = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 4)
    own = (int(h.arrays()["fwd_cut"]), int(h.arrays()["bwd_cut"]))
    for cut in range(L + 1):
        h.set_cuts(cut, L - cut)
        arr = h.arrays()
        assert (arr["fwd_cut"], arr["bwd_cut"]) == (cut, L - cut)
        want = O.expanded_tails(ref, cut, L - cut)
        for key, v in want.items():
            assert np.array_equal(arr[key], v), (cut, key)
        lib_lists = dict(ftail_ptr=arr["ftail_ptr"], ftail_idx=arr["ftail_idx"])
        assert np.array_equal(O.expanded_forward(ref, x, cut, lib_lists), ahat), cut
    h.set_cuts(-1, -1)
    assert (int(h.arrays()["fwd_cut"]), int(h.arrays()["bwd_cut"])) == own
    lib = hb.load_library()
    assert lib.hag_set_cuts(h._h, L + 1, 0) == 2 and lib.hag_set_cuts(h._h, 0, -2) == 2
    assert lib.hag_set_cuts(None, 0, 0) == 1


def test_full_size_search_replays_are_stored(golden_dir):
    """The two largest shapes are reached only by the oracle's memory-light search.  Their stored digests are
    backed by a from-the-definition replay of the whole trace (tests/golden/make_replay_pins.py): every
    recorded redundancy recounted, the arg-max recounted over all pairs at about twenty seeded merges
    and after the last one, the cover condition, both cost forms, the gain per merge, non-increasing
    redundancies, and the layout of the replayed rows reproducing the digest."""
    stored = json.load(open(os.path.join(golden_dir, "structure_hashes.json")))
    for key in ("cfg3@1", "cfg5@1"):
        rec = stored["cases"][key].get("replay_ok")
        assert rec is not None, f"{key}: run tests/golden/make_replay_pins.py"
        assert rec["ok"] is True and all(rec["checks"].values()), key
        assert rec["merges_replayed"] == stored["cases"][key]["num_agg"]
        assert len(rec["argmax_checked_at"]) >= 15 and rec["full_recounts"] == len(rec["argmax_checked_at"]) + 1
        assert rec["redundancy_left_after_last_merge"] <= rec["last_redundancy"] <= rec["first_redundancy"]


def test_stored_structure_hashes(golden_dir):
    """Digests written by tests/golden/make_structure_hashes.py from the oracle alone."""
    import hashlib
    path = os.path.join(golden_dir, "structure_hashes.json")
    if not os.path.exists(path):
        pytest.skip("no stored digests")
    stored = json.load(open(path))
    checked = 0
    for key, rec in stored["cases"].items():
        if rec["host_seconds_hint"] > 30:
            continue
        w = synth.workload(rec["workload"], scale=rec["scale"])
        h = hb.Hag.build(w.graph.row_ptr, w.graph.col_idx, rec["capacity"])
        arr = h.arrays()
        dig = hashlib.sha256()
        for k in stored["array_order"]:
            dig.update(np.ascontiguousarray(arr[k]).tobytes())
        assert dig.hexdigest() == rec["sha256"], key
        checked += 1
    assert checked > 0


def test_empty_and_degenerate_graphs():
    # no nodes
    h = hb.Hag.build(np.zeros(1, np.int64), np.zeros(0, np.int32), 4)
    assert h.info()["n"] == 0 and h.info()["num_agg"] == 0
    # nodes without edges
    h = hb.Hag.build(np.zeros(6, np.int64), np.zeros(0, np.int32), 4)
    arr = h.arrays()
    assert arr["num_agg"] == 0 and arr["res_ptr"].tolist() == [0] * 6 and h.workspace_bytes(64) == 0
    # capacity reached exactly, then workspace size
    g = synth.csr_from_rows([list(range(8))] * 8)
    h = hb.Hag.build(g.row_ptr, g.col_idx, 2)
    assert h.info()["num_agg"] == 2 and h.workspace_bytes(64) == 2 * 64 * 4 and h.workspace_bytes(0) == 0


def test_argument_and_graph_validation():
    lib = hb.load_library()
    rp = np.asarray([0, 2, 3], dtype=np.int64)
    handle = ctypes.c_void_p()

    def build(n, rp_, ci_, cap):
        return lib.hag_build(n, rp_.ctypes.data if rp_ is not None else None,
                             ci_.ctypes.data if ci_ is not None else None, cap, ctypes.byref(handle))

    ok = np.asarray([0, 1, 0], dtype=np.int32)
    assert build(2, rp, ok, 1) == 0
    lib.hag_destroy(handle)
    assert build(2, None, ok, 1) == 1                                           # NULL
    assert lib.hag_build(2, rp.ctypes.data, ok.ctypes.data, 1, None) == 1       # NULL out
    assert build(-1, rp, ok, 1) == 2 and build(2, rp, ok, -1) == 2              # ARG
    assert build(2, rp, ok, 2 ** 31 - 2) == 2                                   # n + capacity overflow
    assert build(2, rp, np.asarray([1, 0, 0], dtype=np.int32), 1) == 3          # unsorted row
    assert build(2, rp, np.asarray([1, 1, 0], dtype=np.int32), 1) == 3          # duplicate
    assert build(2, rp, np.asarray([0, 2, 0], dtype=np.int32), 1) == 3          # out of range
    assert build(2, rp, np.asarray([0, -1, 0], dtype=np.int32), 1) == 3
    assert build(2, np.asarray([0, 3, 2], dtype=np.int64), ok, 1) == 3          # decreasing row_ptr
    assert build(2, np.asarray([1, 2, 3], dtype=np.int64), ok, 1) == 3          # row_ptr[0] != 0
    assert handle.value is None
    # calls on a host-only handle fail with a status, not a crash
    h = hb.Hag.build(rp, ok, 1)
    dummy = ctypes.c_void_p(4096)
    assert lib.hag_aggregate_fwd(h._h, 0, 0, 64, dummy, ctypes.c_void_p(8192), None, None) == 11   # not on device
    assert lib.hag_aggregate_fwd(h._h, 0, 0, 6, dummy, ctypes.c_void_p(8192), None, None) == 8     # row bytes % 16
    assert lib.hag_aggregate_fwd(h._h, 0, 0, 64, ctypes.c_void_p(4100), ctypes.c_void_p(8192), None, None) == 8
    assert lib.hag_aggregate_fwd(h._h, 0, 5, 64, dummy, ctypes.c_void_p(8192), None, None) == 7    # dtype
    assert lib.hag_aggregate_fwd(h._h, 0, 0, 0, dummy, ctypes.c_void_p(8192), None, None) == 2     # D
    assert lib.hag_aggregate_fwd(h._h, 0, 0, 64, None, ctypes.c_void_p(8192), None, None) == 1     # NULL
    assert lib.hag_aggregate_fwd(None, 0, 0, 64, dummy, ctypes.c_void_p(8192), None, None) == 1
    assert lib.hag_get_info(None, None) == 1 and lib.hag_export(h._h, None) == 1
    assert lib.hag_to_device(h._h, -1) == 2
    assert lib.hag_workspace_bytes(None, 4) == 0 and lib.hag_last_launch_count(None) == 0
    assert hb.status_str(3).startswith("malformed") and hb.status_str(99) == "unknown status"
    assert lib.hag_destroy(None) == 0


def test_truncate_equals_a_fresh_build_with_the_smaller_capacity():
    import hashlib

    def digest(h):
        arr = h.arrays()
        dig = hashlib.sha256()
        for k in sorted(arr):
            dig.update(np.ascontiguousarray(arr[k]).tobytes() if hasattr(arr[k], "tobytes") else str(arr[k]).encode())
        info = {k: v for k, v in h.info().items() if k != "build_seconds"}
        return dig.hexdigest(), info

    g = synth.config5_graph(seed=14, n=4000, n_comm=12, s_lo=60, s_hi=900, d_lo=8, d_hi=150)
    full = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 2)
    assert full.info()["num_agg"] == g.n // 2
    for cap in (0, 1, g.n // 8, g.n // 4, g.n // 2):
        assert digest(full.truncate(cap)) == digest(hb.Hag.build(g.row_ptr, g.col_idx, cap)), cap
    lib = hb.load_library()
    out = ctypes.c_void_p()
    assert lib.hag_truncate(full._h, g.n, ctypes.byref(out)) == 2      # the search was cut off by its capacity
    assert lib.hag_truncate(full._h, -1, ctypes.byref(out)) == 2
    assert lib.hag_truncate(None, 1, ctypes.byref(out)) == 1 and lib.hag_truncate(full._h, 1, None) == 1
    # a search that ended by itself knows the answer for any larger capacity
    ring = synth.csr_from_rows([[1, 3], [0, 2], [1, 3], [0, 2]])
    done = hb.Hag.build(ring.row_ptr, ring.col_idx, 100)
    assert done.info()["num_agg"] == 2
    assert digest(done.truncate(50))[0] == digest(hb.Hag.build(ring.row_ptr, ring.col_idx, 50))[0]


def test_build_does_not_depend_on_the_thread_count():
    g = synth.config2_graph(seed=17, n=6000, n_comm=40)
    prev = hb.build_threads(1)
    try:
        one = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 4).arrays()
        for threads in (2, 5, 0):
            hb.build_threads(threads)
            many = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 4).arrays()
            for k, v in one.items():
                assert np.array_equal(np.asarray(v), np.asarray(many[k])), (threads, k)
        assert hb.build_threads(-1) == 0
    finally:
        hb.build_threads(prev)


def test_min_redundancy_stops_the_search_earlier():
    g = synth.config2_graph(seed=19, n=2500, n_comm=25)
    for min_r in (2, 4, 9):
        h = hb.Hag.build(g.row_ptr, g.col_idx, 10 * g.n, min_redundancy=min_r)
        ref = O.greedy_pairmap(g.row_ptr, g.col_idx, 10 * g.n, min_redundancy=min_r)
        arr = h.arrays()
        assert arr["trace"].tolist() == ref.trace.tolist()
        assert (arr["trace"][:, 2] >= min_r).all() and ref.final_max_redundancy < min_r
        layout = O.canonical_hag(g.row_ptr, ref)
        for key in ("level_ptr", "agg_in", "res_ptr", "res_idx", "t_ptr", "t_idx"):
            assert np.array_equal(arr[key], getattr(layout, key)), key
    small = synth.random_digraph(77, 24, 0.4, True, True)
    for min_r in (2, 3, 5):
        a = O.greedy_bruteforce(small.row_ptr, small.col_idx, 100, min_redundancy=min_r)
        b = hb.Hag.build(small.row_ptr, small.col_idx, 100, min_redundancy=min_r).arrays()
        assert a.trace.tolist() == b["trace"].tolist()
    # with the default the extended entry point is hag_build
    assert hb.Hag.build(g.row_ptr, g.col_idx, 100).arrays()["trace"].tolist() == \
        hb.Hag.build(g.row_ptr, g.col_idx, 100, min_redundancy=2).arrays()["trace"].tolist()
    lib = hb.load_library()
    out = ctypes.c_void_p()
    assert lib.hag_build_ex(g.n, g.row_ptr.ctypes.data, g.col_idx.ctypes.data, 10, 1, ctypes.byref(out)) == 2


def test_binding_rejects_wrong_tensors_before_any_launch():
    """The C ABI trusts pointers and sizes; the binding must turn every mismatch into a Python error."""
    torch = pytest.importorskip("torch")
    g = synth.workload(1).graph
    h = hb.Hag.build(g.row_ptr, g.col_idx, 100)
    good = torch.zeros((g.n, 16))
    for call in (lambda t: h.aggregate_fwd(t), lambda t: h.aggregate_bwd(t), lambda t: h.csr_fwd(t), lambda t: h.csr_bwd(t),
                 lambda t: h.max_fwd(t), lambda t: h.aggregate_fwd_static(t, torch.zeros_like(t)),
                 lambda t: h.aggregate_host(t, torch.zeros_like(t))):
        with pytest.raises(ValueError, match="rows"):
            call(torch.zeros((g.n - 1, 16)))                      # too few rows: would be an out-of-range read
        with pytest.raises(ValueError):
            call(torch.zeros(g.n * 16))                           # not 2-D
        with pytest.raises(ValueError):
            call(torch.zeros((g.n, 32))[:, ::2])                  # not contiguous
        with pytest.raises(TypeError):
            call(torch.zeros((g.n, 16), dtype=torch.float64))
        with pytest.raises(hb.HagError) as info:                  # right shape, but the handle is host-only
            call(good)
        assert info.value.status == hb.HAG_ERR_NOT_ON_DEVICE
    with pytest.raises(ValueError):
        h.aggregate_host(good, torch.zeros((g.n, 8)))             # out does not match
    with pytest.raises(ValueError):
        h.max_bwd(torch.zeros((g.n - 1, 16)), good, None, good)


def _emulate_pass(p, n, k, src, d):
    """Walks the row list of one pass in list order on the CPU (fp64), the way the single-launch kernel's warps
    are handed the rows, and checks what the kernel relies on: groups of four rows lie in one phase; the rows of
    other phases that a row reads (aggregation nodes, chunk rows: ids >= n) were written by phases <= the phase it
    waits for (the kernel itself reports a grab only after the phase before it is complete, so "phase q complete"
    implies all earlier ones); only the last phase writes graph-node rows; every row is written exactly once.
    Returns (graph-node rows, aggregation-node rows, writes per row)."""
    rows, ids, c = p["rows"], p["ids"], p["n_chunk_rows"]
    assert rows.shape[0] % 4 == 0 and int(p["phase_size"].sum()) == rows.shape[0]
    word = rows[:, 3].astype(np.int64) & 0xffffffff
    req, phase, n_sec = (word & 255) - 1, (word >> 8) & 255, word >> 16
    assert (np.diff(phase) >= 0).all() and (phase.reshape(-1, 4) == phase[::4, None]).all()
    assert np.array_equal(np.bincount(phase, minlength=p["phase_size"].shape[0]), p["phase_size"])
    last = int(phase.max())
    val = np.zeros((n + k + c, d))
    val[:n] = src
    out = np.zeros((n, d))
    written_in = np.full(n + k + c, -1)             # phase that wrote an aggregation-node or chunk row
    writes = np.zeros(n + k + c, dtype=np.int64)
    for i in range(rows.shape[0]):
        b, e, row = (int(v) for v in rows[i, :3])
        if row < 0:
            continue
        acc = np.zeros(d)
        # the entries read before the wait are rows of the layer input, the last n_sec are rows this pass writes
        assert (ids[b:e - n_sec[i]] < n).all() and (ids[e - n_sec[i]:e] >= n).all() and (n_sec[i] > 0) == (req[i] >= 0), i
        for s_ in ids[b:e]:
            if s_ >= n:
                assert 0 <= written_in[s_] <= req[i] < phase[i], (i, s_, written_in[s_], req[i])
            acc += val[s_]
        writes[row] += 1
        if row >= n:
            val[row] = acc
            written_in[row] = phase[i]
            assert phase[i] < last
        else:
            out[row] = acc
            assert phase[i] == last
    return out, val[n:n + k], writes


@pytest.mark.parametrize("maker,cap_frac", [
    (lambda: synth.clique_union_graph(seed=15, n=1500, n_groups=400, g_lo=3, g_hi=40), 0.25),
    (lambda: synth.config2_graph(seed=11, n=3000, n_comm=30), 0.25),
    (lambda: synth.config4_graph(seed=13, n_graphs=20, graph_size=60), 0.25),
    (lambda: synth.workload(1).graph, 0.0),
])
def test_single_launch_item_lists_evaluate_algorithm_2_for_every_cut(maker, cap_frac):
    g = maker()
    cap = int(g.n * cap_frac)
    h = hb.Hag.build(g.row_ptr, g.col_idx, cap)
    arr = h.arrays()
    n, k, L = g.n, arr["num_agg"], arr["num_levels"]
    x = synth.features(5, n, 3, "int").astype(np.float64)
    gr = synth.features(6, n, 3, "int").astype(np.float64)
    want_f, _ = O.direct_forward(g.row_ptr, g.col_idx, x, "sum")
    want_b, _ = O.direct_backward(g.row_ptr, g.col_idx, gr, "sum")
    ref = O.canonical_hag(g.row_ptr, O.greedy_pairmap(g.row_ptr, g.col_idx, cap))
    ahat = np.zeros((n + k, 3))
    ahat[:n] = x
    for j in range(k):
        ahat[n + j] = ahat[ref.agg_in[2 * j]] + ahat[ref.agg_in[2 * j + 1]]
    cuts = sorted({(-1, -1), (0, 0), (L, L), (L // 2, (L + 1) // 2), (1 if L else 0, L)})
    for fc, bc in cuts:
        h.set_cuts(fc, bc)
        arr = h.arrays()
        out, agg, writes = _emulate_pass(h.pass_rows(0), n, k, x, 3)
        assert (writes == 1).all()
        assert np.array_equal(out, want_f) and np.array_equal(agg, ahat[n:])
        gx, _, writes = _emulate_pass(h.pass_rows(1), n, k, gr, 3)
        assert (writes == 1).all() and np.array_equal(gx, want_b)
        assert h.workspace_bytes(4) >= 16 * (k + max(h.pass_rows(0)["n_chunk_rows"], h.pass_rows(1)["n_chunk_rows"]))
    out, _, writes = _emulate_pass(h.pass_rows(2), n, 0, x, 3)
    assert np.array_equal(out, want_f) and (writes == 1).all()
    gx, _, writes = _emulate_pass(h.pass_rows(3), n, 0, gr, 3)
    assert np.array_equal(gx, want_b) and (writes == 1).all()
    assert h.csr_workspace_bytes(4) >= 16 * max(h.pass_rows(2)["n_chunk_rows"], h.pass_rows(3)["n_chunk_rows"])


def test_injected_host_allocation_failures_return_a_status_and_leave_nothing_behind():
    lib = hb.load_library()
    g = synth.config2_graph(seed=19, n=2500, n_comm=25)
    out = ctypes.c_void_p()
    try:
        for countdown in (0, 1):          # the search, then the layout
            assert lib.hag_test_fail_allocation(0, countdown) == 0
            st = lib.hag_build(g.n, g.row_ptr.ctypes.data, g.col_idx.ctypes.data, g.n // 4, ctypes.byref(out))
            assert st == hb.HAG_ERR_OOM_HOST and out.value is None
            assert hb.status_str(st) == "out of host memory"
        # the hook fires once: the next build succeeds
        assert lib.hag_build(g.n, g.row_ptr.ctypes.data, g.col_idx.ctypes.data, g.n // 4, ctypes.byref(out)) == 0
        lib.hag_destroy(out)
        assert lib.hag_test_fail_allocation(2, 0) == 2
    finally:
        lib.hag_test_fail_allocation(0, -1)


def test_import_of_a_recorded_trace_reproduces_the_build_and_rejects_what_does_not_replay():
    import hashlib

    def digest(h):
        arr = h.arrays()
        dig = hashlib.sha256()
        for k in sorted(arr):
            dig.update(np.ascontiguousarray(arr[k]).tobytes() if hasattr(arr[k], "tobytes") else str(arr[k]).encode())
        info = {k: v for k, v in h.info().items() if k not in ("build_seconds", "capacity")}
        return dig.hexdigest(), info

    g = synth.config2_graph(seed=17, n=6000, n_comm=40)
    built = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 4)
    trace = built.arrays()["trace"]
    assert digest(hb.Hag.from_trace(g.row_ptr, g.col_idx, trace)) == digest(built)
    # a prefix of the trace is the HAG of the smaller capacity; no trace is the GNN-graph itself
    assert digest(hb.Hag.from_trace(g.row_ptr, g.col_idx, trace[:100])) == digest(hb.Hag.build(g.row_ptr, g.col_idx, 100))
    assert hb.Hag.from_trace(g.row_ptr, g.col_idx, trace[:0]).info()["num_agg"] == 0
    lib = hb.load_library()
    out = ctypes.c_void_p()

    def imp(tr, rp=g.row_ptr, ci=g.col_idx):
        tr = np.ascontiguousarray(tr, dtype=np.int32)
        return lib.hag_import(g.n, rp.ctypes.data, ci.ctypes.data, tr.shape[0], tr.ctypes.data, ctypes.byref(out))

    wrong = trace.copy()
    wrong[5, 2] += 1                                   # a redundancy the rows do not have
    assert imp(wrong) == 2 and out.value is None
    wrong = trace.copy()
    wrong[7, :2] = wrong[7, 1], wrong[7, 0]            # pair out of order
    assert imp(wrong) == 2
    wrong = trace.copy()
    wrong[3, 1] = g.n + 50                             # a node that does not exist yet
    assert imp(wrong) == 2
    other = synth.config2_graph(seed=18, n=6000, n_comm=40)
    assert imp(trace, other.row_ptr, other.col_idx) == 2      # the trace of another graph does not replay
    assert lib.hag_import(g.n, g.row_ptr.ctypes.data, g.col_idx.ctypes.data, 3, None, ctypes.byref(out)) == 1
    assert lib.hag_import(g.n, g.row_ptr.ctypes.data, g.col_idx.ctypes.data, -1, None, ctypes.byref(out)) == 2


def test_row_order_is_a_windowed_sort_by_length_that_keeps_every_launch_range():
    """hag_export_row_order: a permutation per list, sorted by length inside windows of 2048 rows that never cross
    from the graph nodes into a level or from a level into the next; absent where neighbouring rows already match."""
    w = synth.workload(6, scale=0.08)
    g = w.graph
    h = hb.Hag.build(g.row_ptr, g.col_idx, w.capacity)
    a = h.arrays()
    n, k = g.n, int(a["num_agg"])
    assert int(a["num_levels"]) >= 3
    level_ptr = np.asarray(a["level_ptr"], dtype=np.int64)
    t_bounds = np.concatenate([[0, n], n + level_ptr[1:]])
    csr_t_ptr = np.zeros(n + 1, np.int64)
    np.add.at(csr_t_ptr, g.col_idx.astype(np.int64) + 1, 1)
    csr_t_ptr = np.cumsum(csr_t_ptr)
    lists = {0: (a["res_ptr"], 0, [0, n]), 1: (a["t_ptr"], 0, t_bounds), 2: (g.row_ptr, 0, [0, n]), 3: (csr_t_ptr, 0, [0, n])}
    for cut_f, cut_b in ((1, 2), (0, 0)):
        h.set_cuts(cut_f, cut_b)
        p = h.pass_rows(0)      # (the expansion lists themselves are checked elsewhere; here their row ranges)
        for which, first_expected in ((4, n + int(level_ptr[cut_f])), (5, n + int(level_ptr[cut_b]))):
            first, order = h.row_order(which)
            assert first == first_expected
            if order.size:
                assert np.array_equal(np.sort(order), first + np.arange(order.size))
    seen_sorted = 0
    for which, (ptr, first_expected, bounds) in lists.items():
        first, order = h.row_order(which)
        assert first == first_expected
        lens = np.diff(np.asarray(ptr, dtype=np.int64))
        if order.size == 0:
            # only where pairs of neighbouring rows lose less than 8 % of the rounds of four loads
            r = (lens + 3) // 4
            if r.size % 2:
                r = np.concatenate([r, [0]])
            assert 2 * r.reshape(-1, 2).max(1).sum() < 1.08 * max(r.sum(), 1)
            continue
        seen_sorted += 1
        assert order.size == lens.size
        assert np.array_equal(np.sort(order), np.arange(order.size))          # a permutation
        for b0, b1 in zip(bounds[:-1], bounds[1:]):
            for w0 in range(int(b0), int(b1), 2048):
                w1 = min(w0 + 2048, int(b1))
                win = order[w0:w1]
                assert win.min() >= w0 and win.max() < w1                      # the window maps onto itself
                assert np.all(np.diff(lens[win]) <= 0)                         # longest first
                same = np.diff(lens[win]) == 0
                assert np.all(np.diff(win)[same] > 0)                          # equal lengths keep their order
    assert seen_sorted >= 2
    lib = hb.load_library()
    assert lib.hag_export_row_order(h._h, 6, ctypes.byref(ctypes.c_int32()), ctypes.byref(ctypes.c_int64()), ctypes.byref(ctypes.c_void_p())) == 2


def test_range_predicates_of_the_device_side_check_on_the_host():
    """hag_device_validate's kernels apply two predicates; here they run on the host (the GPU test only ever validates
    good structures: no kernel is handed a bad index to see the check fire)."""
    lib = hb.load_library()
    pred = lib.hag_test_range_predicates

    def id_ok(i, lo, hi):
        return bool(pred(i, lo, hi, 0, 1, 0, 0, 0, 0) & 1)

    def ptr_ok(i, rows, prev, cur, first, last):
        return bool(pred(0, 0, 1, i, rows, prev, cur, first, last) & 2)

    assert id_ok(0, 0, 1) and id_ok(9, 0, 10) and id_ok(5, 5, 6)
    assert not id_ok(10, 0, 10) and not id_ok(-1, 0, 10) and not id_ok(4, 5, 6) and not id_ok(0, 0, 0)
    assert not id_ok(2 ** 31 - 1, 0, 1000) and not id_ok(-2 ** 31, 0, 1000)
    # a list of 3 rows with pointers 0, 2, 2, 7
    good = [0, 2, 2, 7]
    assert all(ptr_ok(i, 3, good[i - 1] if i else 0, good[i], 0, 7) for i in range(4))
    assert not ptr_ok(0, 3, 0, 1, 0, 7)            # does not start at the list's beginning
    assert not ptr_ok(2, 3, 2, 1, 0, 7)            # steps back
    assert not ptr_ok(3, 3, 2, 6, 0, 7)            # does not end at the list's length
    assert ptr_ok(3, 3, 7, 7, 0, 7) and ptr_ok(0, 0, 0, 0, 0, 0)
    # without a device there is nothing to check
    g = synth.config1_graph()
    h = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 4)
    mask = ctypes.c_uint32(5)
    assert lib.hag_device_validate(h._h, ctypes.byref(mask), None) == hb.HAG_ERR_NOT_ON_DEVICE and mask.value == 0
    assert lib.hag_device_validate(None, None, None) == 1


def test_large_aggregation_node_segments_follow_their_neighbourhoods():
    """Segments of 8192 aggregation-node rows or more (a level of the transposed HAG, an expansion list) are put in
    the order of their first entry before the windows are sorted by length: a permutation of the segment, windows
    sorted by length, and every window's first entries at or above those of the window before."""
    g = synth.config4_graph(seed=9, n_graphs=400, graph_size=100)
    h = hb.Hag.build(g.row_ptr, g.col_idx, g.n // 4)
    a = h.arrays()
    n, k = g.n, int(a["num_agg"])
    level_ptr = np.asarray(a["level_ptr"], dtype=np.int64)
    assert level_ptr[1] >= 8192

    def check_segment(order, first, ptr, idx, s0, s1):
        seg = order[s0:s1]
        assert np.array_equal(np.sort(seg), first + np.arange(s0, s1))                 # the segment maps onto itself
        lens = np.diff(ptr)
        key = np.where(lens > 0, idx[np.minimum(ptr[:-1], len(idx) - 1)], np.iinfo(np.int32).max)
        prev_max = -1
        for w0 in range(s0, s1, 2048):
            win = order[w0:min(w0 + 2048, s1)] - first
            assert np.all(np.diff(lens[win]) <= 0)                                     # longest first inside a window
            assert key[win].min() >= prev_max                                          # windows ascend in their first entries
            prev_max = key[win].max()
        moved = np.flatnonzero(seg != first + np.arange(s0, s1))
        assert moved.size > 0

    t_ptr, t_idx = np.asarray(a["t_ptr"], dtype=np.int64), np.asarray(a["t_idx"])
    first, order = h.row_order(1)
    assert first == 0 and order.size == n + k
    check_segment(order, 0, t_ptr, t_idx, n, n + int(level_ptr[1]))
    for cut_f, cut_b in ((0, 0),):
        h.set_cuts(cut_f, cut_b)
        v = h.arrays()
        for which, ptr_key, idx_key in ((4, "ftail_ptr", "ftail_idx"), (5, "btail_ptr", "btail_idx")):
            first, order = h.row_order(which)
            ptr, idx = np.asarray(v[ptr_key], dtype=np.int64), np.asarray(v[idx_key])
            assert first == n and order.size == k == ptr.size - 1
            check_segment(order, n, ptr, idx, 0, k)
