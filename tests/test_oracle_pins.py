"""Pins for the CPU oracle: it is checked against what the paper and the
mathematics fix, never against itself and never against the CUDA path."""
import json
import os

import numpy as np
import pytest
import scipy.sparse as sp

from oracle import oracle as O
from paper_1906_03707_b200 import synth


def _golden(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return json.load(f)


def _graph_from_rows(rows):
    return synth.csr_from_rows(rows)


SEARCHES = [O.greedy_bruteforce, O.greedy_pairmap, O.greedy_lazy]


# --------------------------------------------------------------------------- #
# worked examples (hand-derived from Algorithm 3, stored under tests/golden)
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("search", SEARCHES)
def test_k4_without_self_loops(golden_dir, search):
    gold = _golden(golden_dir, "k4_no_self_loops.json")
    g = _graph_from_rows(gold["rows"])
    res = search(g.row_ptr, g.col_idx, gold["capacity"])
    assert res.trace.tolist() == gold["trace"]
    assert [r.tolist() for r in res.rows] == gold["final_rows_creation_ids"]
    assert res.final_max_redundancy == 1
    h = O.canonical_hag(g.row_ptr, res)
    c = O.counters(g.row_ptr, h)
    assert (c["e"], c["e_hat"], c["num_levels"]) == (gold["e"], gold["e_hat"], gold["num_levels"])
    assert c["aggregations_gnn"] == gold["aggregations_gnn"]
    assert c["aggregations_hag"] == gold["aggregations_hag"] == c["aggregations_hag_closed_form"]


@pytest.mark.parametrize("search", SEARCHES)
def test_k4_with_self_loops_hierarchy_and_transposes(golden_dir, search):
    gold = _golden(golden_dir, "k4_self_loops.json")
    g = _graph_from_rows(gold["rows"])
    res = search(g.row_ptr, g.col_idx, gold["capacity"])
    assert res.trace.tolist() == gold["trace"]
    h = O.canonical_hag(g.row_ptr, res)
    assert h.level_ptr.tolist() == gold["level_ptr"]
    assert h.agg_in.tolist() == gold["agg_in"]
    assert h.res_ptr.tolist() == gold["res_ptr"]
    assert h.res_idx.tolist() == gold["res_idx"]
    assert h.t_ptr.tolist() == gold["t_ptr"]
    assert h.t_idx.tolist() == gold["t_idx"]
    c = O.counters(g.row_ptr, h)
    assert c["e_hat"] == gold["e_hat"]
    assert c["aggregations_gnn"] == gold["aggregations_gnn"]
    assert c["aggregations_hag"] == gold["aggregations_hag"]


@pytest.mark.parametrize("search", SEARCHES)
def test_level_sorted_renumbering(golden_dir, search):
    gold = _golden(golden_dir, "renumbering_13.json")
    g = _graph_from_rows(gold["rows"])
    res = search(g.row_ptr, g.col_idx, gold["capacity"])
    assert res.trace.tolist() == gold["trace"]
    h = O.canonical_hag(g.row_ptr, res)
    assert h.level_ptr.tolist() == gold["level_ptr"]
    assert h.agg_in.tolist() == gold["agg_in"]
    rows = [h.res_idx[h.res_ptr[v]:h.res_ptr[v + 1]].tolist() for v in range(g.n)]
    assert rows == gold["res_rows"]
    for s in range(g.n + h.num_agg):
        want = gold["transposed"].get(str(s), [])
        assert h.t_idx[h.t_ptr[s]:h.t_ptr[s + 1]].tolist() == want


# --------------------------------------------------------------------------- #
# closed forms
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("search", SEARCHES)
@pytest.mark.parametrize("n", [3, 5, 8, 11])
def test_complete_graph_with_self_loops_closed_form(search, n):
    # every row is the full node set: n-1 merges, each with redundancy n; |E-hat| = 3n-2;
    # aggregations n(n-1) -> n-1; every residual row is the single last aggregation node
    g = _graph_from_rows([list(range(n))] * n)
    res = search(g.row_ptr, g.col_idx, 10 * n)
    assert res.num_agg == n - 1
    assert (res.trace[:, 2] == n).all()
    h = O.canonical_hag(g.row_ptr, res)
    c = O.counters(g.row_ptr, h)
    assert c["e_hat"] == 3 * n - 2
    assert c["aggregations_gnn"] == n * (n - 1)
    assert c["aggregations_hag"] == n - 1
    assert np.diff(h.res_ptr).tolist() == [1] * n
    assert set(h.res_idx.tolist()) == {n + (n - 1) - 1}
    if n == 5:
        assert res.trace[:, :2].tolist() == [[0, 1], [2, 3], [4, 5], [6, 7]]
    if n == 8:
        levels = np.diff(h.level_ptr).tolist()
        assert levels == [4, 2, 1]


@pytest.mark.parametrize("search", SEARCHES)
def test_capacity_limit_on_k8(search):
    g = _graph_from_rows([list(range(8))] * 8)
    res = search(g.row_ptr, g.col_idx, 2)
    assert res.trace.tolist() == [[0, 1, 8], [2, 3, 8]]
    h = O.canonical_hag(g.row_ptr, res)
    c = O.counters(g.row_ptr, h)
    assert c["e_hat"] == 52 and c["aggregations_hag"] == 42
    assert res.final_max_redundancy == 8


@pytest.mark.parametrize("search", SEARCHES)
@pytest.mark.parametrize("k,m", [(2, 2), (3, 3), (5, 4), (2, 7)])
def test_identical_source_sets(search, k, m):
    # k destinations share one source set of size m: m-1 merges, all with redundancy k
    rows = [[] for _ in range(m)] + [list(range(m))] * k
    g = _graph_from_rows(rows)
    res = search(g.row_ptr, g.col_idx, 100)
    assert res.num_agg == m - 1
    assert (res.trace[:, 2] == k).all()
    c = O.counters(g.row_ptr, O.canonical_hag(g.row_ptr, res))
    assert c["aggregations_gnn"] == k * (m - 1)
    assert c["aggregations_hag"] == m - 1
    if (k, m) == (3, 3):
        assert (c["e"], c["e_hat"]) == (9, 7)


@pytest.mark.parametrize("search", SEARCHES)
def test_rings_have_no_or_little_sharing(search):
    for n in (5, 6, 9):
        g = _graph_from_rows([[(v - 1) % n, (v + 1) % n] for v in range(n)])
        res = search(g.row_ptr, g.col_idx, n)
        assert res.num_agg == 0 and res.final_max_redundancy == 1
        h = O.canonical_hag(g.row_ptr, res)
        assert np.array_equal(h.res_idx, g.col_idx) and np.array_equal(h.res_ptr, g.row_ptr)
    g = _graph_from_rows([[1, 3], [0, 2], [1, 3], [0, 2]])
    res = search(g.row_ptr, g.col_idx, 4)
    assert res.trace.tolist() == [[0, 2, 2], [1, 3, 2]]


def test_capacity_zero_is_the_gnn_graph():
    g = synth.config1_graph(seed=5, n=200)
    res = O.greedy_pairmap(g.row_ptr, g.col_idx, 0)
    h = O.canonical_hag(g.row_ptr, res)
    assert h.num_agg == 0 and h.num_levels == 0
    assert np.array_equal(h.res_idx, g.col_idx) and np.array_equal(h.res_ptr, g.row_ptr)
    t_ptr, t_idx = O.transposed_csr(g.row_ptr, g.col_idx)
    assert np.array_equal(h.t_ptr, t_ptr) and np.array_equal(h.t_idx, t_idx)


# --------------------------------------------------------------------------- #
# brute force confirms every merge, ties included
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("seed", range(40))
def test_pairmap_equals_bruteforce_on_tiny_graphs(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(6, 36))
    g = synth.random_digraph(seed, n, p=float(rng.uniform(0.15, 0.6)), undirected=bool(seed % 2),
                             self_loops=bool((seed // 2) % 2))
    for cap in (n // 4, 3 * n):
        a = O.greedy_bruteforce(g.row_ptr, g.col_idx, cap)
        b = O.greedy_pairmap(g.row_ptr, g.col_idx, cap)
        c = O.greedy_lazy(g.row_ptr, g.col_idx, cap)
        assert a.trace.tolist() == b.trace.tolist() == c.trace.tolist()
        assert [r.tolist() for r in a.rows] == [r.tolist() for r in c.rows]
        assert a.final_max_redundancy == c.final_max_redundancy
        assert [r.tolist() for r in a.rows] == [r.tolist() for r in b.rows]
        assert a.final_max_redundancy == b.final_max_redundancy
        # replay from the definition, with an arg-max recount at a few steps
        k = b.num_agg
        rows, fin = O.replay_trace(g.row_ptr, g.col_idx, b.trace, check_argmax_at={0, k // 2, max(k - 1, 0), k})
        assert [r.tolist() for r in rows] == [r.tolist() for r in b.rows]
        assert fin == b.final_max_redundancy
        if k < cap:
            assert fin <= 1
        # the plain-C replay used at full size: same rows, same left-over, and it sees through a wrong trace
        full = O.replay_trace_full(g.row_ptr, g.col_idx, b.trace, check_argmax_at=range(k + 1))
        assert full["ok"] and full["final_max_redundancy"] == a.final_max_redundancy
        assert full["full_recounts"] == k + 1
        assert [r.tolist() for r in full["rows"]] == [r.tolist() for r in a.rows]
        assert O.cover_check_rows(g.row_ptr, g.col_idx, b.trace, full["row_len"], full["row_store"]) == -1
        if k >= 2:
            wrong = b.trace.copy()
            wrong[k - 1, 2] += 1                                        # a redundancy that the rows do not have
            bad = O.replay_trace_full(g.row_ptr, g.col_idx, wrong)
            assert not bad["ok"] and bad["failed_step"] == k - 1 and bad["detail"][0] == b.trace[k - 1, 2]
            if tuple(b.trace[0, :2]) != tuple(b.trace[1, :2]) and b.trace[0, 2] > b.trace[1, 2]:
                wrong = b.trace.copy()
                wrong[[0, 1]] = wrong[[1, 0]]                           # a valid merge taken too early: not the arg-max
                bad = O.replay_trace_full(g.row_ptr, g.col_idx, wrong, check_argmax_at=[0])
                assert not bad["ok"] and bad["failed_step"] == 0
            # a row that lost a source no longer covers its neighbourhood
            rl = full["row_len"].copy()
            u = int(np.argmax(rl))
            rl[u] -= 1
            assert O.cover_check_rows(g.row_ptr, g.col_idx, b.trace, rl, full["row_store"]) == u


# --------------------------------------------------------------------------- #
# invariants on every built HAG
# --------------------------------------------------------------------------- #
def _invariants(g, res, h):
    c = O.counters(g.row_ptr, h)
    r = res.trace[:, 2].astype(np.int64)
    # Theorem 2 with cover as a multiset
    assert O.cover_multiset_ok(g.row_ptr, g.col_idx, h)
    # both forms of the cost function agree when every node aggregates something
    if c["closed_form_applies"]:
        assert c["aggregations_hag"] == c["aggregations_hag_closed_form"]
    # gain per merge: |E-hat| changes by 2 - r_i, aggregations by -(r_i - 1); f = sum (r_i - 1)
    assert c["e_hat"] == c["e"] + int((2 - r).sum())
    assert c["saved_f"] == int((r - 1).sum())
    assert c["aggregations_gnn"] - c["aggregations_hag"] == c["saved_f"]
    # submodularity: the marginal gain never grows
    assert (r >= 2).all() and (np.diff(r) <= 0).all()
    # structure: two inputs each, inputs precede their node, levels are longest paths
    pairs = h.agg_in.reshape(-1, 2)
    assert (pairs[:, 0] < pairs[:, 1]).all()
    ids = g.n + np.arange(h.num_agg)
    assert (pairs[:, 1] < ids).all()
    level = np.zeros(g.n + h.num_agg, dtype=np.int64)
    for j in range(h.num_agg):
        level[g.n + j] = 1 + max(level[pairs[j, 0]], level[pairs[j, 1]])
    assert (np.diff(level[g.n:]) >= 0).all()
    for l in range(1, h.num_levels + 1):
        assert (level[g.n + h.level_ptr[l - 1]: g.n + h.level_ptr[l]] == l).all()
    # transposed HAG is the same edge set
    assert h.t_idx.shape[0] == c["e_hat"]
    return c


@pytest.mark.parametrize("maker", [
    lambda: synth.workload(1).graph,
    lambda: synth.config2_graph(seed=11, n=1500, n_comm=15),
    lambda: synth.config3_graph(seed=12, n=900, n_comm=3, d_lo=10, d_hi=200),
    lambda: synth.config4_graph(seed=13, n_graphs=12, graph_size=40),
    lambda: synth.config5_graph(seed=14, n=2000, n_comm=8, s_lo=60, s_hi=600, d_lo=8, d_hi=100),
    lambda: synth.clique_union_graph(seed=15, n=600, n_groups=150, g_lo=3, g_hi=30),
])
def test_invariants_and_values_on_workload_shapes(maker):
    g = maker()
    res = O.greedy_pairmap(g.row_ptr, g.col_idx, g.n // 4)
    lazy = O.greedy_lazy(g.row_ptr, g.col_idx, g.n // 4)
    assert lazy.trace.tolist() == res.trace.tolist() and lazy.final_max_redundancy == res.final_max_redundancy
    h = O.canonical_hag(g.row_ptr, res)
    c = _invariants(g, res, h)
    assert c["num_agg"] > 0
    x = synth.features(3, g.n, 8, "normal").astype(np.float64)
    gr = synth.upstream_grad(3, g.n, 8, "normal").astype(np.float64)
    for reduce in ("sum", "mean"):
        a, t = O.direct_forward(g.row_ptr, g.col_idx, x, reduce)
        np.testing.assert_allclose(O.hag_forward(h, x, reduce), a, rtol=0, atol=1e-12 * max(1.0, t.max()))
        gx, tg = O.direct_backward(g.row_ptr, g.col_idx, gr, reduce)
        np.testing.assert_allclose(O.hag_backward(h, gr, reduce), gx, rtol=0, atol=1e-12 * max(1.0, tg.max()))


def test_config1_shape_matches_its_statement():
    w = synth.workload(1)
    g = w.graph
    assert g.n == 1000 and w.capacity == 250 and w.d == 16
    # expected directed edges: 2 * (10 * C(100,2) * 0.1 + (C(1000,2) - 10*C(100,2)) * 0.001) + 1000 = 11 800
    assert abs(g.e - 11800) < 600
    res = O.greedy_pairmap(g.row_ptr, g.col_idx, w.capacity)
    assert res.num_agg == 250
    _invariants(g, res, O.canonical_hag(g.row_ptr, res))


# --------------------------------------------------------------------------- #
# the value oracle against library routines and closed forms
# --------------------------------------------------------------------------- #
def _dense_adjacency(g):
    a = np.zeros((g.n, g.n))
    for v in range(g.n):
        a[v, g.col_idx[g.row_ptr[v]:g.row_ptr[v + 1]]] = 1.0
    return a


@pytest.mark.parametrize("undirected", [False, True])
def test_direct_aggregation_is_spmm(undirected):
    g = synth.random_digraph(21, 60, 0.2, undirected=undirected, self_loops=False)
    x = synth.features(1, g.n, 5, "normal").astype(np.float64)
    gr = synth.upstream_grad(1, g.n, 5, "normal").astype(np.float64)
    a_mat = sp.csr_matrix((np.ones(g.e), g.col_idx, g.row_ptr), shape=(g.n, g.n))
    deg = np.diff(g.row_ptr).astype(np.float64)
    inv = np.where(deg > 0, 1.0 / np.maximum(deg, 1), 1.0)
    out, t = O.direct_forward(g.row_ptr, g.col_idx, x, "sum")
    np.testing.assert_allclose(out, a_mat @ x, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(t, a_mat @ np.abs(x), rtol=1e-13, atol=1e-13)
    out_m, _ = O.direct_forward(g.row_ptr, g.col_idx, x, "mean")
    np.testing.assert_allclose(out_m, (a_mat @ x) * inv[:, None], rtol=1e-13, atol=1e-13)
    gx, tg = O.direct_backward(g.row_ptr, g.col_idx, gr, "sum")
    np.testing.assert_allclose(gx, a_mat.T @ gr, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(tg, a_mat.T @ np.abs(gr), rtol=1e-13, atol=1e-13)
    gx_m, _ = O.direct_backward(g.row_ptr, g.col_idx, gr, "mean")
    np.testing.assert_allclose(gx_m, a_mat.T @ (gr * inv[:, None]), rtol=1e-13, atol=1e-13)
    # dense definition, written independently of the CSR walk
    dense = _dense_adjacency(g)
    np.testing.assert_allclose(out, dense @ x, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(gx, dense.T @ gr, rtol=1e-13, atol=1e-13)


def test_gcn_mode_is_the_normalised_sum_with_the_own_row():
    # Table 1, GCN: the argument of Update is (a_v + h_v) / (|N(v)| + 1) = D^-1 (A + I) x with D = deg + 1
    g = synth.random_digraph(23, 50, 0.2, undirected=False, self_loops=False)
    x = synth.features(2, g.n, 4, "normal").astype(np.float64)
    gr = synth.upstream_grad(2, g.n, 4, "normal").astype(np.float64)
    a_mat = sp.csr_matrix((np.ones(g.e), g.col_idx, g.row_ptr), shape=(g.n, g.n)) + sp.identity(g.n)
    inv = 1.0 / (np.diff(g.row_ptr) + 1.0)
    out, t = O.direct_forward(g.row_ptr, g.col_idx, x, "gcn")
    np.testing.assert_allclose(out, (a_mat @ x) * inv[:, None], rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(t, (a_mat @ np.abs(x)) * inv[:, None], rtol=1e-13, atol=1e-13)
    gx, _ = O.direct_backward(g.row_ptr, g.col_idx, gr, "gcn")
    np.testing.assert_allclose(gx, a_mat.T @ (gr * inv[:, None]), rtol=1e-13, atol=1e-13)
    rows = np.asarray([3, 0, 49, 17])
    part, _ = O.direct_backward(g.row_ptr, g.col_idx, gr, "gcn", rows=rows)
    assert np.array_equal(part, gx[rows])
    lhs = float((out * gr).sum())
    rhs = float((x * gx).sum())
    assert abs(lhs - rhs) < 1e-10


def test_direct_aggregation_on_a_star_is_not_its_transpose():
    # node 0 aggregates 1..4; nobody else aggregates anything
    g = _graph_from_rows([[1, 2, 3, 4], [], [], [], []])
    x = np.arange(10, dtype=np.float64).reshape(5, 2)
    out, _ = O.direct_forward(g.row_ptr, g.col_idx, x, "sum")
    assert out.tolist() == [[2 + 4 + 6 + 8, 3 + 5 + 7 + 9], [0, 0], [0, 0], [0, 0], [0, 0]]
    out_m, _ = O.direct_forward(g.row_ptr, g.col_idx, x, "mean")
    assert out_m[0].tolist() == [5.0, 6.0] and not out_m[1:].any()
    gr = np.asarray([[1.0, -2.0], [10, 10], [20, 20], [30, 30], [40, 40]])
    gx, _ = O.direct_backward(g.row_ptr, g.col_idx, gr, "sum")
    assert gx.tolist() == [[0, 0], [1, -2], [1, -2], [1, -2], [1, -2]]
    gx_m, _ = O.direct_backward(g.row_ptr, g.col_idx, gr, "mean")
    assert gx_m.tolist() == [[0, 0], [0.25, -0.5], [0.25, -0.5], [0.25, -0.5], [0.25, -0.5]]


def test_direct_subset_rows_match_full():
    g = synth.config2_graph(seed=31, n=1200, n_comm=12)
    x = synth.features(2, g.n, 4, "uniform").astype(np.float64)
    rows = np.asarray([0, 7, 500, 1199, 3])
    full, tf = O.direct_forward(g.row_ptr, g.col_idx, x, "mean")
    part, tp = O.direct_forward(g.row_ptr, g.col_idx, x, "mean", rows=rows)
    assert np.array_equal(part, full[rows]) and np.array_equal(tp, tf[rows])
    fullb, tb = O.direct_backward(g.row_ptr, g.col_idx, x, "mean")
    partb, tpb = O.direct_backward(g.row_ptr, g.col_idx, x, "mean", rows=rows)
    assert np.array_equal(partb, fullb[rows]) and np.array_equal(tpb, tb[rows])


def test_adjoint_identity_and_linearity():
    g = synth.config2_graph(seed=32, n=1000, n_comm=10)
    res = O.greedy_pairmap(g.row_ptr, g.col_idx, g.n // 4)
    h = O.canonical_hag(g.row_ptr, res)
    x = synth.features(4, g.n, 6, "normal").astype(np.float64)
    y = synth.features(5, g.n, 6, "normal").astype(np.float64)
    gr = synth.upstream_grad(4, g.n, 6, "normal").astype(np.float64)
    for reduce in ("sum", "mean"):
        lhs = float((O.hag_forward(h, x, reduce) * gr).sum())
        rhs = float((x * O.hag_backward(h, gr, reduce)).sum())
        assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))
        lin = O.hag_forward(h, 2.0 * x - 3.0 * y, reduce)
        np.testing.assert_allclose(lin, 2.0 * O.hag_forward(h, x, reduce) - 3.0 * O.hag_forward(h, y, reduce),
                                   rtol=0, atol=1e-10)


def test_integer_features_are_exact():
    g = synth.workload(1).graph
    res = O.greedy_pairmap(g.row_ptr, g.col_idx, 250)
    h = O.canonical_hag(g.row_ptr, res)
    x = synth.features(6, g.n, 16, "int").astype(np.float64)
    a, _ = O.direct_forward(g.row_ptr, g.col_idx, x, "sum")
    assert np.array_equal(O.hag_forward(h, x, "sum"), a)
    assert np.array_equal(a, np.rint(a))


def test_expanded_deep_levels_are_covers_and_transitive_users():
    """For EVERY cut the expansion lists must reproduce the level-by-level values: the forward
    list of a deep node sums to its a-hat, the backward list of a deep node to its gradient;
    cut 0 gives cover(v) itself (Section 3.1, Eq. 1), the deepest cut gives nothing to expand."""
    g = synth.clique_union_graph(seed=16, n=500, n_groups=140, g_lo=3, g_hi=30)
    res = O.greedy_pairmap(g.row_ptr, g.col_idx, g.n // 2)
    h = O.canonical_hag(g.row_ptr, res)
    L = h.num_levels
    assert L >= 4
    rng = np.random.default_rng(0)
    x = rng.integers(-5, 6, size=(g.n, 3)).astype(np.float64)
    ahat = np.concatenate([x, np.zeros((h.num_agg, 3))])
    for j in range(h.num_agg):
        ahat[g.n + j] = ahat[h.agg_in[2 * j]] + ahat[h.agg_in[2 * j + 1]]
    gr = rng.integers(-5, 6, size=(g.n, 3)).astype(np.float64)
    ghat = np.zeros((h.num_agg, 3))
    for j in range(h.num_agg - 1, -1, -1):
        for d in h.t_idx[h.t_ptr[g.n + j]: h.t_ptr[g.n + j + 1]]:
            ghat[j] += gr[d] if d < g.n else ghat[d - g.n]
    level = np.zeros(g.n + h.num_agg, dtype=np.int64)
    for l in range(1, L + 1):
        level[g.n + h.level_ptr[l - 1]: g.n + h.level_ptr[l]] = l
    # cover(v) by its recursive definition, as a multiset of graph nodes
    cover = {}
    for j in range(h.num_agg):
        c = []
        for s_ in h.agg_in[2 * j: 2 * j + 2]:
            c.extend([int(s_)] if s_ < g.n else cover[int(s_)])
        cover[g.n + j] = sorted(c)
    for cut in range(L + 1):
        t = O.expanded_tails(h, cut, cut)
        assert t["fwd_cut"] == cut and t["bwd_cut"] == cut
        j0 = int(h.level_ptr[cut])
        assert t["ftail_ptr"].shape[0] == h.num_agg - j0 + 1 == t["btail_ptr"].shape[0]
        for i in range(h.num_agg - j0):
            ids = t["ftail_idx"][t["ftail_ptr"][i]: t["ftail_ptr"][i + 1]]
            assert len(set(ids.tolist())) == len(ids) and (level[ids] <= cut).all()
            assert np.array_equal(ahat[ids].sum(0), ahat[g.n + j0 + i])
            if cut == 0:
                assert ids.tolist() == cover[g.n + j0 + i]
            ids = t["btail_idx"][t["btail_ptr"][i]: t["btail_ptr"][i + 1]]
            assert (ids < g.n).all() and len(set(ids.tolist())) == len(ids)
            assert np.array_equal(gr[ids].sum(0), ghat[j0 + i])
        assert np.array_equal(O.expanded_forward(h, x, cut, t), ahat)
    with pytest.raises(ValueError):
        O.expanded_tails(h, L + 1, 0)


# --------------------------------------------------------------------------- #
# Graph read-out (mean-pooling layer of Section 5.1)
# --------------------------------------------------------------------------- #
def _ragged_segments(seed, m, max_len, with_empty=True):
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, max_len + 1, size=m)
    if with_empty:
        lens[rng.integers(0, m, size=max(1, m // 7))] = 0
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)


def test_graph_pool_closed_forms():
    # x[v, j] = v + 1000 j: the sum over rows b..e-1 is an arithmetic series
    sp_ = np.array([0, 3, 3, 10, 11, 40], dtype=np.int64)
    n, d = 40, 5
    x = np.arange(n, dtype=np.float64)[:, None] + 1000.0 * np.arange(d)[None, :]
    s, _ = O.graph_pool_forward(sp_, x, "sum")
    mean, t = O.graph_pool_forward(sp_, x, "mean")
    for i in range(5):
        b, e = int(sp_[i]), int(sp_[i + 1])
        k = e - b
        series = (b + e - 1) * k / 2.0
        assert np.array_equal(s[i], series + 1000.0 * np.arange(d) * k)
        if k:
            assert np.allclose(mean[i], (b + e - 1) / 2.0 + 1000.0 * np.arange(d), rtol=1e-15)
            assert np.allclose(t[i], mean[i], rtol=1e-15)          # all terms are positive
        else:
            assert not mean[i].any() and not s[i].any()            # a graph without nodes: zero row


def test_graph_pool_mean_of_a_constant_is_the_constant():
    sp_ = _ragged_segments(3, 50, 30, with_empty=False)
    x = np.full((int(sp_[-1]), 7), -2.75)
    out, t = O.graph_pool_forward(sp_, x, "mean")
    assert np.allclose(out, -2.75, rtol=1e-15) and np.allclose(t, 2.75, rtol=1e-15)


def test_graph_pool_matches_reduceat_and_a_dense_pooling_matrix():
    sp_ = _ragged_segments(4, 60, 25, with_empty=False)
    n = int(sp_[-1])
    x = np.random.default_rng(5).standard_normal((n, 9))
    s, _ = O.graph_pool_forward(sp_, x, "sum")
    assert np.allclose(s, np.add.reduceat(x, sp_[:-1], axis=0), rtol=1e-13, atol=1e-13)
    # P[i, v] = 1/|G_i| for v in G_i: forward is P x, backward is P^T g
    sp2 = _ragged_segments(6, 40, 12)
    n2 = int(sp2[-1])
    p = np.zeros((40, n2))
    for i in range(40):
        if sp2[i + 1] > sp2[i]:
            p[i, sp2[i]:sp2[i + 1]] = 1.0 / (sp2[i + 1] - sp2[i])
    x2 = np.random.default_rng(7).standard_normal((n2, 6))
    g2 = np.random.default_rng(8).standard_normal((40, 6))
    out, _ = O.graph_pool_forward(sp2, x2, "mean")
    gx, _ = O.graph_pool_backward(sp2, g2, n2, "mean")
    assert np.allclose(out, p @ x2, rtol=1e-12, atol=1e-13)
    assert np.allclose(gx, p.T @ g2, rtol=1e-12, atol=1e-13)
    gs, _ = O.graph_pool_backward(sp2, g2, n2, "sum")
    assert np.allclose(gs, (p != 0).T.astype(np.float64) @ g2, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("reduce", ["sum", "mean"])
def test_graph_pool_adjoint_identity(reduce):
    sp_ = _ragged_segments(9, 33, 17)
    n = int(sp_[-1]) + 4                       # trailing rows that belong to no graph
    rng = np.random.default_rng(10)
    x = rng.standard_normal((n, 4))
    g = rng.standard_normal((33, 4))
    out, _ = O.graph_pool_forward(sp_, x, reduce)
    gx, _ = O.graph_pool_backward(sp_, g, n, reduce)
    assert abs((out * g).sum() - (x * gx).sum()) < 1e-10
    assert not gx[int(sp_[-1]):].any()


# --------------------------------------------------------------------------- #
# Element-wise max aggregation (GraphSAGE-P row of Table 1)
# --------------------------------------------------------------------------- #
def _max_bruteforce(g, z, gr):
    """Loops over the definition: a_v[k] = max_{u in N(v)} z_u[k]; each maximiser receives g_v[k]."""
    n, d = z.shape
    a = np.zeros((n, d))
    gz = np.zeros((n, d))
    for v in range(n):
        nb = [int(u) for u in g.col_idx[g.row_ptr[v]:g.row_ptr[v + 1]]]
        for k in range(d):
            if not nb:
                continue
            m = max(z[u, k] for u in nb)
            a[v, k] = m
            for u in nb:
                if z[u, k] == m:
                    gz[u, k] += gr[v, k]
    return a, gz


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("ties", [False, True])
def test_max_matches_bruteforce_on_tiny_graphs(seed, ties):
    rng = np.random.default_rng(100 + seed)
    g = synth.random_digraph(seed=seed, n=int(rng.integers(5, 30)), p=0.3, undirected=bool(seed % 3 == 0), self_loops=bool(seed % 2))
    d = 3
    z = rng.integers(-2, 3, size=(g.n, d)).astype(np.float64) if ties else rng.standard_normal((g.n, d))
    gr = rng.integers(-4, 5, size=(g.n, d)).astype(np.float64)
    a, gz = _max_bruteforce(g, z, gr)
    assert np.array_equal(O.direct_max_forward(g.row_ptr, g.col_idx, z), a)
    got, t = O.direct_max_backward(g.row_ptr, g.col_idx, z, gr)
    assert np.array_equal(got, gz)
    assert (t >= np.abs(got)).all()
    # the row-subset forms used at full size: same loops over the definition, rows in any order
    rows = rng.permutation(g.n)[: max(1, g.n // 2)]
    assert np.array_equal(O.direct_max_forward(g.row_ptr, g.col_idx, z, rows=rows), a[rows])
    sub, tsub = O.direct_max_backward(g.row_ptr, g.col_idx, z, gr, rows=rows)
    assert np.array_equal(sub, gz[rows]) and np.array_equal(tsub, t[rows])


def test_max_is_the_masked_dense_maximum_and_empty_rows_are_zero():
    g = synth.random_digraph(seed=3, n=40, p=0.08, undirected=False, self_loops=False)
    assert (np.diff(g.row_ptr) == 0).any()                     # the case has empty neighbourhoods
    z = np.random.default_rng(4).standard_normal((g.n, 5))
    adj = np.zeros((g.n, g.n), dtype=bool)
    for v in range(g.n):
        adj[v, g.col_idx[g.row_ptr[v]:g.row_ptr[v + 1]]] = True
    dense = np.where(adj[:, :, None], z[None, :, :], -np.inf).max(axis=1)
    dense[~adj.any(axis=1)] = 0.0
    assert np.array_equal(O.direct_max_forward(g.row_ptr, g.col_idx, z), dense)


def test_max_gradient_is_the_finite_difference_of_the_loss():
    # without ties the aggregation is linear around z, so a small step gives the derivative exactly
    g = synth.random_digraph(seed=5, n=9, p=0.45, undirected=False, self_loops=True)
    rng = np.random.default_rng(6)
    z = rng.permutation(g.n * 3).reshape(g.n, 3).astype(np.float64)        # all distinct, gaps of 1
    gr = rng.standard_normal((g.n, 3))
    gz, _ = O.direct_max_backward(g.row_ptr, g.col_idx, z, gr)
    base = (gr * O.direct_max_forward(g.row_ptr, g.col_idx, z)).sum()
    eps = 1.0 / 64.0
    for u in range(g.n):
        for k in range(3):
            zp = z.copy()
            zp[u, k] += eps
            num = ((gr * O.direct_max_forward(g.row_ptr, g.col_idx, zp)).sum() - base) / eps
            assert abs(num - gz[u, k]) < 1e-9


def test_max_closed_forms():
    g = synth.config1_graph()
    n = g.n
    rng = np.random.default_rng(7)
    gr = rng.standard_normal((n, 4))
    # constant features: every in-neighbour ties, so the gradient is that of the sum
    gz, _ = O.direct_max_backward(g.row_ptr, g.col_idx, np.full((n, 4), 1.5), gr)
    want, _ = O.direct_backward(g.row_ptr, g.col_idx, gr, "sum")
    assert np.allclose(gz, want, rtol=1e-13, atol=1e-13)
    # features that grow with the node id: the maximum sits at the last (largest) in-neighbour of the sorted row
    z = np.arange(n, dtype=np.float64)[:, None] * np.ones((1, 4))
    a = O.direct_max_forward(g.row_ptr, g.col_idx, z)
    last = g.col_idx[g.row_ptr[1:] - 1]
    assert np.array_equal(a[:, 0], last.astype(np.float64))
    gz, _ = O.direct_max_backward(g.row_ptr, g.col_idx, z, gr)
    want = np.zeros((n, 4))
    np.add.at(want, last, gr)
    assert np.allclose(gz, want, rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("maker", [lambda: synth.config1_graph(), lambda: synth.workload(2, scale=0.05).graph,
                                   lambda: synth.clique_union_graph(seed=2, n=600, n_groups=150, g_lo=2, g_hi=40, g_alpha=2.0)])
def test_hag_max_equals_direct_max(maker):
    """Theorem 2's cover condition makes Algorithm 2 with any associative, commutative operator reach
    the GNN-graph's result; for max that holds bit for bit, and with integer gradients so does the backward
    pass, ties included."""
    g = maker()
    res = O.greedy_pairmap(g.row_ptr, g.col_idx, g.n // 4)
    h = O.canonical_hag(g.row_ptr, res)
    assert h.num_agg > 0
    rng = np.random.default_rng(8)
    for z in (rng.standard_normal((g.n, 6)), rng.integers(-1, 2, size=(g.n, 6)).astype(np.float64)):
        gr = rng.integers(-3, 4, size=(g.n, 6)).astype(np.float64)
        out, ahat = O.hag_max_forward(h, z)
        assert np.array_equal(out, O.direct_max_forward(g.row_ptr, g.col_idx, z))
        for j in rng.integers(0, h.num_agg, size=20):          # an aggregation node holds the max over its inputs
            p, q = h.agg_in[2 * j], h.agg_in[2 * j + 1]
            assert np.array_equal(ahat[h.n + j], np.maximum(ahat[p], ahat[q]))
        want, _ = O.direct_max_backward(g.row_ptr, g.col_idx, z, gr)
        assert np.array_equal(O.hag_max_backward(h, z, gr), want)
