"""CPU oracle for HAG aggregation -- TEST INFRASTRUCTURE, not part of the product.

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline leg
may import this module.  It imports nothing from the CUDA package and the CUDA
package imports nothing from here.

What it computes, and where the paper (arxiv 1906.03707) defines it:

* ``direct_forward`` / ``direct_backward`` -- Algorithm 1 line 4 (GCN row of
  Table 1) and its gradient (equivalence clause (2), Section 3.2), fp64, straight
  from the definition.  These are the value oracle: by Theorem 2 a HAG reaches
  exactly this result.
* ``greedy_bruteforce`` -- Algorithm 3, set branch, recounting Redundancy for
  every pair from scratch in every iteration (tiny graphs only).
* ``greedy_pairmap`` -- Algorithm 3 with the pair-count heap of the complexity
  appendix (plain C).
* ``greedy_lazy`` -- Algorithm 3 with per-node bounds confirmed by recounts (plain
  C, memory O(|E|)), for the shapes whose pair map does not fit in memory.
* ``canonical_hag`` -- the run-time layout: levels (longest path from a source),
  level-sorted renumbering, input pairs, residual CSR, transposed HAG.
* ``hag_forward`` / ``hag_backward`` -- Algorithm 2 and its adjoint over that
  layout, fp64.
* ``cover_multiset_ok``, ``counters``, ``replay_trace`` -- Theorem 2's condition,
  the cost function of Section 4.1 in both forms, f = |E| - |E-hat| + |V_A| of
  the Theorem 4 proof, and a from-the-definition replay of a merge trace;
  ``replay_trace_full`` / ``cover_check_rows`` -- the same two checks in plain C,
  for the full-size workload shapes.
* ``expanded_tails`` / ``expanded_forward`` -- for GIVEN cuts, the cover-restricted
  input lists (Section 3.1, Eq. 1) and transitive users of the deep levels.  The
  choice of a cut is a launch heuristic of whoever evaluates the HAG; the paper
  fixes nothing about it, so nothing here chooses one.

* ``graph_pool_forward`` / ``graph_pool_backward`` -- the mean-pooling layer that the
  experimental setup (Section 5.1) puts after the GNN layers for graph
  classification: one output row per graph of a batch, the mean (or sum) of the
  rows of its nodes, and the gradient of that; fp64, one slice sum per graph.

* ``direct_max_forward`` / ``direct_max_backward`` -- the element-wise max Aggregate of
  the GraphSAGE-P row of Table 1 from its definition, and its gradient;
  ``hag_max_forward`` / ``hag_max_backward`` -- Algorithm 2 with max as the operator
  (a set Aggregate in the sense of Section 3.1) and its gradient over the
  transposed HAG.  Reading: on a tie every in-neighbour that attains the maximum
  receives the gradient component (the paper does not say; ties have probability
  zero for continuous activations).

Readings of points the paper leaves open:
redundancy counts graph nodes u in V only (the rewrite loop of Algorithm 3 runs
over V); pairs are unordered over V and V_A; ties go to the lexicographically
smallest (v1, v2), v1 < v2, aggregation nodes numbered N, N+1, ... as created;
the loop stops when the best redundancy is <= 1 or |V_A| = capacity; an empty
neighbourhood yields a zero row; mean divides by the in-degree in the input graph.

Parity pins: see tests/test_oracle_pins.py.  The three searches must agree
merge for merge; the memory-light one is what reaches the two largest workload
shapes, and it is pinned against brute force and against the pair-count heap.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle.c with gcc (building the checker is not using it)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"])
    return _SO


def _c():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32 = ctypes.c_int64, ctypes.c_int32
        p = ctypes.c_void_p
        lib.o1_direct_forward.argtypes = [i64, p, p, i64, p, ctypes.c_int, p, i64, p, p]
        lib.o1_direct_forward.restype = None
        lib.o2_direct_backward.argtypes = [i64, p, p, i64, p, ctypes.c_int, p, i64, p, p]
        lib.o2_direct_backward.restype = None
        lib.o4_hag_forward.argtypes = [i64, i64, p, p, p, p, i64, p, ctypes.c_int, p, p]
        lib.o4_hag_forward.restype = None
        lib.o4_hag_backward.argtypes = [i64, i64, p, p, p, i64, p, ctypes.c_int, p, p]
        lib.o4_hag_backward.restype = None
        lib.o6_max_forward.argtypes = [i64, p, p, i64, p, p]
        lib.o6_max_forward.restype = None
        lib.o6_max_forward_rows.argtypes = [i64, p, p, i64, p, p, i64, p]
        lib.o6_max_forward_rows.restype = None
        lib.o6_max_backward.argtypes = [i64, p, p, i64, p, p, p, p, p]
        lib.o6_max_backward.restype = None
        lib.o7_hag_max_forward.argtypes = [i64, i64, p, p, p, i64, p, p, p]
        lib.o7_hag_max_forward.restype = None
        lib.o7_hag_max_backward.argtypes = [i64, i64, p, p, i64, p, p, p, p, p]
        lib.o7_hag_max_backward.restype = None
        lib.o_count_pair.argtypes = [i64, p, p, p, i32, i32]
        lib.o_count_pair.restype = i64
        lib.o_max_pair_recount.argtypes = [i64, p, p, p, i64, i32, p, p]
        lib.o_max_pair_recount.restype = i64
        lib.o3b_greedy.argtypes = [i64, p, p, i64, i32, p, p, p, p, p, p]
        lib.o3b_greedy.restype = i64
        lib.o3c_greedy.argtypes = [i64, p, p, i64, i32, p, p, p, p, p, p]
        lib.o3c_greedy.restype = i64
        lib.o_replay_trace.argtypes = [i64, p, p, i64, p, p, p, i32, i64, p, p, p, p]
        lib.o_replay_trace.restype = i64
        lib.o_cover_check.argtypes = [i64, p, p, i64, p, p, p, p]
        lib.o_cover_check.restype = i64
        _lib = lib
    return _lib


def _mode(reduce) -> int:
    return {"sum": 0, "mean": 1, "gcn": 2}[reduce]


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _csr(row_ptr, col_idx):
    rp = np.ascontiguousarray(row_ptr, dtype=np.int64)
    ci = np.ascontiguousarray(col_idx, dtype=np.int32)
    return rp, ci


# --------------------------------------------------------------------------- #
# O1 / O2: the value oracle
# --------------------------------------------------------------------------- #
def direct_forward(row_ptr, col_idx, x, reduce="sum", rows=None):
    """a_v = sum_{u in N(v)} x_u (mean: / |N(v)|) in fp64.  Returns (a, T) with
    T = sum |x_u| (same scaling), the scale of the comparison tolerance.
    ``rows``: optional subset of nodes; the result then has one row per entry."""
    rp, ci = _csr(row_ptr, col_idx)
    n = rp.shape[0] - 1
    x = np.ascontiguousarray(x, dtype=np.float64)
    d = x.shape[1]
    sel = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    m = n if sel is None else sel.shape[0]
    out = np.empty((m, d), dtype=np.float64)
    ab = np.empty((m, d), dtype=np.float64)
    _c().o1_direct_forward(n, _ptr(rp), _ptr(ci), d, _ptr(x), _mode(reduce), _ptr(sel), m, _ptr(out), _ptr(ab))
    return out, ab


def direct_backward(row_ptr, col_idx, g, reduce="sum", rows=None):
    """gx_u = sum_{v : u in N(v)} s_v g_v, s_v = 1 (sum) or 1/|N(v)| (mean), fp64.
    Returns (gx, T).  ``rows``: optional subset of source nodes u."""
    rp, ci = _csr(row_ptr, col_idx)
    n = rp.shape[0] - 1
    g = np.ascontiguousarray(g, dtype=np.float64)
    d = g.shape[1]
    slot = None
    m = n
    if rows is not None:
        sel = np.ascontiguousarray(rows, dtype=np.int64)
        m = sel.shape[0]
        slot = np.full(n, -1, dtype=np.int64)
        slot[sel] = np.arange(m, dtype=np.int64)
        if np.unique(sel).shape[0] != m:
            raise ValueError("rows must be distinct")
    out = np.empty((m, d), dtype=np.float64)
    ab = np.empty((m, d), dtype=np.float64)
    _c().o2_direct_backward(n, _ptr(rp), _ptr(ci), d, _ptr(g), _mode(reduce), _ptr(slot), m, _ptr(out), _ptr(ab))
    return out, ab


def graph_pool_forward(seg_ptr, x, reduce="mean"):
    """Graph-level read-out of Section 5.1: graph i owns the node rows
    seg_ptr[i] .. seg_ptr[i+1]-1; out_i = sum of those rows (mean: divided by their
    number; a graph without nodes gives a zero row).  Returns (out, T), T = the same
    with |x| (the scale of the comparison tolerance)."""
    sp = np.ascontiguousarray(seg_ptr, dtype=np.int64)
    x = np.ascontiguousarray(x, dtype=np.float64)
    m = sp.shape[0] - 1
    out = np.zeros((m, x.shape[1]), dtype=np.float64)
    ab = np.zeros((m, x.shape[1]), dtype=np.float64)
    for i in range(m):
        b, e = int(sp[i]), int(sp[i + 1])
        if e <= b:
            continue
        w = 1.0 / (e - b) if reduce == "mean" else 1.0
        out[i] = x[b:e].sum(axis=0) * w
        ab[i] = np.abs(x[b:e]).sum(axis=0) * w
    return out, ab


def graph_pool_backward(seg_ptr, g, n_rows, reduce="mean"):
    """Gradient of graph_pool_forward: every node row of graph i receives g_i
    (mean: divided by the number of nodes of the graph); rows outside every graph
    receive zero.  Returns (gx, T) with T = |gx|."""
    sp = np.ascontiguousarray(seg_ptr, dtype=np.int64)
    g = np.ascontiguousarray(g, dtype=np.float64)
    gx = np.zeros((int(n_rows), g.shape[1]), dtype=np.float64)
    for i in range(sp.shape[0] - 1):
        b, e = int(sp[i]), int(sp[i + 1])
        if e <= b:
            continue
        w = 1.0 / (e - b) if reduce == "mean" else 1.0
        gx[b:e] = g[i] * w
    return gx, np.abs(gx)


# --------------------------------------------------------------------------- #
# O3: Algorithm 3
# --------------------------------------------------------------------------- #
@dataclass
class SearchResult:
    """Outcome of Algorithm 3 in creation-id space."""

    n: int
    trace: np.ndarray          # int32[num_agg, 3]: v1, v2 (v1 < v2, creation ids), redundancy
    rows: list                 # rows[u] = remaining in-neighbours of graph node u, ascending creation ids
    final_max_redundancy: int  # best redundancy left when the loop stopped

    @property
    def num_agg(self) -> int:
        return int(self.trace.shape[0])


def greedy_bruteforce(row_ptr, col_idx, capacity, min_redundancy=2) -> SearchResult:
    """Algorithm 3 exactly as stated: every iteration recounts, for every
    unordered pair, how many graph nodes aggregate both; takes the largest
    (ties: smallest v1, then smallest v2); stops at redundancy <= 1."""
    rp, ci = _csr(row_ptr, col_idx)
    n = rp.shape[0] - 1
    rows = [set(int(c) for c in ci[rp[u]:rp[u + 1]]) for u in range(n)]
    trace = []
    last_max = 0
    while True:
        counts = {}
        for u in range(n):
            members = sorted(rows[u])
            for i in range(len(members)):
                for j in range(i + 1, len(members)):
                    key = (members[i], members[j])
                    counts[key] = counts.get(key, 0) + 1
        best_pair, best = None, 0
        for key, c in counts.items():
            if c > best or (c == best and key < best_pair):
                best_pair, best = key, c
        last_max = best
        if len(trace) >= capacity or best < min_redundancy:     # 2: the paper's "Redundancy > 1"
            break
        v1, v2 = best_pair
        w = n + len(trace)
        for u in range(n):
            if v1 in rows[u] and v2 in rows[u]:
                rows[u].discard(v1)
                rows[u].discard(v2)
                rows[u].add(w)
        trace.append((v1, v2, best))
    tr = np.asarray(trace, dtype=np.int32).reshape(-1, 3)
    return SearchResult(n, tr, [np.asarray(sorted(r), dtype=np.int32) for r in rows], int(last_max))


def greedy_lazy(row_ptr, col_idx, capacity, min_redundancy=2) -> SearchResult:
    """Algorithm 3 without a count per pair (C, memory O(|E|)): per-node upper bounds on the best
    redundancy, confirmed by a recount from the definition before every merge.  For graphs whose
    pair map does not fit in memory."""
    return _greedy_c("o3c_greedy", row_ptr, col_idx, capacity, min_redundancy)


def greedy_pairmap(row_ptr, col_idx, capacity, min_redundancy=2) -> SearchResult:
    """Algorithm 3 with the pair-count map and heap of the complexity appendix (C)."""
    return _greedy_c("o3b_greedy", row_ptr, col_idx, capacity, min_redundancy)


def _greedy_c(fn, row_ptr, col_idx, capacity, min_redundancy) -> SearchResult:
    rp, ci = _csr(row_ptr, col_idx)
    n = rp.shape[0] - 1
    cap = int(capacity)
    t1 = np.zeros(max(cap, 1), dtype=np.int32)
    t2 = np.zeros(max(cap, 1), dtype=np.int32)
    tr = np.zeros(max(cap, 1), dtype=np.int32)
    cur_len = np.zeros(max(n, 1), dtype=np.int32)
    cur_idx = np.zeros(max(ci.shape[0], 1), dtype=np.int32)
    fin = np.zeros(1, dtype=np.int32)
    k = getattr(_c(), fn)(n, _ptr(rp), _ptr(ci), cap, int(min_redundancy), _ptr(t1), _ptr(t2), _ptr(tr), _ptr(cur_len), _ptr(cur_idx), _ptr(fin))
    if k < 0:
        raise MemoryError(f"{fn} failed with code {k}")
    trace = np.stack([t1[:k], t2[:k], tr[:k]], axis=1).astype(np.int32).reshape(-1, 3)
    rows = [cur_idx[rp[u]:rp[u] + cur_len[u]].copy() for u in range(n)]
    return SearchResult(n, trace, rows, int(fin[0]))


# --------------------------------------------------------------------------- #
# the run-time layout
# --------------------------------------------------------------------------- #
@dataclass
class CanonicalHag:
    n: int
    num_agg: int
    num_levels: int
    level_ptr: np.ndarray   # int64[L+1]; level l (1-based) = canonical ids n+level_ptr[l-1] .. n+level_ptr[l]-1
    agg_in: np.ndarray      # int32[2*num_agg]; (lo, hi) canonical ids of node n+j
    res_ptr: np.ndarray     # int64[n+1]
    res_idx: np.ndarray     # int32[.]; remaining in-neighbours, ascending canonical id
    t_ptr: np.ndarray       # int64[n+num_agg+1]
    t_idx: np.ndarray       # int32[|E-hat|]; destinations ascending; < n = output row, >= n = aggregation node
    in_degree: np.ndarray   # int32[n]; |N(v)| in the input graph
    creation_to_canonical: np.ndarray  # int32[num_agg]

    @property
    def e_hat(self) -> int:
        return int(2 * self.num_agg + self.res_idx.shape[0])


def canonical_hag(row_ptr, search: SearchResult) -> CanonicalHag:
    """Level of a graph node (as a source) is 0; level of an aggregation node is
    1 + the larger level of its two inputs (the longest path from a source).
    Canonical id = n + rank in the stable sort by (level, creation index)."""
    rp = np.asarray(row_ptr, dtype=np.int64)
    n = search.n
    k = search.num_agg
    level = np.zeros(n + k, dtype=np.int64)
    for j in range(k):
        v1, v2 = int(search.trace[j, 0]), int(search.trace[j, 1])
        level[n + j] = 1 + max(level[v1], level[v2])
    agg_level = level[n:]
    order = np.argsort(agg_level, kind="stable")            # creation indices in canonical order
    c2c = np.empty(k, dtype=np.int32)
    c2c[order] = np.arange(k, dtype=np.int32)
    id_map = np.concatenate([np.arange(n, dtype=np.int64), n + c2c.astype(np.int64)])
    num_levels = int(agg_level.max()) if k else 0
    level_ptr = np.zeros(num_levels + 1, dtype=np.int64)
    if k:
        level_ptr[1:] = np.cumsum(np.bincount(agg_level, minlength=num_levels + 1)[1:])
    agg_in = np.zeros(2 * k, dtype=np.int32)
    for j in range(k):
        a, b = id_map[search.trace[j, 0]], id_map[search.trace[j, 1]]
        pos = c2c[j]
        agg_in[2 * pos], agg_in[2 * pos + 1] = min(a, b), max(a, b)
    res_ptr = np.zeros(n + 1, dtype=np.int64)
    parts = []
    for u in range(n):
        r = np.sort(id_map[search.rows[u].astype(np.int64)])
        parts.append(r)
        res_ptr[u + 1] = res_ptr[u] + r.shape[0]
    res_idx = (np.concatenate(parts) if parts else np.zeros(0)).astype(np.int32)
    # transposed HAG: every edge (source -> destination), grouped by source, destinations ascending
    src = np.concatenate([agg_in.astype(np.int64), res_idx.astype(np.int64)])
    dst = np.concatenate([np.repeat(n + np.arange(k, dtype=np.int64), 2),
                          np.repeat(np.arange(n, dtype=np.int64), np.diff(res_ptr))])
    o = np.lexsort((dst, src))
    t_idx = dst[o].astype(np.int32)
    t_ptr = np.zeros(n + k + 1, dtype=np.int64)
    np.cumsum(np.bincount(src, minlength=n + k), out=t_ptr[1:])
    in_degree = np.diff(rp).astype(np.int32)
    return CanonicalHag(n, k, num_levels, level_ptr, agg_in, res_ptr, res_idx, t_ptr, t_idx, in_degree, c2c)


def expanded_tails(h: CanonicalHag, fwd_cut: int, bwd_cut: int) -> dict:
    """Deep levels evaluated without their intermediate nodes, for GIVEN cuts.

    Forward, cut c (0 <= c <= L): an aggregation node deeper than level c is the
    Aggregate over its cover restricted to ids of level <= c, i.e. its inputs with
    every input deeper than c replaced, recursively, by that input's own list
    (Section 3.1, Eq. 1: aggr(v) aggregates cover(v); with c = 0 the list IS
    cover(v)).  Backward, cut c: a node deeper than c collects the gradient of
    every graph-node output that uses it, directly or through deeper nodes (the
    transitive users over the transposed HAG).  Which cut a library picks is a
    launch heuristic that the paper does not fix: every cut gives the same values,
    so the cut is an input here and only the lists are derived.  Lists are sorted;
    a source reached along several paths would appear several times (it never
    does when the cover condition of Theorem 2 holds)."""
    n, k, L = h.n, h.num_agg, h.num_levels
    if not (0 <= fwd_cut <= L and 0 <= bwd_cut <= L):
        raise ValueError("cut outside 0..num_levels")
    level = np.zeros(n + k, dtype=np.int64)
    for l in range(1, L + 1):
        level[n + h.level_ptr[l - 1]: n + h.level_ptr[l]] = l
    pairs = h.agg_in.reshape(-1, 2)

    fl = {}
    for j in range(int(h.level_ptr[fwd_cut]), k):
        out = []
        for s in pairs[j]:
            s = int(s)
            out.extend([s] if level[s] <= fwd_cut else fl[s])
        fl[n + j] = sorted(out)

    users = {}
    for j in range(k - 1, int(h.level_ptr[bwd_cut]) - 1, -1):
        out = []
        for d in h.t_idx[h.t_ptr[n + j]: h.t_ptr[n + j + 1]]:
            d = int(d)
            out.extend([d] if d < n else users[d])
        users[n + j] = sorted(out)

    def pack(ids, lists):
        ptr = np.zeros(len(ids) + 1, dtype=np.int64)
        flat = []
        for i, w in enumerate(ids):
            flat.extend(lists[w])
            ptr[i + 1] = len(flat)
        return ptr, np.asarray(flat, dtype=np.int32)

    f_ids = [n + j for j in range(int(h.level_ptr[fwd_cut]), k)]
    b_ids = [n + j for j in range(int(h.level_ptr[bwd_cut]), k)]
    ftail_ptr, ftail_idx = pack(f_ids, fl)
    btail_ptr, btail_idx = pack(b_ids, users)
    return dict(fwd_cut=fwd_cut, bwd_cut=bwd_cut, ftail_ptr=ftail_ptr, ftail_idx=ftail_idx,
                btail_ptr=btail_ptr, btail_idx=btail_idx)


def expanded_forward(h: CanonicalHag, x, fwd_cut: int, tails: dict):
    """Algorithm 2 lines 3-6 with the deep levels taken from the given expansion lists:
    levels 1..fwd_cut as pair sums, every deeper node as the sum over its list.  Returns
    the (n + num_agg) x d buffer of a-hat values (fp64); it must equal what the plain level
    order gives, which is how a set of lists from anywhere is checked for validity."""
    x = np.asarray(x, dtype=np.float64)
    n, k = h.n, h.num_agg
    ahat = np.zeros((n + k, x.shape[1]), dtype=np.float64)
    ahat[:n] = x
    j0 = int(h.level_ptr[fwd_cut])
    for j in range(j0):
        ahat[n + j] = ahat[h.agg_in[2 * j]] + ahat[h.agg_in[2 * j + 1]]
    ptr, idx = tails["ftail_ptr"], tails["ftail_idx"]
    deep = np.zeros((k - j0, x.shape[1]), dtype=np.float64)
    for i in range(k - j0):
        deep[i] = ahat[idx[ptr[i]:ptr[i + 1]]].sum(axis=0)      # all ids in a list are of level <= fwd_cut
    ahat[n + j0:] = deep
    return ahat


def transposed_csr(row_ptr, col_idx):
    """Out-neighbour CSR of the input graph (destinations ascending): (t_ptr int64, t_idx int32)."""
    rp, ci = _csr(row_ptr, col_idx)
    n = rp.shape[0] - 1
    dst = np.repeat(np.arange(n, dtype=np.int64), np.diff(rp))
    o = np.lexsort((dst, ci.astype(np.int64)))
    t_ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(ci, minlength=n), out=t_ptr[1:])
    return t_ptr, dst[o].astype(np.int32)


# --------------------------------------------------------------------------- #
# O4: Algorithm 2 over the layout
# --------------------------------------------------------------------------- #
def hag_forward(h: CanonicalHag, x, reduce="sum"):
    x = np.ascontiguousarray(x, dtype=np.float64)
    d = x.shape[1]
    scratch = np.empty((h.n + h.num_agg, d), dtype=np.float64)
    out = np.empty((h.n, d), dtype=np.float64)
    _c().o4_hag_forward(h.n, h.num_agg, _ptr(np.ascontiguousarray(h.agg_in)), _ptr(np.ascontiguousarray(h.res_ptr)),
                        _ptr(np.ascontiguousarray(h.res_idx)), _ptr(np.ascontiguousarray(h.in_degree)), d, _ptr(x),
                        int(reduce == "mean"), _ptr(scratch), _ptr(out))
    return out


def hag_backward(h: CanonicalHag, g, reduce="sum"):
    g = np.ascontiguousarray(g, dtype=np.float64)
    d = g.shape[1]
    scratch = np.empty((max(h.num_agg, 1), d), dtype=np.float64)
    gx = np.empty((h.n, d), dtype=np.float64)
    _c().o4_hag_backward(h.n, h.num_agg, _ptr(np.ascontiguousarray(h.t_ptr)), _ptr(np.ascontiguousarray(h.t_idx)),
                         _ptr(np.ascontiguousarray(h.in_degree)), d, _ptr(g), int(reduce == "mean"), _ptr(scratch), _ptr(gx))
    return gx


def direct_max_forward(row_ptr, col_idx, z, rows=None):
    """a_v = element-wise max over u in N(v) of z_u (zero row for an empty N(v)), fp64.
    ``rows``: optional subset of nodes; the result then has one row per entry."""
    rp, ci = _csr(row_ptr, col_idx)
    z = np.ascontiguousarray(z, dtype=np.float64)
    if rows is None:
        out = np.empty_like(z)
        _c().o6_max_forward(rp.shape[0] - 1, _ptr(rp), _ptr(ci), z.shape[1], _ptr(z), _ptr(out))
        return out
    sel = np.ascontiguousarray(rows, dtype=np.int64)
    out = np.empty((sel.shape[0], z.shape[1]), dtype=np.float64)
    _c().o6_max_forward_rows(rp.shape[0] - 1, _ptr(rp), _ptr(ci), z.shape[1], _ptr(z), _ptr(sel), sel.shape[0], _ptr(out))
    return out


def direct_max_backward(row_ptr, col_idx, z, g, rows=None):
    """gz_u[k] = sum over v with u in N(v) and z_u[k] == a_v[k] of g_v[k].  Returns (gz, T),
    T the same sum over |g| (the scale of the comparison tolerance).  ``rows``: optional subset of
    source nodes u (one result row per entry): only the maxima of their out-neighbours are evaluated."""
    rp, ci = _csr(row_ptr, col_idx)
    z = np.ascontiguousarray(z, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.float64)
    if rows is None:
        a = direct_max_forward(rp, ci, z)
        gz = np.empty_like(z)
        ab = np.empty_like(z)
        _c().o6_max_backward(rp.shape[0] - 1, _ptr(rp), _ptr(ci), z.shape[1], _ptr(z), _ptr(a), _ptr(g), _ptr(gz), _ptr(ab))
        return gz, ab
    t_ptr, t_idx = transposed_csr(rp, ci)                      # out-neighbours v of every u, ascending
    sel = np.asarray(rows, dtype=np.int64)
    gz = np.zeros((sel.shape[0], z.shape[1]), dtype=np.float64)
    ab = np.zeros_like(gz)
    for i, u in enumerate(sel):
        vs = t_idx[t_ptr[u]:t_ptr[u + 1]].astype(np.int64)
        if vs.size == 0:
            continue
        hit = direct_max_forward(rp, ci, z, rows=vs) == z[u]   # v receives from u where u attains v's maximum
        gz[i] = np.where(hit, g[vs], 0.0).sum(axis=0)
        ab[i] = np.where(hit, np.abs(g[vs]), 0.0).sum(axis=0)
    return gz, ab


def hag_max_forward(h: CanonicalHag, z):
    """Algorithm 2 with max.  Returns (out, ahat): ahat has n + num_agg rows, the last
    num_agg being the maxima held by the aggregation nodes."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    d = z.shape[1]
    ahat = np.empty((h.n + h.num_agg, d), dtype=np.float64)
    out = np.empty((h.n, d), dtype=np.float64)
    _c().o7_hag_max_forward(h.n, h.num_agg, _ptr(np.ascontiguousarray(h.agg_in)), _ptr(np.ascontiguousarray(h.res_ptr)),
                            _ptr(np.ascontiguousarray(h.res_idx)), d, _ptr(z), _ptr(ahat), _ptr(out))
    return out, ahat


def hag_max_backward(h: CanonicalHag, z, g):
    """Gradient of hag_max_forward over the transposed HAG."""
    g = np.ascontiguousarray(g, dtype=np.float64)
    out, ahat = hag_max_forward(h, z)
    d = g.shape[1]
    ghat = np.empty((max(h.num_agg, 1), d), dtype=np.float64)
    gz = np.empty((h.n, d), dtype=np.float64)
    _c().o7_hag_max_backward(h.n, h.num_agg, _ptr(np.ascontiguousarray(h.t_ptr)), _ptr(np.ascontiguousarray(h.t_idx)), d,
                             _ptr(ahat), _ptr(out), _ptr(g), _ptr(ghat), _ptr(gz))
    return gz


# --------------------------------------------------------------------------- #
# O5: counters and invariants
# --------------------------------------------------------------------------- #
def counters(row_ptr, h: CanonicalHag) -> dict:
    """Binary aggregations in both forms of the cost function, |E-hat|, and the
    saved-aggregation count f of the Theorem 4 proof."""
    rp = np.asarray(row_ptr, dtype=np.int64)
    e = int(rp[-1])
    deg = np.diff(rp)
    res_deg = np.diff(h.res_ptr)
    aggr_gnn = int(np.maximum(deg - 1, 0).sum())
    aggr_hag_sum_form = int(np.maximum(res_deg - 1, 0).sum()) + h.num_agg * (2 - 1)
    aggr_hag_closed_form = h.e_hat - h.n - h.num_agg
    return dict(n=h.n, e=e, num_agg=h.num_agg, e_hat=h.e_hat, num_levels=h.num_levels,
                aggregations_gnn=aggr_gnn, aggregations_hag=aggr_hag_sum_form,
                aggregations_hag_closed_form=aggr_hag_closed_form,
                closed_form_applies=bool((deg >= 1).all() and (res_deg >= 1).all()),
                saved_f=e - h.e_hat + h.num_agg)


def cover_multiset_ok(row_ptr, col_idx, h: CanonicalHag) -> bool:
    """Theorem 2: cover(v) = N(v) for every graph node, with cover taken as a
    MULTISET (sum needs every source exactly once).  Expands aggregation nodes
    recursively into their input nodes."""
    rp, ci = _csr(row_ptr, col_idx)
    covers = [None] * h.num_agg
    for j in range(h.num_agg):
        parts = []
        for s in (int(h.agg_in[2 * j]), int(h.agg_in[2 * j + 1])):
            parts.append(np.asarray([s], dtype=np.int64) if s < h.n else covers[s - h.n])
        covers[j] = np.concatenate(parts)
    for v in range(h.n):
        parts = []
        for s in h.res_idx[h.res_ptr[v]:h.res_ptr[v + 1]]:
            s = int(s)
            parts.append(np.asarray([s], dtype=np.int64) if s < h.n else covers[s - h.n])
        cov = np.sort(np.concatenate(parts)) if parts else np.zeros(0, dtype=np.int64)
        if not np.array_equal(cov, ci[rp[v]:rp[v + 1]].astype(np.int64)):
            return False
    return True


def replay_trace(row_ptr, col_idx, trace, check_argmax_at=()):
    """Re-run a merge trace from the definition: before merge i, Redundancy(v1, v2)
    counted over all rows must equal the recorded r_i; the rewrite is then applied.
    At the steps in ``check_argmax_at`` the recorded pair is also checked to be the
    arg-max with the lowest-pair-id tie-break, by recounting every node's best
    partner from scratch.  Returns (rows, final_max_redundancy_or_None)."""
    rp, ci = _csr(row_ptr, col_idx)
    n = rp.shape[0] - 1
    trace = np.asarray(trace, dtype=np.int64).reshape(-1, 3)
    k = trace.shape[0]
    lib = _c()
    cur_idx = ci.copy()
    cur_len = np.diff(rp).astype(np.int32)
    counts = np.zeros(n + k + 1, dtype=np.int32)
    part = ctypes.c_int32(0)
    check = set(int(s) for s in check_argmax_at)

    def global_argmax(n_ids):
        best, arg = 0, None
        for a in range(n_ids):
            c = lib.o_max_pair_recount(n, _ptr(rp), _ptr(cur_len), _ptr(cur_idx), n_ids, a, _ptr(counts), ctypes.byref(part))
            if c > best and part.value > a:
                best, arg = int(c), (a, int(part.value))
            elif c > best:
                best, arg = int(c), (int(part.value), a)
        return best, arg

    for i in range(k):
        v1, v2, r = int(trace[i, 0]), int(trace[i, 1]), int(trace[i, 2])
        if not v1 < v2 < n + i:
            raise AssertionError(f"merge {i}: bad pair ({v1},{v2})")
        got = lib.o_count_pair(n, _ptr(rp), _ptr(cur_len), _ptr(cur_idx), v1, v2)
        if got != r or r < 2:
            raise AssertionError(f"merge {i}: recorded redundancy {r}, recount {got}")
        if i in check:
            best, arg = global_argmax(n + i)
            if best != r or arg != (v1, v2):
                raise AssertionError(f"merge {i}: recorded ({v1},{v2}) r={r}, arg-max is {arg} r={best}")
        w = n + i
        for u in range(n):
            row = cur_idx[rp[u]:rp[u] + cur_len[u]]
            i1 = np.searchsorted(row, v1)
            i2 = np.searchsorted(row, v2)
            if i1 < row.shape[0] and row[i1] == v1 and i2 < row.shape[0] and row[i2] == v2:
                keep = row[(row != v1) & (row != v2)]
                m = keep.shape[0]
                cur_idx[rp[u]:rp[u] + m] = keep
                cur_idx[rp[u] + m] = w
                cur_len[u] = m + 1
    final = None
    if -1 in check or k in check:
        final, _ = global_argmax(n + k)
    rows = [cur_idx[rp[u]:rp[u] + cur_len[u]].copy() for u in range(n)]
    return rows, final


def replay_trace_full(row_ptr, col_idx, trace, check_argmax_at=(), min_redundancy=2):
    """The same replay in plain C (oracle.c: o_replay_trace), for traces of any length.

    Before every merge the recorded redundancy is recounted from the definition over the
    current rows; at the steps in ``check_argmax_at`` every pair's redundancy is recounted
    and the recorded pair must be the arg-max with the lowest-pair-id tie-break; a step equal
    to the number of merges recounts once more after the last merge.  Returns a dict:
    ok, failed_step, failure, rows (list of arrays, creation ids), final_max_redundancy
    (None unless the terminal recount was asked for), full_recounts, pair_count_updates."""
    rp, ci = _csr(row_ptr, col_idx)
    n = rp.shape[0] - 1
    tr = np.ascontiguousarray(np.asarray(trace, dtype=np.int32).reshape(-1, 3))
    k = tr.shape[0]
    t1, t2, r = (np.ascontiguousarray(tr[:, j]) for j in range(3))
    steps = np.asarray(sorted(set(int(s) for s in check_argmax_at)), dtype=np.int64)
    cur_len = np.zeros(max(n, 1), dtype=np.int32)
    cur_idx = np.zeros(max(ci.shape[0], 1), dtype=np.int32)
    report = np.zeros(8, dtype=np.int64)
    _c().o_replay_trace(n, _ptr(rp), _ptr(ci), k, _ptr(t1), _ptr(t2), _ptr(r), int(min_redundancy),
                        steps.shape[0], _ptr(steps), _ptr(cur_len), _ptr(cur_idx), _ptr(report))
    what = {1: "bad pair ids", 2: "recorded redundancy differs from the recount", 3: "merge below the stop value",
            4: "another pair has a larger redundancy or comes first", 5: "out of memory"}
    ok = report[0] < 0
    return dict(ok=bool(ok), failed_step=None if ok else int(report[0]), failure=None if ok else what[int(report[1])],
                detail=[int(v) for v in report[5:8]],
                rows=[cur_idx[rp[u]:rp[u] + cur_len[u]].copy() for u in range(n)] if ok else None,
                row_len=cur_len[:n].copy(), row_store=cur_idx,
                final_max_redundancy=None if report[2] < 0 else int(report[2]),
                full_recounts=int(report[3]), pair_count_updates=int(report[4]))


def cover_check_rows(row_ptr, col_idx, trace, row_len, row_store) -> int:
    """Theorem 2 on rows in creation-id space (oracle.c: o_cover_check): every row, with its
    aggregation nodes expanded down to graph nodes, must be N(u) of the input graph with every
    source exactly once.  Returns -1 when all rows pass, else the first failing row."""
    rp, ci = _csr(row_ptr, col_idx)
    tr = np.asarray(trace, dtype=np.int32).reshape(-1, 3)
    t1, t2 = np.ascontiguousarray(tr[:, 0]), np.ascontiguousarray(tr[:, 1])
    rl = np.ascontiguousarray(row_len, dtype=np.int32)
    rs = np.ascontiguousarray(row_store, dtype=np.int32)
    return int(_c().o_cover_check(rp.shape[0] - 1, _ptr(rp), _ptr(ci), tr.shape[0], _ptr(t1), _ptr(t2), _ptr(rl), _ptr(rs)))
