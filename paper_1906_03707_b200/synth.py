"""Seeded synthetic inputs: graphs, features and upstream gradients.

This module only *draws inputs*.  It holds none of the method's arithmetic (no
aggregation, no HAG search, no layout code), so both the CUDA library and the
CPU checker may be fed from it.  Everything is a pure function of its seed
(numpy ``PCG64`` streams), vectorised so that the million-node shape is
produced in seconds.

Graphs are returned as a CSR of IN-neighbours: row ``v`` lists the sources
``u`` that ``v`` aggregates (the edge (u, v) of the paper's HAG definition),
columns sorted ascending and duplicate free, ``row_ptr`` int64, ``col_idx``
int32.  Undirected graphs are symmetrised.

The five ``config*`` functions give the shapes of the paper's workloads
(community structured node-classification graphs with heavy-tailed degrees, a
dense-neighbourhood graph, a block-diagonal batch of small dense graphs, a
million-node scale shape); every one takes size arguments so the tests can draw
the same structure at a fraction of the size.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


# --------------------------------------------------------------------------- #
# containers
# --------------------------------------------------------------------------- #
@dataclass
class Graph:
    """CSR of in-neighbours.  ``row_ptr``: int64[N+1]; ``col_idx``: int32[E]."""

    n: int
    row_ptr: np.ndarray
    col_idx: np.ndarray
    name: str = ""
    meta: dict = field(default_factory=dict)

    @property
    def e(self) -> int:
        return int(self.row_ptr[-1])


@dataclass
class Workload:
    """One benchmark/test case: a graph plus how it is aggregated."""

    graph: Graph
    d: int                 # feature width D
    dtype: str             # "f32" | "bf16" (storage type of x, out, g, gx)
    reduce: str            # "sum" | "mean"
    capacity: int          # |V_A| upper limit handed to the search
    feat_dist: str         # "uniform" | "normal"
    seed: int
    layers: int = 1
    name: str = ""


# --------------------------------------------------------------------------- #
# CSR helpers (input plumbing only)
# --------------------------------------------------------------------------- #
def csr_from_directed_pairs(n: int, src: np.ndarray, dst: np.ndarray, name: str = "", meta=None) -> Graph:
    """Build the in-neighbour CSR from directed edges (src -> dst), dropping duplicates."""
    src = np.asarray(src, dtype=np.int64)
    dst = np.asarray(dst, dtype=np.int64)
    key = dst * np.int64(n) + src
    key.sort()                                        # sorted by (dst, src)
    if key.shape[0] > 1:                              # drop duplicates (what np.unique returns, without its hashing pass)
        keep = np.empty(key.shape[0], dtype=bool)
        keep[0] = True
        np.not_equal(key[1:], key[:-1], out=keep[1:])
        key = key[keep]
    d = key // n
    s = (key - d * n).astype(np.int32)
    counts = np.bincount(d, minlength=n).astype(np.int64)
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    return Graph(n=n, row_ptr=row_ptr, col_idx=s, name=name, meta=dict(meta or {}))


def csr_from_undirected_pairs(n: int, a: np.ndarray, b: np.ndarray, self_loops: bool, name: str = "", meta=None) -> Graph:
    """Symmetrise undirected pairs {a, b} (self pairs dropped), optionally add every self-loop."""
    a = np.asarray(a, dtype=np.int64)
    b = np.asarray(b, dtype=np.int64)
    keep = a != b
    a, b = a[keep], b[keep]
    src = np.concatenate([a, b])
    dst = np.concatenate([b, a])
    if self_loops:
        loops = np.arange(n, dtype=np.int64)
        src = np.concatenate([src, loops])
        dst = np.concatenate([dst, loops])
    return csr_from_directed_pairs(n, src, dst, name=name, meta=meta)


def csr_from_rows(rows) -> Graph:
    """Small hand-written graphs: ``rows[v]`` is the list of in-neighbours of v."""
    n = len(rows)
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    cols = []
    for v, r in enumerate(rows):
        r = sorted(set(int(u) for u in r))
        cols.extend(r)
        row_ptr[v + 1] = len(cols)
    return Graph(n=n, row_ptr=row_ptr, col_idx=np.asarray(cols, dtype=np.int32))


def permute_ids(g: Graph, seed: int) -> Graph:
    """Relabel nodes by a random permutation (locality stress test)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    perm = rng.permutation(g.n).astype(np.int64)
    dst = np.repeat(np.arange(g.n, dtype=np.int64), np.diff(g.row_ptr))
    return csr_from_directed_pairs(g.n, perm[g.col_idx], perm[dst], name=g.name + "+perm", meta=g.meta)


# --------------------------------------------------------------------------- #
# random pieces
# --------------------------------------------------------------------------- #
def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), int(stream)]))


def truncated_power_law(rng: np.random.Generator, n: int, lo: int, hi: int, alpha: float) -> np.ndarray:
    """n iid integers with P(d) proportional to d**-alpha on [lo, hi]."""
    support = np.arange(lo, hi + 1, dtype=np.float64)
    cdf = np.cumsum(support ** (-alpha))
    cdf /= cdf[-1]
    idx = np.searchsorted(cdf, rng.random(n), side="right")
    return (lo + np.minimum(idx, hi - lo)).astype(np.int64)


def _weighted_endpoints(rng, cum_w: np.ndarray, starts: np.ndarray, ends: np.ndarray, group: np.ndarray) -> np.ndarray:
    """For each requested draw (one per entry of ``group``) pick an index in
    [starts[g], ends[g]) with probability proportional to the weights whose
    inclusive cumulative sum is ``cum_w`` (global, over all groups)."""
    base = np.where(starts[group] > 0, cum_w[np.maximum(starts[group], 1) - 1], 0.0)
    top = cum_w[ends[group] - 1]
    r = base + rng.random(group.shape[0]) * (top - base)
    idx = np.searchsorted(cum_w, r, side="right")
    return np.clip(idx, starts[group], ends[group] - 1)


def degree_corrected_communities(
    rng: np.random.Generator,
    n: int,
    member_node: np.ndarray,     # int64[M]  node of each membership, grouped by community
    member_comm: np.ndarray,     # int64[M]  community of each membership, non-decreasing
    member_theta: np.ndarray,    # float64[M] propensity of the node inside that community
    target_deg: np.ndarray,      # int64[n]
    f_in: float,
    f_out: float,
):
    """Degree-corrected planted partition.  Inside each community c place
    round(f_in * S_c / 2) undirected edges (S_c = sum of propensities), each
    endpoint drawn independently with probability proportional to its
    propensity; then round(f_out * sum(target_deg) / 2) edges with both
    endpoints drawn proportionally to target_deg over all nodes.  Returns the
    raw endpoint arrays (self pairs and duplicates still in)."""
    n_comm = int(member_comm.max()) + 1 if member_comm.size else 0
    sizes = np.bincount(member_comm, minlength=n_comm).astype(np.int64)
    ends = np.cumsum(sizes)
    starts = ends - sizes
    cum = np.cumsum(member_theta)
    s_c = np.bincount(member_comm, weights=member_theta, minlength=n_comm)
    m_c = np.rint(f_in * s_c / 2.0).astype(np.int64)
    m_c[sizes < 2] = 0
    group = np.repeat(np.arange(n_comm, dtype=np.int64), m_c)
    ia = _weighted_endpoints(rng, cum, starts, ends, group)
    ib = _weighted_endpoints(rng, cum, starts, ends, group)
    a_in, b_in = member_node[ia], member_node[ib]

    m_out = int(np.rint(f_out * float(target_deg.sum()) / 2.0))
    cum_t = np.cumsum(target_deg.astype(np.float64))
    one = np.zeros(m_out, dtype=np.int64)
    s0 = np.zeros(1, dtype=np.int64)
    e0 = np.full(1, n, dtype=np.int64)
    a_out = _weighted_endpoints(rng, cum_t, s0, e0, one)
    b_out = _weighted_endpoints(rng, cum_t, s0, e0, one)
    return np.concatenate([a_in, a_out]), np.concatenate([b_in, b_out])


# --------------------------------------------------------------------------- #
# the five workload shapes
# --------------------------------------------------------------------------- #
def config1_graph(seed: int = 0, n: int = 1000, comm_size: int = 100, p_in: float = 0.1, p_out: float = 0.001) -> Graph:
    """Planted partition: community = v // comm_size, every pair a<b independently
    with p_in (same community) or p_out; symmetrised; all self-loops added."""
    rng = _rng(seed)
    u = rng.random((n, n))
    comm = np.arange(n) // comm_size
    same = comm[:, None] == comm[None, :]
    upper = np.triu(np.ones((n, n), dtype=bool), k=1)
    hit = upper & (u < np.where(same, p_in, p_out))
    a, b = np.nonzero(hit)
    return csr_from_undirected_pairs(n, a, b, self_loops=True, name="cfg1-planted-partition",
                                     meta=dict(seed=seed, n=n, comm_size=comm_size, p_in=p_in, p_out=p_out))


def config2_graph(seed: int = 1, n: int = 50_000, n_comm: int = 500, d_lo: int = 15, d_hi: int = 1000,
                  alpha: float = 2.0, f_in: float = 0.95, f_out: float = 0.05) -> Graph:
    """Overlapping communities: each node joins k in {1,2,3} distinct communities
    (uniform); target degree from a truncated power law; propensity t_v / k in each
    of its communities; 5 % of the edge mass is placed at random; self-loops added."""
    rng = _rng(seed)
    t = truncated_power_law(rng, n, d_lo, d_hi, alpha)
    n_comm = max(3, int(n_comm))
    k = rng.integers(1, 4, size=n)
    # three distinct communities per node, uniform without replacement; the first k are used
    c0 = rng.integers(0, n_comm, size=n)
    c1 = (c0 + 1 + rng.integers(0, n_comm - 1, size=n)) % n_comm
    c2 = rng.integers(0, n_comm - 2, size=n)
    lo, hi = np.minimum(c0, c1), np.maximum(c0, c1)
    c2 = c2 + (c2 >= lo)
    c2 = c2 + (c2 >= hi)
    c = np.stack([c0, c1, c2], axis=1)
    slot = np.arange(3)[None, :] < k[:, None]
    node = np.repeat(np.arange(n, dtype=np.int64)[:, None], 3, axis=1)[slot]
    comm = c[slot].astype(np.int64)
    theta = np.repeat((t / k)[:, None], 3, axis=1)[slot]
    order = np.lexsort((node, comm))
    a, b = degree_corrected_communities(rng, n, node[order], comm[order], theta[order], t, f_in, f_out)
    return csr_from_undirected_pairs(n, a, b, self_loops=True, name="cfg2-overlapping-communities",
                                     meta=dict(seed=seed, n=n, n_comm=n_comm, d_lo=d_lo, d_hi=d_hi, alpha=alpha,
                                               f_in=f_in, f_out=f_out))


def config3_graph(seed: int = 2, n: int = 233_000, n_comm: int = 50, d_lo: int = 27, d_hi: int = 1400,
                  alpha: float = 2.0, f_in: float = 0.90, f_out: float = 0.10) -> Graph:
    """Dense-neighbourhood node-classification shape: equal communities in
    contiguous id blocks, power-law target degrees, 10 % inter-community edge
    mass, self-loops added."""
    rng = _rng(seed)
    t = truncated_power_law(rng, n, d_lo, d_hi, alpha)
    block = -(-n // n_comm)
    comm = (np.arange(n, dtype=np.int64) // block)
    node = np.arange(n, dtype=np.int64)
    a, b = degree_corrected_communities(rng, n, node, comm, t.astype(np.float64), t, f_in, f_out)
    return csr_from_undirected_pairs(n, a, b, self_loops=True, name="cfg3-dense-neighbourhoods",
                                     meta=dict(seed=seed, n=n, n_comm=n_comm, d_lo=d_lo, d_hi=d_hi, alpha=alpha,
                                               f_in=f_in, f_out=f_out))


def config4_graph(seed: int = 3, n_graphs: int = 5000, graph_size: int = 100, p: float = 0.5) -> Graph:
    """Graph-classification batch: disjoint Erdos-Renyi graphs, block diagonal, no self-loops."""
    rng = _rng(seed)
    iu, ju = np.triu_indices(graph_size, k=1)
    a_parts, b_parts = [], []
    chunk = max(1, 4_000_000 // max(1, iu.size))
    for g0 in range(0, n_graphs, chunk):
        g1 = min(n_graphs, g0 + chunk)
        hit = rng.random((g1 - g0, iu.size)) < p
        gi, pi = np.nonzero(hit)
        base = (g0 + gi).astype(np.int64) * graph_size
        a_parts.append(base + iu[pi])
        b_parts.append(base + ju[pi])
    a = np.concatenate(a_parts) if a_parts else np.zeros(0, np.int64)
    b = np.concatenate(b_parts) if b_parts else np.zeros(0, np.int64)
    n = n_graphs * graph_size
    return csr_from_undirected_pairs(n, a, b, self_loops=False, name="cfg4-er-batch",
                                     meta=dict(seed=seed, n_graphs=n_graphs, graph_size=graph_size, p=p))


def config5_graph(seed: int = 4, n: int = 1_000_000, n_comm: int = 2000, s_lo: int = 60, s_hi: int = 20_000,
                  s_alpha: float = 1.8, d_lo: int = 15, d_hi: int = 800, alpha: float = 2.0,
                  f_in: float = 0.95, f_out: float = 0.05) -> Graph:
    """Scale shape: community sizes iid from a truncated power law, rescaled to
    sum to n, contiguous id blocks; power-law target degrees; 5 % random edge
    mass; no self-loops."""
    rng = _rng(seed)
    raw = truncated_power_law(rng, n_comm, s_lo, s_hi, s_alpha).astype(np.float64)
    sizes = np.maximum(2, np.floor(raw * (n / raw.sum()))).astype(np.int64)
    # hand the rounding remainder to the largest communities, one node each
    diff = int(n - sizes.sum())
    order = np.argsort(-sizes, kind="stable")
    i = 0
    while diff != 0:
        j = order[i % n_comm]
        step = 1 if diff > 0 else -1
        if sizes[j] + step >= 2:
            sizes[j] += step
            diff -= step
        i += 1
    comm = np.repeat(np.arange(n_comm, dtype=np.int64), sizes)
    t = truncated_power_law(rng, n, d_lo, d_hi, alpha)
    node = np.arange(n, dtype=np.int64)
    a, b = degree_corrected_communities(rng, n, node, comm, t.astype(np.float64), t, f_in, f_out)
    return csr_from_undirected_pairs(n, a, b, self_loops=False, name="cfg5-scale",
                                     meta=dict(seed=seed, n=n, n_comm=n_comm, s_lo=s_lo, s_hi=s_hi, s_alpha=s_alpha,
                                               d_lo=d_lo, d_hi=d_hi, alpha=alpha, f_in=f_in, f_out=f_out))


def clique_union_graph(seed: int, n: int, n_groups: int, g_lo: int, g_hi: int, g_alpha: float = 2.0,
                       self_loops: bool = True) -> Graph:
    """Bipartite-projection shape (co-authorship / shared-commenter style): every
    group is a clique over its members; group sizes from a truncated power law,
    members drawn uniformly (a member drawn twice for one group counts once)."""
    rng = _rng(seed)
    sizes = truncated_power_law(rng, n_groups, g_lo, min(g_hi, n), g_alpha)
    members = rng.integers(0, n, size=int(sizes.sum()))
    starts = np.concatenate([[0], np.cumsum(sizes)[:-1]])
    a_parts, b_parts = [], []
    for sz in np.unique(sizes):
        rows = np.nonzero(sizes == sz)[0]
        block = members[starts[rows][:, None] + np.arange(sz)[None, :]]       # one group per row
        iu, ju = np.triu_indices(int(sz), k=1)
        a_parts.append(block[:, iu].ravel())
        b_parts.append(block[:, ju].ravel())
    a = np.concatenate(a_parts) if a_parts else np.zeros(0, np.int64)
    b = np.concatenate(b_parts) if b_parts else np.zeros(0, np.int64)
    return csr_from_undirected_pairs(n, a, b, self_loops=self_loops, name="clique-union",
                                     meta=dict(seed=seed, n=n, n_groups=n_groups, g_lo=g_lo, g_hi=g_hi))


def random_digraph(seed: int, n: int, p: float, undirected: bool, self_loops: bool) -> Graph:
    """Tiny uniform random graphs for brute-force checks."""
    rng = _rng(seed)
    hit = rng.random((n, n)) < p
    np.fill_diagonal(hit, False)
    if undirected:
        hit = np.triu(hit, 1)
        a, b = np.nonzero(hit)
        return csr_from_undirected_pairs(n, a, b, self_loops=self_loops, name="tiny-undirected")
    src, dst = np.nonzero(hit)
    if self_loops:
        loops = np.arange(n)
        src, dst = np.concatenate([src, loops]), np.concatenate([dst, loops])
    return csr_from_directed_pairs(n, src, dst, name="tiny-directed")


# --------------------------------------------------------------------------- #
# features and upstream gradients
# --------------------------------------------------------------------------- #
def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 values rounded to the nearest bf16 (ties to even), returned as fp32."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """The uint16 bf16 payload of values that are already bf16-representable."""
    return (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def features(seed: int, n: int, d: int, dist: str, dtype: str = "f32", stream: int = 0) -> np.ndarray:
    """n x d fp32 matrix; ``dist`` in {"uniform" (U[-1,1]), "normal" (N(0,1)),
    "int" (integers in [-4,4], exact in any summation order)}.  For dtype
    "bf16" the values are rounded to bf16 first (still returned as fp32)."""
    rng = _rng(seed, 1 + stream)
    if dist == "uniform":
        x = rng.random((n, d), dtype=np.float32) * np.float32(2.0) - np.float32(1.0)
    elif dist == "normal":
        x = rng.standard_normal((n, d), dtype=np.float32)
    elif dist == "int":
        x = rng.integers(-4, 5, size=(n, d)).astype(np.float32)
    else:
        raise ValueError(dist)
    if dtype == "bf16":
        x = round_to_bf16(x)
    elif dtype != "f32":
        raise ValueError(dtype)
    return x


def upstream_grad(seed: int, n: int, d: int, dist: str, dtype: str = "f32") -> np.ndarray:
    """Independent stream (seed + 1000) with the same distribution as the features."""
    return features(seed + 1000, n, d, dist, dtype, stream=7)


# --------------------------------------------------------------------------- #
# the named workloads (full size by default, ``scale`` < 1 shrinks them)
# --------------------------------------------------------------------------- #
def workload(index: int, scale: float = 1.0, capacity_frac: float = 0.25) -> Workload:
    """Workload ``index`` (1-5 are the named shapes, 6 a clique-union graph).  ``scale`` shrinks the node count while keeping the
    generator, degree law, community size and feature shape."""
    if index == 1:
        n = max(200, int(round(1000 * scale)) // 100 * 100)
        g = config1_graph(seed=0, n=n)
        return Workload(g, 16, "f32", "sum", g.n // 4 if capacity_frac == 0.25 else int(g.n * capacity_frac),
                        "uniform", 0, name="cfg1")
    if index == 2:
        n = max(1000, int(round(50_000 * scale)))
        g = config2_graph(seed=1, n=n, n_comm=max(2, int(round(500 * scale))))
        return Workload(g, 64, "f32", "mean", int(g.n * capacity_frac), "normal", 1, name="cfg2")
    if index == 3:
        n_comm = max(1, int(round(50 * scale)))
        g = config3_graph(seed=2, n=4660 * n_comm, n_comm=n_comm)
        return Workload(g, 128, "f32", "sum", int(g.n * capacity_frac), "normal", 2, layers=2, name="cfg3")
    if index == 4:
        g = config4_graph(seed=3, n_graphs=max(2, int(round(5000 * scale))))
        return Workload(g, 64, "f32", "sum", int(g.n * capacity_frac), "uniform", 3, name="cfg4")
    if index == 5:
        n = max(2000, int(round(1_000_000 * scale)))
        g = config5_graph(seed=4, n=n, n_comm=max(2, int(round(2000 * scale))),
                          s_hi=max(120, min(20_000, n // 4)))
        return Workload(g, 256, "bf16", "sum", int(g.n * capacity_frac), "normal", 4, name="cfg5")
    if index == 6:
        # beyond the five named shapes: a union of cliques (co-authorship / shared-commenter projection), the regime
        # of the paper's collaboration datasets: a deep hierarchy and a several-fold reduction of reads
        n = max(2000, int(round(100_000 * scale)))
        g = clique_union_graph(seed=5, n=n, n_groups=max(20, int(round(30_000 * scale))), g_lo=2,
                               g_hi=max(20, min(400, n // 50)), g_alpha=2.3)
        return Workload(g, 64, "f32", "sum", int(g.n * capacity_frac), "normal", 5, name="clique-union")
    raise ValueError(index)
