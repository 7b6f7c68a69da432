"""Host-side helpers for running the path on several GPUs.

The aggregation of disjoint graphs (a graph-classification batch) or of
independent workloads needs no exchange between GPUs: every rank builds the HAG
of its own units and runs the same kernels.  What remains to be agreed between
ranks is bookkeeping only: who owns which units, and the timing reduction
(max over ranks) behind a throughput figure.  ``torch.distributed`` is used for
that reduction alone; there is no data-path collective.
"""
from __future__ import annotations

import numpy as np

from .synth import Graph


def shard_range(n_units: int, rank: int, world: int):
    """Contiguous, balanced split of ``n_units`` independent units: (first, count)
    for ``rank``.  The first ``n_units % world`` ranks get one extra unit."""
    if world <= 0 or not 0 <= rank < world:
        raise ValueError("bad rank/world")
    base, extra = divmod(int(n_units), int(world))
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def shard_columns(d: int, rank: int, world: int, elem_bytes: int = 4):
    """Feature-column split of one graph over ranks: (first column, count) for ``rank``.
    Aggregation treats every column alike, so each rank can hold the whole structure and
    a slice of the columns of x and needs no exchange.  Slices are multiples of 16 bytes
    (the kernels' row granularity); ranks at the end may get nothing when D is small."""
    if d <= 0 or (d * elem_bytes) % 16:
        raise ValueError("row size must be a positive multiple of 16 bytes")
    per16 = 16 // elem_bytes if elem_bytes <= 16 else 1
    first, count = shard_range(d // per16, rank, world)
    return first * per16, count * per16


def shard_block_diagonal(g: Graph, graph_size: int, rank: int, world: int) -> Graph:
    """The sub-batch of a block-diagonal batch of equal-size graphs owned by ``rank``,
    re-indexed from 0.  Raises if an edge leaves its block (the batch would not be
    a set of independent problems)."""
    if g.n % graph_size:
        raise ValueError("node count is not a multiple of graph_size")
    first_g, count_g = shard_range(g.n // graph_size, rank, world)
    lo, hi = first_g * graph_size, (first_g + count_g) * graph_size
    e0, e1 = int(g.row_ptr[lo]), int(g.row_ptr[hi])
    cols = g.col_idx[e0:e1].astype(np.int64)
    rows = np.repeat(np.arange(lo, hi, dtype=np.int64), np.diff(g.row_ptr[lo:hi + 1]))
    if cols.size and not np.array_equal(cols // graph_size, rows // graph_size):
        raise ValueError("an edge crosses graphs: not block diagonal")
    row_ptr = (g.row_ptr[lo:hi + 1] - g.row_ptr[lo]).astype(np.int64)
    return Graph(n=hi - lo, row_ptr=row_ptr, col_idx=(cols - lo).astype(np.int32),
                 name=f"{g.name}[rank {rank}/{world}]", meta=dict(g.meta, first_node=lo))


def max_over_ranks(value: float, device=None) -> float:
    """MAX-reduce a per-rank time over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    """SUM-reduce per-rank unit counts (bytes, rows) over the default process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, ms_this_rank: float, device=None) -> float:
    """Whole-job throughput: the units all ranks processed / the slowest rank's time (units per second)."""
    total = sum_over_ranks(units_this_rank, device)
    ms = max_over_ranks(ms_this_rank, device)
    return total / (ms * 1e-3)
